"""The allocation-free decode-attention entry point against the regular one.

Some users of the library cannot allocate device memory (a frozen memory pool, a host
process that budgets all of HBM itself), so they cannot hand fkv_init_cache a workspace.
fkv_decode_attn_dense_noalloc serves them from a fixed scratch array inside the library.
This test calls it through the C ABI twice in a row - the second call finds the first
call's leftovers in the scratch - and holds each result against fkv_decode_attn on a
cache filled with the same K and V, and against the CPU oracle's attention over the same
bytes.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_03203_b200 import binding, workloads as wl
from util import bits, bits_to_f64

pytestmark = pytest.mark.gpu

ATTN_TOL = 2e-2


def _close(a, b):
    a, b = bits_to_f64(bits(a)), bits_to_f64(bits(b))
    allowed = np.maximum(ATTN_TOL, 2.0 ** -7 * np.abs(b))   # one bf16 step where that is coarser than 2e-2
    return bool(np.all(np.abs(a - b) <= allowed))


def _close_to_oracle(got, q, K, V, g):
    """Every KV head against the CPU oracle's attention over the same bytes, element by element."""
    gb, qb, Kb, Vb = bits(got), bits(q), bits(K), bits(V)
    for h in range(K.shape[0]):
        ref, ref64 = oracle.attend(qb[h * g:(h + 1) * g], Kb[h], Vb[h])
        err = np.abs(bits_to_f64(gb[h * g:(h + 1) * g]) - bits_to_f64(ref))
        if not np.all(err <= np.maximum(ATTN_TOL, 2.0 ** -7 * np.abs(ref64))):
            return False
    return True


# The entry point takes one split per 256 pairs, at most 16: the cases sit on both sides of the first
# split boundary (255 / 256 / 257), of the point where the split count stops growing (4096 / 4097), far
# beyond it (20000: many rows per warp and split), and at the smallest sizes (one pair, one query head).
@pytest.mark.parametrize("n,g,D,Hkv", [(3000, 4, 128, 8), (777, 7, 128, 4), (100, 4, 64, 2), (1, 1, 128, 1),
                                       (255, 4, 128, 2), (256, 8, 128, 2), (257, 1, 64, 3), (4096, 4, 128, 2),
                                       (4097, 8, 64, 2), (5000, 8, 64, 16), (20000, 4, 128, 2)])
def test_noalloc_matches_cache_path_twice(n, g, D, Hkv):
    w = wl.Workload("noalloc", 1, Hkv, g, D, (n,), (1 << 20,), 0, 41, "channel_lognormal")
    cache = binding.from_workload(w)
    K, V, A, pos = (t.cuda() for t in wl.layer_inputs(w, 0, 0))
    cache.prefill(0, 0, K, V, A, pos)
    out_static = torch.empty((Hkv * g, D), dtype=torch.bfloat16, device="cuda")
    for call in range(2):
        q = wl.queries(w, 0, step=call).cuda()                 # [1][Hq][D], different each call
        ref = cache.decode_attn(0, q)[0]
        got = binding.decode_attn_dense_noalloc(q[0].contiguous(), K, V, g, out=out_static)
        torch.cuda.synchronize()
        assert _close(got, ref), (n, g, D, call)
        assert _close_to_oracle(got, q[0], K, V, g), (n, g, D, call)
    assert cache.device_status()[0] == 0


def test_noalloc_rejects_unaligned_rows():
    q = torch.zeros((4, 128), dtype=torch.bfloat16, device="cuda")
    buf = torch.zeros((1 * 8 * 128 + 1,), dtype=torch.bfloat16, device="cuda")
    kv = buf[1:].view(1, 8, 128)                               # starts 2 bytes past an aligned address
    with pytest.raises(binding.FkvError) as e:
        binding.decode_attn_dense_noalloc(q, kv, kv, 4)
    assert e.value.code == -1


def test_noalloc_rejects_sizes_beyond_its_scratch():
    q = torch.zeros((17 * 4, 128), dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros((17, 8, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.FkvError) as e:
        binding.decode_attn_dense_noalloc(q, kv, kv, 4)        # 17 KV heads > 16
    assert e.value.code == -3
    q9 = torch.zeros((2 * 9, 128), dtype=torch.bfloat16, device="cuda")
    kv2 = torch.zeros((2, 8, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.FkvError) as e:
        binding.decode_attn_dense_noalloc(q9, kv2, kv2, 9)     # group of 9 > 8
    assert e.value.code == -3
