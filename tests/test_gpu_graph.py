"""GPU tests: the decode step recorded into a CUDA graph and replayed.

A replay advances the lengths on the device only, so the kernel itself has to cope with segments that have
outgrown what the host saw when the launch was recorded (more pages per split) and with appends past the
capacity (skipped, status bit set).  Every replay is compared with the same step made by ordinary calls on a
second cache, and the last one with the oracle.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
from harness import Loaded
from paper_2602_03203_b200 import binding, workloads as wl
from util import bits, bits_to_f64

pytestmark = pytest.mark.gpu

ATTN_TOL = 2e-2


def _static_inputs(w, L):
    ks = torch.stack([wl.new_kv(w, l, 0)[0] for l in range(L)]).cuda()
    vs = torch.stack([wl.new_kv(w, l, 0)[1] for l in range(L)]).cuda()
    qs = torch.stack([wl.queries(w, l, 0) for l in range(L)]).cuda()
    return ks, vs, qs


def _record(cache, ks, vs, qs, out):
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        cache.decode_step(ks, vs, qs, out)
    torch.cuda.synchronize()
    return graph


@pytest.mark.parametrize("lens", [(40, 7, 16), (1000, 333, 4096)])
def test_replayed_decode_step_matches_ordinary_calls(lens):
    L = 2
    w = wl.Workload("graph", L, 2, 4, 128, lens, (1 << 20,) * 3, 0, 24, "normal")
    steps = 150   # the shortest segments grow by several pages: far past the recorded pages per split
    a = Loaded(w, max_tokens=max(lens) + steps + 8)
    b = Loaded(w, max_tokens=max(lens) + steps + 8)
    ks, vs, qs = _static_inputs(w, L)
    out_g = torch.zeros_like(qs)
    snap = a.cache.snapshot()
    graph = _record(a.cache, ks, vs, qs, out_g)     # recording does not run the step ...
    a.cache.restore(snap)                           # ... but the host's lengths moved: put both back
    for step in range(steps):
        graph.replay()
        out_e = b.cache.decode_step(ks, vs, qs)
        torch.cuda.synchronize()
        # Same arithmetic per page; only the split boundaries (hence the order of the final sums) may differ.
        err = (out_g.float() - out_e.float()).abs().max().item()
        assert err <= ATTN_TOL, (step, err)
    a.cache.sync_lengths()
    for l in range(L):
        assert a.cache.lengths(l) == b.cache.lengths(l)
        assert a.cache.lengths(l) == [n + steps for n in lens]
    assert a.cache.device_status()[0] == 0 and b.cache.device_status()[0] == 0
    # Content and last output against the oracle.
    og, qb = bits(out_g), bits(qs)
    g = w.group_size
    for l in range(L):
        for s in range(w.batch):
            for h in range(w.num_kv_heads):
                ka, va, _, pa = a.export(l, s, h)
                kb, vb, _, pb = b.export(l, s, h)
                assert np.array_equal(ka, kb) and np.array_equal(va, vb) and np.array_equal(pa, pb)
                assert ka.shape[0] == lens[s] + steps
                ref, ref64 = oracle.attend(qb[l, s, h * g:(h + 1) * g], ka, va)
                err = np.abs(bits_to_f64(og[l, s, h * g:(h + 1) * g]) - bits_to_f64(ref))
                assert (err <= np.maximum(ATTN_TOL, 2.0 ** -7 * np.abs(ref64))).all()


def test_replay_past_capacity_is_skipped_and_flagged():
    L = 1
    lens = (30, 5)
    w = wl.Workload("graphcap", L, 2, 4, 64, lens, (1 << 20,) * 2, 0, 24, "normal")
    ld = Loaded(w, max_tokens=48)
    cap = ld.cache.cap
    ks, vs, qs = _static_inputs(w, L)
    out = torch.zeros_like(qs)
    snap = ld.cache.snapshot()
    graph = _record(ld.cache, ks, vs, qs, out)
    ld.cache.restore(snap)
    for _ in range(cap - lens[0] + 5):   # sequence 0 hits the capacity, sequence 1 does not
        graph.replay()
    torch.cuda.synchronize()
    status, _ = ld.cache.device_status()
    assert status == binding.DEV_CAPACITY
    ld.cache.sync_lengths()
    assert ld.cache.lengths(0) == [cap, lens[1] + cap - lens[0] + 5]
    # The full sequence still attends over its cap pairs; the output is finite and matches the oracle.
    og, qb = bits(out), bits(qs)
    g = w.group_size
    for s in range(2):
        for h in range(w.num_kv_heads):
            k2, v2, _, _ = ld.export(0, s, h)
            ref, ref64 = oracle.attend(qb[0, s, h * g:(h + 1) * g], k2, v2)
            err = np.abs(bits_to_f64(og[0, s, h * g:(h + 1) * g]) - bits_to_f64(ref))
            assert (err <= np.maximum(ATTN_TOL, 2.0 ** -7 * np.abs(ref64))).all()
