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


def test_overlapped_decode_steps_are_reproducible_at_full_occupancy():
    """The decode step of the Qwen3-4B-shaped configuration at B = 8192 puts three CTAs of consecutive layers'
    launches on every SM, and an engine refills the SAME k / v / q buffers before every token.  Three repeats
    of the same eight tokens must agree bit for bit (a page slot released before its last read, or an input
    read at the wrong time, shows up as a run-to-run difference), and sampled heads must match the oracle."""
    import dataclasses
    w = wl.config(3, budget=8192)
    w = dataclasses.replace(w, lens=tuple(min(n, b) for n, b in zip(w.lens, w.budgets)))
    L, T = w.num_layers, 8
    pages = binding.pages_for(w, L, 64)
    need = binding.workspace_bytes_for(w, L, num_pages=pages, max_tokens=max(w.lens) + 64)
    free, _ = torch.cuda.mem_get_info()
    if need * 2.5 > free:   # workspace, its snapshot and generator scratch
        pytest.skip(f"needs {need * 2.5 / 1e9:.1f} GB of device memory")
    cache = binding.from_workload(w, L, num_pages=pages, max_tokens=max(w.lens) + 64)
    for l in range(L):
        K, V, A, pos = wl.layer_inputs(w, l, 0, "cuda")
        cache.prefill(l, 0, K, V, A, pos)
    snap = cache.snapshot()
    gen = torch.Generator(device="cuda")
    kd = torch.empty((L, 1, w.num_kv_heads, w.head_dim), device="cuda", dtype=torch.bfloat16)
    vd = torch.empty_like(kd)
    qd = torch.empty((L, 1, w.num_q_heads, w.head_dim), device="cuda", dtype=torch.bfloat16)

    def run():
        cache.restore(snap)
        gen.manual_seed(7)
        outs, qs = [], []
        for _ in range(T):
            for buf in (kd, vd, qd):
                buf.copy_(torch.randn(buf.shape, device="cuda", generator=gen))
            outs.append(cache.decode_step(kd, vd, qd))
            qs.append(qd.clone())
        torch.cuda.synchronize()
        return torch.stack(outs), torch.stack(qs)

    first, qs = run()
    for _ in range(2):
        again, _ = run()
        assert torch.equal(first, again)
    assert cache.device_status()[0] == 0
    g, n0 = w.group_size, w.lens[0]
    ob, qb = bits(first), bits(qs)
    for l, h in [(0, 0), (5, 3), (18, 5), (35, 7)]:
        k2, v2, _, _ = (bits(x) if x.dtype == torch.bfloat16 else x for x in cache.export_head(l, 0, h))
        for t in (0, 3, T - 1):
            n = n0 + t + 1
            ref, ref64 = oracle.attend(qb[t, l, 0, h * g:(h + 1) * g], k2[:n], v2[:n])
            err = np.abs(bits_to_f64(ob[t, l, 0, h * g:(h + 1) * g]) - bits_to_f64(ref))
            assert (err <= np.maximum(ATTN_TOL, 2.0 ** -7 * np.abs(ref64))).all(), (l, h, t, err.max())


@pytest.mark.parametrize("lens,Hkv", [((3000,), 2), ((700, 5000), 1)])
def test_replayed_per_layer_calls_match_ordinary_calls(lens, Hkv):
    """The per-layer entry point (fkv_append_decode_attn) recorded layer by layer and replayed.  At these sizes its
    launches are the ones whose splits form a thread-block cluster and merge through distributed shared memory; every
    replay is compared with the same calls made directly on a second cache, and the last one with the oracle."""
    L, steps = 3, 40
    w = wl.Workload("graph_layer", L, Hkv, 4, 128, lens, (1 << 20,) * len(lens), 0, 27, "channel_lognormal")
    a = Loaded(w, max_tokens=max(lens) + steps + 8)
    b = Loaded(w, max_tokens=max(lens) + steps + 8)
    ks, vs, qs = _static_inputs(w, L)
    out_g = torch.zeros_like(qs)
    a.cache.append_decode_attn(0, ks[0], vs[0], qs[0], out_g[0])   # first launches (set-up) before the capture
    b.cache.append_decode_attn(0, ks[0], vs[0], qs[0])
    torch.cuda.synchronize()
    snap = a.cache.snapshot()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for l in range(L):
            a.cache.append_decode_attn(l, ks[l], vs[l], qs[l], out_g[l])
    torch.cuda.synchronize()
    a.cache.restore(snap)
    for step in range(steps):
        graph.replay()
        out_e = torch.stack([b.cache.append_decode_attn(l, ks[l], vs[l], qs[l]) for l in range(L)])
        torch.cuda.synchronize()
        assert torch.equal(out_g, out_e), step          # same launches, same splits: the same bits
    a.cache.sync_lengths()
    for l in range(L):
        assert a.cache.lengths(l) == b.cache.lengths(l)
    og, qb, g = bits(out_g), bits(qs), w.group_size
    for l in range(L):
        for s in range(w.batch):
            for h in range(Hkv):
                ka, va, _, _ = a.export(l, s, h)
                ref, ref64 = oracle.attend(qb[l, s, h * g:(h + 1) * g], ka, va)
                err = np.abs(bits_to_f64(og[l, s, h * g:(h + 1) * g]) - bits_to_f64(ref))
                assert np.all(err <= np.maximum(ATTN_TOL, 2.0 ** -7 * np.abs(ref64)))
    assert a.cache.device_status()[0] == 0 and b.cache.device_status()[0] == 0
