"""The R-KV baseline score (Appendix E.2) on the GPU against the CPU oracle, through the C ABI.

The score's similarity term is the n x n contraction of a segment's keys on the tensor cores (pairs of
CTAs that multiply as one; single CTAs for launches of four tiles or fewer); the cases span one pair,
lengths around the 128-row operand tiles and the units of two and four tiles, ragged last tiles, several
segments of different lengths per launch, ranges of CTA pairs that cut through segments, both head
dimensions, duplicate and zero keys.  Tolerance: 1e-3 on the scores (the figure every score of this library is held to); selection and
compaction from the GPU's own scores are bit-exact.
"""
import numpy as np
import pytest
import torch

import oracle
from harness import Loaded, kept_set_within_band
from paper_2602_03203_b200 import binding, workloads as wl
from util import bits, npf

pytestmark = pytest.mark.gpu

SCORE_TOL = 1e-3


@pytest.mark.parametrize("lens,g,D,Hkv", [((1, 2), 4, 64, 2), ((100, 128), 4, 128, 2), ((129, 255), 1, 128, 1),
                                          ((256, 257), 7, 128, 2), ((300, 700, 1000, 17), 4, 128, 2),
                                          ((1500,), 8, 64, 3), ((2049, 640), 2, 128, 4),
                                          ((512, 513, 1024, 1025), 2, 128, 1), ((511, 769), 4, 64, 2)])
def test_rkv_scores_match_oracle(lens, g, D, Hkv):
    w = wl.Workload("rkv", 2, Hkv, g, D, lens, tuple(1 << 20 for _ in lens), 0, 51, "channel_lognormal")
    ld = Loaded(w)
    worst = 0.0
    for l in range(w.num_layers):
        got = npf(ld.cache.score_rkv(l))
        snap = npf(ld.cache.score_rkv(l, 1.0, 0.0))
        for s, n in enumerate(lens):
            for h in range(Hkv):
                K, V, A, _ = ld.head(l, s, h)
                ref = oracle.score_rkv(K, A, g)
                worst = max(worst, float(np.abs(got[s, h, :n] - ref).max()))
                # similarity weight 0: the SnapKV score, bit for bit
                assert np.array_equal(snap[s, h, :n], oracle.score_feature(A, g, oracle.SNAPKV_COLUMN))
    assert worst <= SCORE_TOL, worst
    assert ld.cache.device_status()[0] == 0


def test_rkv_pairs_of_ctas_with_ragged_ranges():
    # 332 tiles over 74 pairs of CTAs: five tiles a pair, so units of four tiles and of one, ranges that start and
    # end in the middle of segments, pairs whose second CTA has no rows.  Sampled rows: the oracle takes them one by
    # one (first and last rows, unit and tile boundaries of each segment, random ones).
    lens = (9000, 7000, 5000)
    w = wl.Workload("rkv_pairs", 1, 2, 4, 128, lens, tuple(1 << 20 for _ in lens), 0, 57, "channel_lognormal")
    ld = Loaded(w)
    got = npf(ld.cache.score_rkv(0))
    rng = np.random.default_rng(11)
    for s, n in enumerate(lens):
        rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, 383, 384, 511, 512, 639, 640, n - 129, n - 128, n - 1],
                                         rng.integers(0, n, 120)])).astype(np.int32)
        for h in range(w.num_kv_heads):
            K, V, A, _ = ld.head(0, s, h)
            ref = oracle.score_rkv(K, A, w.group_size, rows=rows)
            assert np.abs(got[s, h, rows] - ref).max() <= SCORE_TOL, (s, h)
    assert ld.cache.device_status()[0] == 0


def test_rkv_duplicate_and_zero_keys():
    # Exact duplicate rows (config 5's tie pattern) have a twin at cosine 1; a zero key has cosine 0 with all.
    w = wl.shrink(wl.config(5), num_layers=1, max_len=900, batch=1)
    ld = Loaded(w)
    K, V, A, pos = ld.head(0, 0, 0)
    got = npf(ld.cache.score_rkv(0, 0.0, 1.0))[0, 0, :w.lens[0]]
    ref = oracle.score_rkv(K, A, w.group_size, 0.0, 1.0)
    assert np.abs(got - ref).max() <= SCORE_TOL
    _, inv, cnt = np.unique(K, axis=0, return_inverse=True, return_counts=True)
    dup = cnt[inv.reshape(-1)] > 1
    assert dup.any() and np.all(np.abs(got[dup] + 1.0) <= 1e-5)
    w2 = wl.Workload("rkv0", 1, 1, 2, 64, (40,), (1 << 20,), 0, 52, "normal")
    c = binding.from_workload(w2)
    K2, V2, A2, p2 = wl.layer_inputs(w2, 0, 0)
    K2[0, 7] = 0
    c.prefill(0, 0, K2.cuda(), V2.cuda(), A2.cuda(), p2.cuda())
    got2 = npf(c.score_rkv(0, 0.0, 1.0))[0, 0, :40]
    assert got2[7] == 0.0
    assert np.abs(got2 - oracle.score_rkv(bits(K2[0]), npf(A2[0]), 2, 0.0, 1.0)).max() <= SCORE_TOL


@pytest.mark.parametrize("cfg,kw", [(1, {}), (2, dict(num_layers=2, max_len=1100)), (4, dict(num_layers=1, max_len=900, batch=3))])
def test_evict_rkv_end_to_end(cfg, kw):
    w = wl.shrink(wl.config(cfg), **kw) if kw else wl.config(cfg)
    ld = Loaded(w)
    scores = {l: npf(ld.cache.score_rkv(l)) for l in range(ld.L)}
    ld.cache.evict_rkv()
    for l in range(ld.L):
        for s in range(w.batch):
            n, B, R = w.lens[s], w.budgets[s], w.recent_keep
            for h in range(w.num_kv_heads):
                K, V, A, pos = ld.head(l, s, h)
                k2, v2, a2, p2 = ld.export(l, s, h)
                kept_g = np.searchsorted(pos, p2).astype(np.int32)
                assert np.array_equal(kept_g, oracle.select(scores[l][s, h, :n], B, R))     # bit-exact from the same scores
                phi = oracle.score_rkv(K, A, w.group_size)
                assert kept_set_within_band(phi, oracle.select(phi, B, R), kept_g, n, B, R, SCORE_TOL)
                Ko, Vo, Ao, po = oracle.compact(K, V, A, pos, kept_g)
                assert np.array_equal(k2, Ko) and np.array_equal(v2, Vo) and np.array_equal(a2, Ao) and np.array_equal(p2, po)
    assert ld.cache.device_status()[0] == 0


def test_rkv_one_layer_of_the_32k_configuration():
    # 8 KV heads x 32768 pairs (one layer of config 3): 275 GFLOP per head.  The oracle computes 96 sampled
    # rows per head one by one (first and last rows, tile and unit boundaries, random ones).
    w = wl.config(3)
    c = binding.from_workload(w, 1)
    K, V, A, pos = wl.layer_inputs(w, 0, 0, "cuda")
    c.prefill(0, 0, K, V, A, pos)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    c.score_rkv(0)
    ev[0].record(); got = c.score_rkv(0); ev[1].record(); torch.cuda.synchronize()
    ms = ev[0].elapsed_time(ev[1])
    n = w.lens[0]
    flops = 2.0 * n * n * w.head_dim * w.num_kv_heads
    print(f"R-KV score of one layer: {ms:.2f} ms, {flops / ms / 1e9:.0f} TFLOP/s")
    got = npf(got)
    rng = np.random.default_rng(7)
    rows = np.unique(np.concatenate([[0, 1, 127, 128, 255, 256, 257, n - 129, n - 128, n - 1], rng.integers(0, n, 86)])).astype(np.int32)
    Kb, Ab = bits(K), npf(A)
    for h in range(w.num_kv_heads):
        ref = oracle.score_rkv(Kb[h], Ab[h], w.group_size, rows=rows)
        assert np.abs(got[0, h, rows] - ref).max() <= SCORE_TOL
    assert c.device_status()[0] == 0


def test_rkv_with_an_empty_sequence_and_per_sequence_budgets():
    # Three sequence slots, the middle one never filled; the other two with their own budgets.
    w = wl.Workload("rkv_e", 1, 2, 4, 128, (400, 300, 650), (1 << 20, 1 << 20, 1 << 20), 16, 53, "normal")
    c = binding.from_workload(w)
    host = {}
    for s in (0, 2):
        K, V, A, pos = wl.layer_inputs(w, 0, s)
        c.prefill(0, s, K.cuda(), V.cuda(), A.cuda(), pos.cuda())
        host[s] = (bits(K), npf(A), npf(pos))
    c.set_budget(0, 100); c.set_budget(2, 333)
    sc = npf(c.score_rkv(0))
    c.evict_rkv(0)
    assert c.lengths(0) == [100, 0, 333]
    for s, B in ((0, 100), (2, 333)):
        Kb, A, pos = host[s]
        n = w.lens[s]
        for h in range(2):
            assert np.abs(sc[s, h, :n] - oracle.score_rkv(Kb[h], A[h], 4)).max() <= SCORE_TOL
            _, _, _, p2 = c.export_head(0, s, h)
            assert np.array_equal(npf(p2), pos[oracle.select(sc[s, h, :n], B, 16)])
    assert c.device_status()[0] == 0
