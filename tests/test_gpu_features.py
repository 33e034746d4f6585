"""Attention-feature maintenance (Appendix B.1) against the oracle: the library records the decode
queries of a chunk and recomputes every pair's window and cumulative features at the eviction."""
import numpy as np
import pytest
import torch

import oracle
from harness import kept_set_within_band
from paper_2602_03203_b200 import binding, workloads as wl
from util import bits, npf

pytestmark = pytest.mark.gpu

FEAT_ATOL, FEAT_RTOL = 2e-6, 2e-3     # probabilities <= 1; bf16 products accumulated in fp32 vs fp64
SCORE_TOL = 1e-3


def _run_chunk(w, W, steps, L=None):
    """Prefill, then `steps` fused append+attention tokens; returns the cache and the host-side history."""
    L = L or w.num_layers
    c = binding.from_workload(w, L, feature_window=W)
    st = {}
    for l in range(L):
        c.load_scorers(l, *wl.scorer_params(w, l))
        for s in range(w.batch):
            K, V, A, pos = wl.layer_inputs(w, l, s)
            c.prefill(l, s, K.cuda(), V.cuda(), A.cuda(), pos.cuda())
            for h in range(w.num_kv_heads):
                st[(l, s, h)] = dict(K=bits(K)[h], V=bits(V)[h], A=npf(A)[h].copy(), q=[], nv=[])
    g = w.group_size
    for step in range(steps):
        for l in range(L):
            k, v = wl.new_kv(w, l, step)
            q = wl.queries(w, l, step)
            c.append_decode_attn(l, k.cuda(), v.cuda(), q.cuda())
            kb, vb, qb = bits(k), bits(v), bits(q)
            for s in range(w.batch):
                for h in range(w.num_kv_heads):
                    d = st[(l, s, h)]
                    d["K"] = np.concatenate([d["K"], kb[s, h][None]]); d["V"] = np.concatenate([d["V"], vb[s, h][None]])
                    d["A"] = np.concatenate([d["A"], np.zeros((1, d["A"].shape[1]), np.float32)])
                    d["q"].append(qb[s, h * g:(h + 1) * g]); d["nv"].append(len(d["K"]))
    return c, st


def _expected(d, W):
    q = np.stack(d["q"][-W:]); nv = np.array(d["nv"][-W:], np.int32)     # the ring keeps the last W queries
    return oracle.features(d["K"], q, nv, d["A"])


@pytest.mark.parametrize("g,D,W,steps", [(4, 128, 64, 40), (4, 128, 32, 45), (7, 128, 40, 40), (4, 64, 64, 33),
                                         (1, 128, 16, 7), (8, 64, 24, 50), (2, 64, 8, 13), (4, 128, 8, 5)])
def test_update_features_matches_oracle(g, D, W, steps):
    w = wl.Workload("feat", 2, 2, g, D, (100, 37), (1 << 20,) * 2, 0, 51, "normal")
    c, st = _run_chunk(w, W, steps)
    for l in range(2):
        c.update_features(l)
    for (l, s, h), d in st.items():
        _, _, a2, _ = c.export_head(l, s, h)
        exp = _expected(d, W)
        got = npf(a2)
        assert got.shape == exp.shape
        assert np.all(np.abs(got - exp) <= FEAT_ATOL + FEAT_RTOL * np.abs(exp)), (l, s, h, np.abs(got - exp).max())
    assert c.device_status()[0] == 0


@pytest.mark.parametrize("g,D,W,hkv,lens,steps", [
    # all four heads' records resident, four accumulators, four 32-query chunks per row, 4 tiles per CTA
    (4, 128, 128, 4, (2700, 2300, 2500, 1900, 2900, 2100), 128),
    # more than 128 queries: two accumulators shared by two warpgroups each, records streamed per tile
    (4, 128, 256, 4, (1300, 1100, 1500, 900, 1250, 1400, 1000, 1350), 256),
    # odd group (the last head of a tile is multiplied alone), narrow accumulators
    (7, 128, 64, 2, (5100, 4700, 5300, 4900), 64),
    # head_dim 64, three chunks per row
    (4, 64, 96, 4, (2600, 2200, 3000, 2400, 2800), 96),
    # one and two heads per group: a statistics slot is reused only after several segments
    (1, 128, 64, 8, (1500, 700, 300, 1100, 200, 900), 64),
    (2, 64, 32, 8, (1300, 500, 800, 1700, 150, 1000), 32),
    # more tokens than the ring holds (slot order is not time order) and a partial last chunk: the general path
    (4, 128, 64, 4, (2100, 1700, 2500, 1300), 90),
    (4, 128, 128, 4, (2100, 1700, 2500, 1300), 50),
])
def test_update_features_many_tiles(g, D, W, hkv, lens, steps):
    # Enough tiles that every CTA of the feature kernel walks several of them, crosses segment and sequence
    # boundaries and reuses its shared-memory stages and tensor-memory accumulators.  With steps = W (a whole number
    # of 32-query chunks, ring not wrapped) all tiles but the last of a segment take the unmasked path.
    w = wl.Workload("featbig", 1, hkv, g, D, lens, (1 << 20,) * len(lens), 0, 54, "normal")
    c = binding.from_workload(w, 1, feature_window=W, max_tokens=max(lens) + steps + 16)
    c.load_scorers(0, *wl.scorer_params(w, 0))
    st = {}
    for s in range(w.batch):
        K, V, A, pos = wl.layer_inputs(w, 0, s)
        c.prefill(0, s, K.cuda(), V.cuda(), A.cuda(), pos.cuda())
        for h in range(hkv):
            n = lens[s]
            Kf = np.zeros((n + steps, D), np.uint16); Kf[:n] = bits(K)[h]
            Af = np.zeros((n + steps, 6 * g), np.float32); Af[:n] = npf(A)[h]
            st[(s, h)] = dict(K=Kf, A=Af, q=np.zeros((steps, g, D), np.uint16), n=n)
    for step in range(steps):
        k, v = wl.new_kv(w, 0, step)
        q = wl.queries(w, 0, step)
        c.append_decode_attn(0, k.cuda(), v.cuda(), q.cuda())
        kb, qb = bits(k), bits(q)
        for (s, h), d in st.items():
            d["K"][d["n"] + step] = kb[s, h]
            d["q"][step] = qb[s, h * g:(h + 1) * g]
    c.update_features(0)
    assert c.device_status()[0] == 0
    # a sample of segments: first, last, and those in between where CTA ranges change segment
    keys = sorted(st.keys())
    for (s, h) in keys[::max(1, len(keys) // 9)] + [keys[-1]]:
        d = st[(s, h)]
        nv = (d["n"] + 1 + np.arange(steps)).astype(np.int32)
        exp = oracle.features(d["K"], d["q"][-W:], nv[-W:], d["A"])     # the ring keeps the last W queries
        _, _, a2, _ = c.export_head(0, s, h)
        got = npf(a2)
        assert got.shape == exp.shape
        bad = np.abs(got - exp) > FEAT_ATOL + FEAT_RTOL * np.abs(exp)
        assert not bad.any(), (s, h, np.argwhere(bad)[:4], np.abs(got - exp).max())


def test_no_recorded_query_leaves_features_alone():
    w = wl.Workload("feat0", 1, 2, 4, 128, (200,), (100,), 0, 52, "normal")
    c, st = _run_chunk(w, 32, 0)
    c.update_features(0)
    c.evict(0)                       # one-shot compression after prefill: the prefilled features are scored
    for h in range(2):
        d = st[(0, 0, h)]
        W1, b1, W2, b2 = (npf(t)[h] for t in wl.scorer_params(w, 0))
        phi = oracle.score(d["K"], d["V"], d["A"], W1, b1, W2, float(b2))
        kept = oracle.select(phi, 100, 0)
        _, _, a2, p2 = c.export_head(0, 0, h)
        assert kept_set_within_band(phi, kept, npf(p2), 200, 100, 0, SCORE_TOL)
        assert np.array_equal(npf(a2), d["A"][npf(p2)])


def test_decode_evict_cycle_with_maintained_features():
    # Two chunks of L tokens with an eviction after each (the protocol of Section 3.1, R = L): the scorer
    # sees features the library derived from its own record; the oracle is fed the same queries.
    B, Lev = 128, 32
    w = wl.Workload("featcyc", 1, 2, 4, 128, (B,), (B,), Lev, 53, "channel_lognormal")
    c = binding.from_workload(w, feature_window=Lev)
    c.load_scorers(0, *wl.scorer_params(w, 0))
    K, V, A, pos = wl.layer_inputs(w, 0, 0)
    c.prefill(0, 0, K.cuda(), V.cuda(), A.cuda(), pos.cuda())
    st = {h: dict(K=bits(K)[h], V=bits(V)[h], A=npf(A)[h].copy(), pos=npf(pos).copy()) for h in range(2)}
    g = w.group_size
    W1, b1, W2, b2 = (npf(t) for t in wl.scorer_params(w, 0))
    for chunk in range(2):
        qs = {h: [] for h in range(2)}; nvs = {h: [] for h in range(2)}
        for step in range(Lev):
            k, v = wl.new_kv(w, 0, chunk * Lev + step); q = wl.queries(w, 0, chunk * Lev + step)
            c.append_decode_attn(0, k.cuda(), v.cuda(), q.cuda())
            for h in range(2):
                d = st[h]
                d["K"] = np.concatenate([d["K"], bits(k)[0, h][None]]); d["V"] = np.concatenate([d["V"], bits(v)[0, h][None]])
                d["A"] = np.concatenate([d["A"], np.zeros((1, 6 * g), np.float32)])
                d["pos"] = np.concatenate([d["pos"], [d["pos"][-1] + 1]]).astype(np.int32)
                qs[h].append(bits(q)[0, h * g:(h + 1) * g]); nvs[h].append(len(d["K"]))
        c.evict(0)
        assert c.lengths(0) == [B]
        for h in range(2):
            d = st[h]
            A1 = oracle.features(d["K"], np.stack(qs[h]), np.array(nvs[h], np.int32), d["A"])
            phi = oracle.score(d["K"], d["V"], A1, W1[h], b1[h], W2[h], float(b2[h]))
            kept = oracle.select(phi, B, Lev)
            _, _, a2, p2 = c.export_head(0, 0, h)
            kept_g = np.searchsorted(d["pos"], npf(p2)).astype(np.int32)
            assert kept_set_within_band(phi, kept, kept_g, len(phi), B, Lev, SCORE_TOL)
            got = npf(a2)
            assert np.all(np.abs(got - A1[kept_g]) <= FEAT_ATOL + FEAT_RTOL * np.abs(A1[kept_g]))
            st[h] = dict(K=d["K"][kept_g], V=d["V"][kept_g], A=got.copy(), pos=d["pos"][kept_g])   # follow the GPU's state
    assert c.device_status()[0] == 0


@pytest.mark.parametrize("column", [oracle.H2O_COLUMN, oracle.SNAPKV_COLUMN])
def test_baseline_eviction_on_maintained_features(column):
    # H2O / SnapKV (Appendix E.2) on the library's own features: a chunk of decoding, then an eviction
    # whose score is a feature column.  No scorer is loaded.  The kept set follows from the refreshed
    # features the library exports; those features are checked against the oracle's.
    B, Lev = 96, 32
    w = wl.Workload("base", 1, 2, 4, 128, (B, 70), (B, B), 8, 54, "normal")
    c = binding.from_workload(w, feature_window=Lev)
    st = {}
    for s in range(2):
        K, V, A, pos = wl.layer_inputs(w, 0, s)
        c.prefill(0, s, K.cuda(), V.cuda(), A.cuda(), pos.cuda())
        for h in range(2):
            st[(s, h)] = dict(K=bits(K)[h], A=npf(A)[h].copy(), q=[], nv=[])
    g = w.group_size
    for step in range(Lev):
        k, v = wl.new_kv(w, 0, step); q = wl.queries(w, 0, step)
        c.append_decode_attn(0, k.cuda(), v.cuda(), q.cuda())
        for (s, h), d in st.items():
            d["K"] = np.concatenate([d["K"], bits(k)[s, h][None]])
            d["A"] = np.concatenate([d["A"], np.zeros((1, 6 * g), np.float32)])
            d["q"].append(bits(q)[s, h * g:(h + 1) * g]); d["nv"].append(len(d["K"]))
    c.update_features(0)
    feats = {key: npf(c.export_head(0, key[0], key[1])[2]) for key in st}
    c.evict_by_feature(column, 0)
    assert c.lengths(0) == [B, B]
    for (s, h), d in st.items():
        exp = oracle.features(d["K"], np.stack(d["q"]), np.array(d["nv"], np.int32), d["A"])
        assert np.all(np.abs(feats[(s, h)] - exp) <= FEAT_ATOL + FEAT_RTOL * np.abs(exp))
        n = len(d["K"])
        # NOTE the eviction refreshes the features once more (the chunk is still open after update_features):
        # window columns are recomputed (same values), the cumulative columns move again.
        again = oracle.features(d["K"], np.stack(d["q"]), np.array(d["nv"], np.int32), feats[(s, h)])
        _, _, a2, p2 = c.export_head(0, s, h)
        kept = oracle.select(oracle.score_feature(again, g, column), B, 8)
        phi = oracle.score_feature(again, g, column)
        assert kept_set_within_band(phi, kept, npf(p2), n, B, 8, 1e-5)
        assert npf(p2)[-8:].tolist() == list(range(n - 8, n))
    assert c.device_status()[0] == 0


def test_baseline_eviction_bit_exact_on_given_features():
    # With the features given (no window), the baseline score is a pure function of the stored rows:
    # the kept list must equal the oracle's, bit for bit.
    w = wl.Workload("base2", 2, 2, 7, 64, (500, 333), (200, 100), 16, 55, "normal")
    c = binding.from_workload(w)
    hold = {}
    for l in range(2):
        for s in range(2):
            K, V, A, pos = wl.layer_inputs(w, l, s)
            c.prefill(l, s, K.cuda(), V.cuda(), A.cuda(), pos.cuda())
            hold[(l, s)] = npf(A)
    c.evict_by_feature(oracle.H2O_COLUMN)
    for (l, s), A in hold.items():
        for h in range(2):
            kept = oracle.select(oracle.score_feature(A[h], 7, oracle.H2O_COLUMN), w.budgets[s], 16)
            assert np.array_equal(npf(c.export_head(l, s, h)[3]), kept)
    assert c.device_status()[0] == 0
