"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element.

Tolerances:
  scores          max abs error <= 1e-3 (fp32 accumulation of bf16 inputs vs fp64)
  selection       bit-exact given identical scores
  compaction      bit-exact rows and positions
  end to end      kept sets differ only at pairs within 1e-3 of the (B - r)-th oracle score
  attention       max abs error <= 2e-2 on bf16 outputs
"""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from harness import Loaded, kept_set_within_band
from paper_2602_03203_b200 import binding, workloads as wl
from util import bits, bits_to_f64, npf

pytestmark = pytest.mark.gpu

SCORE_TOL = 1e-3
# N(0,1) inputs and fp32 weights below 0.1: sums of about 2D products of magnitude <= 0.3 accumulated in fp32
# (2^-24 relative per step), weights carried to 2^-17 relative: errors of a few 1e-6.
SCORE_TOL_FP32_WEIGHTS = 3e-5
ATTN_TOL = 2e-2


def small(idx, **kw):
    """Reduced copies of the five configs: same per-segment structure, oracle-sized."""
    presets = {
        1: dict(),
        2: dict(num_layers=2, max_len=1500),
        3: dict(num_layers=2, max_len=2100),
        4: dict(num_layers=1, max_len=1700, batch=4),
        5: dict(num_layers=1, max_len=2200, batch=2),
    }
    p = dict(presets[idx]); p.update(kw)
    return wl.shrink(wl.config(idx), **p) if p else wl.config(idx)


# ------------------------------------------------------------------ layout round trip
@pytest.mark.parametrize("cfg", [1, 4])
def test_prefill_export_roundtrip(cfg):
    w = small(cfg, num_layers=1, max_len=333)   # ragged: not a multiple of the page size
    ld = Loaded(w)
    for s in range(w.batch):
        assert ld.cache.lengths(0)[s] == w.lens[s]
        for h in range(w.num_kv_heads):
            K, V, A, pos = ld.head(0, s, h)
            k2, v2, a2, p2 = ld.export(0, s, h)
            assert np.array_equal(K, k2) and np.array_equal(V, v2)
            assert np.array_equal(A, a2) and np.array_equal(pos, p2)
    assert ld.cache.device_status()[0] == 0


def test_append_rows_and_positions():
    w = small(1, max_len=30)
    ld = Loaded(w)
    n0 = w.lens[0]
    ks, vs = [], []
    for step in range(20):   # crosses a page boundary
        k, v = wl.new_kv(w, 0, step)
        ld.cache.append(0, k.cuda(), v.cuda())
        ks.append(bits(k)); vs.append(bits(v))
    assert ld.cache.lengths(0)[0] == n0 + 20
    for h in range(w.num_kv_heads):
        k2, v2, a2, p2 = ld.export(0, 0, h)
        K, V, A, pos = ld.head(0, 0, h)
        assert np.array_equal(k2[:n0], K) and np.array_equal(v2[:n0], V)
        assert np.array_equal(k2[n0:], np.stack([x[0, h] for x in ks]))
        assert np.array_equal(v2[n0:], np.stack([x[0, h] for x in vs]))
        assert np.all(a2[n0:] == 0)
        assert p2.tolist() == list(range(n0 + 20))   # NULL pos continues from the last position
    assert ld.cache.device_status()[0] == 0


# ------------------------------------------------------------------ kernel 1: scores
@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_score_parity(cfg):
    w = small(cfg)
    ld = Loaded(w)
    worst = 0.0
    for l in range(ld.L):
        got = npf(ld.cache.score(l))
        for s in range(w.batch):
            n = w.lens[s]
            for h in range(w.num_kv_heads):
                K, V, A, _ = ld.head(l, s, h)
                ref = oracle.score(K, V, A, *ld.weights(l, h), act=w.activation)
                worst = max(worst, float(np.abs(got[s, h, :n] - ref).max()))
    assert worst <= SCORE_TOL, worst
    assert ld.cache.device_status()[0] == 0


@pytest.mark.parametrize("g,D", [(1, 64), (2, 128), (3, 64), (5, 128), (6, 64), (8, 128), (8, 64)])
def test_score_group_sizes_and_head_dims(g, D):
    # Feature widths 6g that are and are not multiples of the 8-column tf32 steps (the column after the last
    # feature is the position id and must never be read as one), both head dimensions, ring sizes that follow
    # from the page size; three segments of different lengths so that every CTA crosses segment boundaries.
    w = wl.Workload("gd", 1, 3, g, D, (700, 33, 1234), (1 << 20,) * 3, 0, 61, "channel_lognormal")
    ld = Loaded(w)
    got = npf(ld.cache.score(0))
    worst = 0.0
    for s, n in enumerate(w.lens):
        for h in range(w.num_kv_heads):
            K, V, A, _ = ld.head(0, s, h)
            ref = oracle.score(K, V, A, *ld.weights(0, h))
            worst = max(worst, float(np.abs(got[s, h, :n] - ref).max()))
    assert worst <= SCORE_TOL, worst
    assert ld.cache.device_status()[0] == 0


@pytest.mark.parametrize("act", [binding.ACT_SILU, binding.ACT_GELU_TANH, binding.ACT_SIGMOID])
def test_score_other_activations(act):
    w = dataclasses.replace(small(1), activation=act)
    ld = Loaded(w)
    got = npf(ld.cache.score(0))
    for h in range(w.num_kv_heads):
        K, V, A, _ = ld.head(0, 0, h)
        ref = oracle.score(K, V, A, *ld.weights(0, h), act=act)
        assert np.abs(got[0, h, :w.lens[0]] - ref).max() <= SCORE_TOL


def _score_with_weights(w, W1, b1, W2, b2):
    """Scores of config-1 data under the given scorer of every head: (GPU fp32, oracle fp32)."""
    ld = Loaded(w)
    for h in range(w.num_kv_heads):
        ld.cache.load_scorer(0, h, torch.from_numpy(W1[h]), torch.from_numpy(b1[h]), torch.from_numpy(W2[h]), float(b2[h]))
    got = npf(ld.cache.score(0))
    ref = np.stack([oracle.score(*ld.head(0, 0, h)[:3], W1[h], b1[h], W2[h], float(b2[h])) for h in range(w.num_kv_heads)])
    assert ld.cache.device_status()[0] == 0
    return got[0, :, :w.lens[0]], ref, ld


def test_score_weights_half_way_between_bf16_values():
    # Appendix B.1 gives W1 no precision, so weights arrive as fp32.  Here every K/V weight lies EXACTLY half-way
    # between two neighbouring bf16 values (17 significant bits): stored as a single bf16 it would be off by
    # 2^-9 relative whichever way it is rounded, and the scores by ~1e-3; stored as rounding + remainder it is
    # exact, and what is left is fp32 accumulation (~1e-6).  A dropped, mis-signed or truncated remainder fails.
    w = small(1)
    rng = np.random.default_rng(5)
    Hk, X, H, D = w.num_kv_heads, w.x_dim, w.scorer_hidden, w.head_dim
    W1 = rng.uniform(-1, 1, (Hk, X, H)).astype(np.float32) / np.float32(np.sqrt(X))
    kv = W1[:, :2 * D].view(np.uint32)
    W1[:, :2 * D] = ((kv & np.uint32(0xFFFF0000)) | np.uint32(0x8000)).view(np.float32)
    b1 = rng.uniform(-0.1, 0.1, (Hk, H)).astype(np.float32)
    W2 = rng.uniform(-0.25, 0.25, (Hk, H)).astype(np.float32)
    b2 = rng.uniform(-0.25, 0.25, Hk).astype(np.float32)
    got, ref, ld = _score_with_weights(w, W1, b1, W2, b2)
    assert np.abs(got - ref).max() <= SCORE_TOL_FP32_WEIGHTS, np.abs(got - ref).max()
    # the same weights rounded to ONE bf16 value (to nearest even) must be measurably worse in the oracle itself,
    # or the case would prove nothing
    W1r = W1.copy()
    W1r[:, :2 * D] = torch.from_numpy(W1[:, :2 * D].copy()).to(torch.bfloat16).float().numpy()
    worse = np.stack([oracle.score(*ld.head(0, 0, h)[:3], W1r[h], b1[h], W2[h], float(b2[h])) for h in range(Hk)])
    assert np.abs(worse - ref).max() > 10 * SCORE_TOL_FP32_WEIGHTS


def test_score_plain_fp32_weights_tight():
    # Unrounded U(+-1/sqrt(fan_in)) weights, as a trainer hands them over: far inside 1e-3.
    w = small(1)
    ld = Loaded(w)
    got = npf(ld.cache.score(0))
    for h in range(w.num_kv_heads):
        K, V, A, _ = ld.head(0, 0, h)
        W1 = ld.weights(0, h)[0]
        assert np.any(torch.from_numpy(W1[:2 * w.head_dim].copy()).to(torch.bfloat16).float().numpy() != W1[:2 * w.head_dim])
        ref = oracle.score(K, V, A, *ld.weights(0, h))
        assert np.abs(got[0, h, :w.lens[0]] - ref).max() <= SCORE_TOL_FP32_WEIGHTS


def test_score_duplicates_tie_bit_for_bit():
    # Config 5 injects exact duplicate rows; their scores must be identical bit patterns
    # (the scorer may not depend on where a row sits in a tile).
    w = small(5)
    ld = Loaded(w)
    got = npf(ld.cache.score(0))
    K, V, A, _ = ld.head(0, 0, 0)
    rows = np.concatenate([K.view(np.uint16).astype(np.uint32), V.astype(np.uint32), A.view(np.uint32)], axis=1)
    _, inv, cnt = np.unique(rows, axis=0, return_inverse=True, return_counts=True)
    dup_groups = np.where(cnt > 1)[0]
    assert len(dup_groups) > 0
    sc = got[0, 0, :w.lens[0]].view(np.uint32)
    for gidx in dup_groups:
        members = np.where(inv == gidx)[0]
        assert len(set(sc[members].tolist())) == 1


# ------------------------------------------------------------------ kernel 2: selection (bit-exact)
def _select_case(n, B, R, scores_fn, batch=2, Hkv=2):
    w = wl.Workload("sel", 1, Hkv, 4, 64, (n,) * batch, (B,) * batch, R, 11, "normal")
    ld = Loaded(w)
    cap = ld.cache.cap
    rng = np.random.default_rng(n * 31 + B * 7 + R)
    sc = np.full((batch, Hkv, cap), np.nan, np.float32)
    for s in range(batch):
        for h in range(Hkv):
            sc[s, h, :n] = scores_fn(rng, n)
    idx, cnt = ld.cache.select(0, torch.from_numpy(sc).cuda())
    idx, cnt = npf(idx), npf(cnt)
    for s in range(batch):
        for h in range(Hkv):
            ref = oracle.select(sc[s, h, :n], B, R)
            assert cnt[s, h] == len(ref)
            assert np.array_equal(idx[s, h, :len(ref)], ref), (n, B, R, s, h)
    assert ld.cache.device_status()[0] == 0


def _normal(rng, n):
    return rng.standard_normal(n).astype(np.float32)


def _ties(rng, n):
    return (np.round(rng.standard_normal(n) * 4) / 4).astype(np.float32)


def _special(rng, n):
    x = rng.standard_normal(n).astype(np.float32)
    for val in (np.nan, -0.0, 0.0, np.inf, -np.inf, 1e-40, -1e-40):
        x[rng.integers(0, n, max(1, n // 50))] = val
    return x


@pytest.mark.parametrize("n,B,R", [(512, 256, 0), (512, 256, 32), (5000, 1234, 0), (4097, 4096, 0), (9000, 2048, 256),
                                   (300, 300, 0), (200, 300, 16), (777, 100, 100), (777, 100, 500), (17, 1, 0),
                                   (4099, 3, 1)])
@pytest.mark.parametrize("fn", [_normal, _ties, _special])
def test_select_bit_exact(n, B, R, fn):
    _select_case(n, B, R, fn)


def test_select_all_equal_and_few_distinct():
    _select_case(3000, 1000, 10, lambda rng, n: np.ones(n, np.float32))
    _select_case(3000, 1000, 0, lambda rng, n: rng.integers(0, 2, n).astype(np.float32))
    _select_case(3000, 2999, 0, lambda rng, n: -np.abs(rng.standard_normal(n)).astype(np.float32))


# ------------------------------------------------------------------ kernel 3: compaction (bit-exact)
@pytest.mark.parametrize("cfg", [1, 4])
def test_compact_bit_exact(cfg):
    w = small(cfg, num_layers=1, max_len=1111)
    ld = Loaded(w)
    cap = ld.cache.cap
    rng = np.random.default_rng(3)
    idx = np.full((w.batch, w.num_kv_heads, cap), -1, np.int32)
    cnt = np.zeros((w.batch, w.num_kv_heads), np.int32)
    for s in range(w.batch):
        for h in range(w.num_kv_heads):
            kept = oracle.select(rng.standard_normal(w.lens[s]).astype(np.float32), w.budgets[s], w.recent_keep)
            idx[s, h, :len(kept)] = kept
            cnt[s, h] = len(kept)
    free0 = ld.cache.device_status()[1]
    ld.cache.compact(0, torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda())
    for s in range(w.batch):
        assert ld.cache.lengths(0)[s] == min(w.budgets[s], w.lens[s])
        for h in range(w.num_kv_heads):
            K, V, A, pos = ld.head(0, s, h)
            ref = oracle.compact(K, V, A, pos, idx[s, h, :cnt[s, h]])
            got = ld.export(0, s, h)
            for a, b in zip(ref, got):
                assert np.array_equal(a, b)
            assert np.all(np.diff(got[3]) > 0)
    bits_, free1 = ld.cache.device_status()
    assert bits_ == 0
    old = sum(-(-n // 16) for n in w.lens) * w.num_kv_heads
    new = sum(-(-min(b, n) // 16) for b, n in zip(w.budgets, w.lens)) * w.num_kv_heads
    assert free1 - free0 == old - new    # pages of the old layout went back to the pool


# ------------------------------------------------------------------ evict end to end
@pytest.mark.parametrize("cfg,all_layers", [(1, True), (2, True), (3, False), (4, True), (5, False)])
def test_evict_end_to_end(cfg, all_layers):
    w = small(cfg)
    ld = Loaded(w)
    layers = list(range(ld.L))
    gpu_scores = {l: npf(ld.cache.score(l)) for l in layers}
    if all_layers:
        ld.cache.evict(binding.ALL_LAYERS)
    else:
        for l in layers:
            ld.cache.evict(l)
    for l in layers:
        for s in range(w.batch):
            n, B = w.lens[s], w.budgets[s]
            assert ld.cache.lengths(l)[s] == min(B, n)
            for h in range(w.num_kv_heads):
                K, V, A, pos = ld.head(l, s, h)
                phi = oracle.score(K, V, A, *ld.weights(l, h), act=w.activation)
                kept_o = oracle.select(phi, B, w.recent_keep)
                k2, v2, a2, p2 = ld.export(l, s, h)
                assert len(p2) == min(B, n) and np.all(np.diff(p2) > 0)
                kept_g = np.searchsorted(pos, p2).astype(np.int32)
                assert np.array_equal(pos[kept_g], p2)
                # bit-exact given identical scores: the oracle's selection from the GPU's own scores
                assert np.array_equal(kept_g, oracle.select(gpu_scores[l][s, h, :n], B, w.recent_keep))
                # end to end: differences only inside the tolerance band around the cut
                assert kept_set_within_band(phi, kept_o, kept_g, n, B, w.recent_keep, SCORE_TOL)
                # rows moved intact
                assert np.array_equal(k2, K[kept_g]) and np.array_equal(v2, V[kept_g])
                assert np.array_equal(a2, A[kept_g])
    assert ld.cache.device_status()[0] == 0
    # evicting again at the budget is a no-op
    launches = ld.cache.launch_count()
    ld.cache.evict(binding.ALL_LAYERS)
    assert ld.cache.launch_count() == launches


# ------------------------------------------------------------------ kernel 4: attention
def _attn_check(ld, layer, step=0):
    w = ld.w
    q = wl.queries(w, layer, step)
    out = ld.cache.decode_attn(layer, q.cuda())
    torch.cuda.synchronize()
    out_b, qb = bits(out), bits(q)
    worst = 0.0
    g = w.group_size
    for s in range(w.batch):
        for h in range(w.num_kv_heads):
            k2, v2, _, _ = ld.export(layer, s, h)
            ref, ref64 = oracle.attend(qb[s, h * g:(h + 1) * g], k2, v2)
            err = np.abs(bits_to_f64(out_b[s, h * g:(h + 1) * g]) - bits_to_f64(ref))
            # 2e-2 absolute; where one bf16 step is coarser than that (|o| >= 2.56) one step is allowed,
            # since two correctly rounded results can land on neighbouring bf16 values.
            allowed = np.maximum(ATTN_TOL, 2.0 ** -7 * np.abs(ref64))
            worst = max(worst, float((err / allowed).max()) * ATTN_TOL)
    return worst


@pytest.mark.parametrize("n", [1, 15, 16, 17, 63, 64, 65, 1000, 4096, 9001])
@pytest.mark.parametrize("g,D", [(4, 128), (7, 128), (4, 64), (8, 64), (1, 128)])
def test_attention_parity_lengths(n, g, D):
    w = wl.Workload("attn", 1, 2, g, D, (n, max(1, n // 2)), (1 << 20, 1 << 20), 0, 21, "normal")
    ld = Loaded(w)
    assert _attn_check(ld, 0) <= ATTN_TOL
    assert ld.cache.device_status()[0] == 0


@pytest.mark.parametrize("n,g", [(20000, 4), (20000, 8), (2049, 4), (513, 7)])
def test_attention_single_segment_many_splits(n, g):
    # One KV head of one sequence: the launch uses the largest split count (32 for long segments), so the merge
    # sees a partial in every lane, CTAs without pages, and more partials than one pass per warp takes.
    w = wl.Workload("attn1", 1, 1, g, 128, (n,), (1 << 20,), 0, 22, "normal")
    ld = Loaded(w)
    assert _attn_check(ld, 0) <= ATTN_TOL
    assert ld.cache.device_status()[0] == 0


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_attention_after_evict(cfg):
    w = small(cfg)
    ld = Loaded(w)
    ld.cache.evict(binding.ALL_LAYERS)
    for l in range(ld.L):
        assert _attn_check(ld, l) <= ATTN_TOL
    # a few appended pairs are attended too
    for step in range(3):
        for l in range(ld.L):
            k, v = wl.new_kv(w, l, step)
            ld.cache.append(l, k.cuda(), v.cuda())
    for l in range(ld.L):
        assert ld.cache.lengths(l) == [min(b, n) + 3 for b, n in zip(w.budgets, w.lens)]
        assert _attn_check(ld, l, 1) <= ATTN_TOL
    assert ld.cache.device_status()[0] == 0


def test_attention_empty_sequence_gives_zeros():
    w = wl.Workload("attn0", 1, 2, 4, 128, (40, 40), (64, 64), 0, 22, "normal")
    c = binding.from_workload(w)
    K, V, A, pos = wl.layer_inputs(w, 0, 1)
    c.prefill(0, 1, K.cuda(), V.cuda(), A.cuda(), pos.cuda())   # sequence 0 stays empty
    q = wl.queries(w, 0).cuda()
    out = c.decode_attn(0, q, out=torch.full_like(q, 7.0))
    assert torch.all(out[0] == 0) and torch.all(torch.isfinite(out[1].float()))


# ------------------------------------------------------------------ append + attention in one launch
@pytest.mark.parametrize("n0", [0, 1, 15, 16, 31, 1000, 4090])
@pytest.mark.parametrize("g,D", [(4, 128), (7, 128), (4, 64)])
def test_fused_append_attention(n0, g, D):
    # 36 tokens, each appended and attended by ONE launch, crossing page boundaries (and opening the
    # very first page when the sequence starts empty); sequence 1 is shorter than sequence 0.
    Hkv, steps = 2, 36
    lens = (n0, n0 // 2)
    w = wl.Workload("fused", 1, Hkv, g, D, tuple(max(1, n) for n in lens), (1 << 20,) * 2, 0, 23, "normal")
    c = binding.from_workload(w)
    hist = {}
    for s in range(2):
        K, V, A, pos = wl.layer_inputs(w, 0, s)
        if lens[s] > 0:
            c.prefill(0, s, K.cuda(), V.cuda(), A.cuda(), pos.cuda())
        for h in range(Hkv):
            hist[(s, h)] = [bits(K)[h][:lens[s]], bits(V)[h][:lens[s]]]
    worst = 0.0
    for step in range(steps):
        k, v = wl.new_kv(w, 0, step)
        q = wl.queries(w, 0, step)
        out = c.append_decode_attn(0, k.cuda(), v.cuda(), q.cuda())
        ob, qb, kb, vb = bits(out), bits(q), bits(k), bits(v)
        assert c.lengths(0) == [lens[0] + step + 1, lens[1] + step + 1]
        for (s, h), hv in hist.items():
            hv[0] = np.concatenate([hv[0], kb[s, h][None]]); hv[1] = np.concatenate([hv[1], vb[s, h][None]])
            ref, ref64 = oracle.attend(qb[s, h * g:(h + 1) * g], hv[0], hv[1])
            err = np.abs(bits_to_f64(ob[s, h * g:(h + 1) * g]) - bits_to_f64(ref))
            worst = max(worst, float((err / np.maximum(ATTN_TOL, 2.0 ** -7 * np.abs(ref64))).max()))
    assert worst <= 1.0
    for (s, h), hv in hist.items():   # the rows are in the cache, positions continue
        k2, v2, a2, p2 = c.export_head(0, s, h)
        assert np.array_equal(bits(k2), hv[0]) and np.array_equal(bits(v2), hv[1])
        assert npf(p2).tolist() == list(range(lens[s] + steps))
        assert np.all(npf(a2)[lens[s]:] == 0)
    assert c.device_status()[0] == 0


def test_fused_append_mask_and_decode_step_match_separate_calls():
    # The fused launch (with a sequence mask) and the all-layer decode step give what
    # fkv_append followed by fkv_decode_attn gives, bit for bit.
    w = wl.Workload("fusedm", 3, 2, 4, 128, (100, 47, 16), (1 << 20,) * 3, 0, 24, "normal")
    a, b = Loaded(w), Loaded(w)
    for step in range(20):
        ks = torch.stack([wl.new_kv(w, l, step)[0] for l in range(3)]).cuda()
        vs = torch.stack([wl.new_kv(w, l, step)[1] for l in range(3)]).cuda()
        qs = torch.stack([wl.queries(w, l, step) for l in range(3)]).cuda()
        if step % 2 == 0:
            out_a = a.cache.decode_step(ks, vs, qs)
            mask = 0
        else:
            mask = 0b101
            out_a = torch.stack([a.cache.append_decode_attn(l, ks[l], vs[l], qs[l], seq_mask=mask) for l in range(3)])
        outs = []
        for l in range(3):
            b.cache.append(l, ks[l], vs[l], seq_mask=mask)
            outs.append(b.cache.decode_attn(l, qs[l]))
        assert torch.equal(out_a, torch.stack(outs))
        assert [a.cache.lengths(l) for l in range(3)] == [b.cache.lengths(l) for l in range(3)]
    for l in range(3):
        for s in range(3):
            for h in range(2):
                for x, y in zip(a.export(l, s, h), b.export(l, s, h)):
                    assert np.array_equal(x, y)
    assert a.cache.device_status()[0] == 0 and b.cache.device_status()[0] == 0


def test_batch_of_96_sequences():
    # The efficiency table of Section 4.3 runs up to 96 concurrent sequences: more than one 64-bit word of the
    # sequence mask.  One eviction and masked appends over 96 short sequences of different lengths.
    rng = np.random.default_rng(96)
    lens = tuple(int(x) for x in rng.integers(40, 140, 96))
    w = wl.Workload("b96", 1, 2, 4, 64, lens, tuple(48 for _ in lens), 8, 25, "normal")
    ld = Loaded(w)
    scores = npf(ld.cache.score(0))
    ld.cache.evict(0)
    assert ld.cache.lengths(0) == [min(48, n) for n in lens]
    mask = (1 << 95) | (1 << 64) | (1 << 63) | 1 | (1 << 17)
    k, v = (t.cuda() for t in wl.new_kv(w, 0, 0))
    q = wl.queries(w, 0, 0).cuda()
    out = ld.cache.append_decode_attn(0, k, v, q, seq_mask=mask)
    ld.cache.append(0, k, v, seq_mask=1 << 70)
    want = [min(48, n) + (1 if (mask >> s) & 1 or s == 70 else 0) for s, n in enumerate(lens)]
    assert ld.cache.lengths(0) == want
    g = w.group_size
    for s in (0, 1, 17, 63, 64, 70, 95):
        for h in range(2):
            K, V, A, pos = ld.head(0, s, h)
            kept = oracle.select(scores[s, h, :lens[s]], 48, 8)
            k2, v2, _, p2 = ld.export(0, s, h)
            nk = len(kept)
            assert np.array_equal(p2[:nk], pos[kept]) and np.array_equal(k2[:nk], K[kept])
            assert len(p2) == want[s]
            if (mask >> s) & 1:
                assert np.array_equal(k2[nk], bits(k)[s, h])
                ref, ref64 = oracle.attend(bits(q)[s, h * g:(h + 1) * g], k2, v2)
                err = np.abs(bits_to_f64(bits(out)[s, h * g:(h + 1) * g]) - bits_to_f64(ref))
                assert np.all(err <= np.maximum(ATTN_TOL, 2.0 ** -7 * np.abs(ref64)))
    assert ld.cache.device_status()[0] == 0


# ------------------------------------------------------------------ the decode protocol of Section 3.1
def test_decode_schedule_sawtooth():
    # cache at B, then L appended tokens -> B + L -> evict back to B, keeping the last L (R = L).
    B, L_ev, steps = 256, 32, 96
    w = wl.Workload("sched", 2, 2, 4, 128, (B,), (B,), L_ev, 31, "channel_lognormal")
    ld = Loaded(w)
    state = {(l, h): list(ld.head(l, 0, h)) for l in range(2) for h in range(2)}
    for step in range(steps):
        for l in range(2):
            k, v = wl.new_kv(w, l, step)
            ld.cache.append(l, k.cuda(), v.cuda())
            for h in range(2):
                K, V, A, pos = state[(l, h)]
                state[(l, h)] = [np.concatenate([K, bits(k)[0, h][None]]), np.concatenate([V, bits(v)[0, h][None]]),
                                 np.concatenate([A, np.zeros((1, A.shape[1]), np.float32)]),
                                 np.concatenate([pos, [pos[-1] + 1]]).astype(np.int32)]
        if (step + 1) % L_ev == 0:
            assert ld.cache.lengths(0) == [B + L_ev]
            ld.cache.evict(binding.ALL_LAYERS)
            assert ld.cache.lengths(0) == [B] and ld.cache.lengths(1) == [B]
            for (l, h), (K, V, A, pos) in state.items():
                phi = oracle.score(K, V, A, *ld.weights(l, h))
                kept = oracle.select(phi, B, L_ev)
                k2, v2, a2, p2 = ld.export(l, 0, h)
                kept_g = np.searchsorted(pos, p2).astype(np.int32)
                assert kept_set_within_band(phi, kept, kept_g, len(pos), B, L_ev, SCORE_TOL)
                assert kept_g[-L_ev:].tolist() == list(range(len(pos) - L_ev, len(pos)))
                state[(l, h)] = [K[kept_g], V[kept_g], A[kept_g], pos[kept_g]]   # follow the GPU's choice
    for l in range(2):
        assert _attn_check(ld, l, 5) <= ATTN_TOL
    assert ld.cache.device_status()[0] == 0


# ------------------------------------------------------------------ determinism
def test_two_runs_are_bit_identical():
    outs = []
    for _ in range(2):
        w = small(4)
        ld = Loaded(w)
        sc = ld.cache.score(0).clone()
        ld.cache.evict(binding.ALL_LAYERS)
        o = ld.cache.decode_attn(0, wl.queries(w, 0).cuda()).clone()
        pos = [ld.export(0, s, h)[3] for s in range(w.batch) for h in range(w.num_kv_heads)]
        outs.append((sc, o, pos))
        ld.cache.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    assert all(np.array_equal(a, b) for a, b in zip(outs[0][2], outs[1][2]))


# ------------------------------------------------------------------ failures are reported, never faults
def test_errors_are_status_codes():
    with pytest.raises(binding.FkvError) as e:
        binding.Cache(1, 2, 4, 96, 1, 64, 128)                      # head_dim not supported
    assert e.value.code == -1
    w = small(1, max_len=100)                                        # one sequence of 100 pairs, B = 50
    assert w.lens == (100,) and w.budgets == (50,)
    c = binding.Cache(1, 2, 4, 64, 1, 50, 128, num_pages=20)          # deliberately tiny pool
    K, V, A, pos = wl.layer_inputs(w, 0, 0)
    c.prefill(0, 0, K.cuda(), V.cuda(), A.cuda(), pos.cuda())        # 2 heads x 7 pages = 14 of 20 pages
    with pytest.raises(binding.FkvError) as e:
        c.prefill(0, 0, K.cuda(), V.cuda())
    assert e.value.code == -1                                        # prefill of a non-empty sequence
    with pytest.raises(binding.FkvError) as e:
        c.evict(0)
    assert e.value.code == -5                                        # scorers not loaded
    c.load_scorers(0, *wl.scorer_params(w, 0))
    c.evict(0)                                                       # needs 2 x 4 fresh pages, only 6 are free
    bits_, free = c.device_status()
    assert bits_ & binding.DEV_POOL_EXHAUSTED and free == 6
    k2, _, _, _ = c.export_head(0, 0, 0)                             # the step was skipped: rows are untouched
    assert np.array_equal(bits(k2), bits(K[0, :len(k2)]))
    c.reset()                                                        # the documented way on after a device error
    assert c.device_status() == (0, 20)
    c.close()
    big = binding.Cache(1, 2, 4, 64, 1, 64, 32)
    k, v = wl.new_kv(w, 0, 0)
    for _ in range(32):
        big.append(0, k.cuda(), v.cuda())
    with pytest.raises(binding.FkvError) as e:
        big.append(0, k.cuda(), v.cuda())
    assert e.value.code == -3                                        # capacity
    assert big.device_status()[0] == 0


@pytest.mark.parametrize("free_pages", [0, 1])
def test_fused_append_without_free_pages_moves_no_head(free_pages):
    # A sequence whose length is a multiple of the page size needs a fresh page on EVERY head for its next
    # pair.  With none free (or fewer than heads) the append is abandoned for all heads: lengths stay, the
    # stored rows stay, the pool-exhausted bit is set, and a second attempt changes nothing either.  After
    # fkv_reset the same cache works again.
    n0, Hkv, g, D = 32, 2, 4, 64
    w = wl.Workload("tiny_pool", 1, Hkv, g, D, (n0,), (64,), 0, 21, "normal")
    c = binding.Cache(1, Hkv, g, D, 1, 64, 128, num_pages=Hkv * (n0 // 16) + free_pages)
    K, V, A, pos = (t.cuda() for t in wl.layer_inputs(w, 0, 0))
    c.prefill(0, 0, K, V, A, pos)
    assert c.device_status() == (0, free_pages)
    k, v = (t.cuda() for t in wl.new_kv(w, 0, 0))
    q = wl.queries(w, 0, 0).cuda()
    for attempt in range(2):
        c.append_decode_attn(0, k, v, q)
        status, free = c.device_status()
        assert status & binding.DEV_POOL_EXHAUSTED and free == 0
        c.sync_lengths()                                              # the documented step after a device error
        assert c.lengths(0) == [n0]
        for h in range(Hkv):                                          # the stored rows are untouched
            k2, v2, _, p2 = c.export_head(0, 0, h)
            assert np.array_equal(bits(k2), bits(K[h])) and np.array_equal(bits(v2), bits(V[h]))
            assert p2.tolist() == list(range(n0))
    c.reset()
    assert c.device_status() == (0, Hkv * (n0 // 16) + free_pages)
    c.prefill(0, 0, K[:, :20].contiguous(), V[:, :20].contiguous(), A[:, :20].contiguous(), pos[:20].contiguous())
    out = c.append_decode_attn(0, k, v, q)
    assert c.device_status()[0] == 0 and c.lengths(0) == [21]
    for h in range(Hkv):
        k2, v2, _, _ = c.export_head(0, 0, h)
        assert np.array_equal(bits(k2)[:20], bits(K[h, :20])) and np.array_equal(bits(k2)[20], bits(k)[0, h])
        ref, ref64 = oracle.attend(bits(q)[0, h * g:(h + 1) * g], bits(k2), bits(v2))
        err = np.abs(bits_to_f64(bits(out)[0, h * g:(h + 1) * g]) - bits_to_f64(ref))
        assert np.all(err <= np.maximum(ATTN_TOL, 2.0 ** -7 * np.abs(ref64)))
    c.close()


# ------------------------------------------------------------------ the sampled action (Section 3.1, Eq. 2; App. B.2)
@pytest.mark.parametrize("n,B,R", [(512, 256, 0), (600, 344, 32), (5000, 4744, 0), (4097, 4096, 0), (9000, 8744, 256),
                                   (300, 300, 0), (777, 100, 100), (1000, 600, 0), (40000, 39000, 0), (70001, 60000, 5),
                                   (65536, 49152, 0), (65536, 65000, 256)])
@pytest.mark.parametrize("fn", [_normal, _ties, _special])
def test_select_sampled_bit_exact(n, B, R, fn):
    # Given the same scores and the same Gumbel draws the kept list is the oracle's, bit for bit
    # (candidates, ranks, fp32 perturbation and ties all agree).
    batch, Hkv = 2, 2
    w = wl.Workload("sels", 1, Hkv, 4, 64, (n,) * batch, (B,) * batch, R, 13, "normal")
    c = binding.from_workload(w)
    for s in range(batch):
        K, V, A, pos = wl.layer_inputs(w, 0, s, "cuda")
        c.prefill(0, s, K, V, A, pos)
    rng = np.random.default_rng(n * 7 + B + R)
    sc = np.full((batch, Hkv, c.cap), np.nan, np.float32)
    for s in range(batch):
        for h in range(Hkv):
            sc[s, h, :n] = fn(rng, n)
    stride = max(1, min(2 * max(n - B, 0), n))
    noise = wl.gumbel_noise(w, 0, stride)
    if fn is _ties:
        noise = torch.round(noise * 2) / 2        # ties among the perturbed values as well
    idx, cnt = c.select_sampled(0, torch.from_numpy(sc).cuda(), noise.cuda())
    idx, cnt = npf(idx), npf(cnt)
    for s in range(batch):
        for h in range(Hkv):
            ref, _ = oracle.select_sampled(sc[s, h, :n], B, R, npf(noise)[s, h])
            assert cnt[s, h] == len(ref)
            assert np.array_equal(idx[s, h, :len(ref)], ref), (n, B, R, s, h)
    assert c.device_status()[0] == 0


@pytest.mark.parametrize("cfg", [1, 2, 4])
def test_evict_sampled_end_to_end(cfg):
    w = small(cfg)
    ld = Loaded(w)
    stride = max(min(2 * (n - b), n) for n, b in zip(w.lens, w.budgets))
    noise = torch.stack([wl.gumbel_noise(w, l, stride) for l in range(ld.L)])
    gpu_scores = {l: npf(ld.cache.score(l)) for l in range(ld.L)}
    ld.cache.evict_sampled(noise.cuda())
    for l in range(ld.L):
        for s in range(w.batch):
            n, B = w.lens[s], w.budgets[s]
            assert ld.cache.lengths(l)[s] == min(B, n)
            for h in range(w.num_kv_heads):
                K, V, A, pos = ld.head(l, s, h)
                k2, v2, a2, p2 = ld.export(l, s, h)
                kept_g = np.searchsorted(pos, p2).astype(np.int32)
                ref, cand = oracle.select_sampled(gpu_scores[l][s, h, :n], B, w.recent_keep, npf(noise)[l, s, h])
                assert np.array_equal(kept_g, ref)
                assert np.array_equal(k2, K[kept_g]) and np.array_equal(v2, V[kept_g]) and np.array_equal(a2, A[kept_g])
                assert np.all(np.diff(p2) > 0)
    assert ld.cache.device_status()[0] == 0


def test_evict_sampled_zero_noise_equals_evict_and_short_noise_is_rejected():
    w = small(3)
    a, b = Loaded(w), Loaded(w)
    stride = 2 * (w.lens[0] - w.budgets[0])
    a.cache.evict(binding.ALL_LAYERS)
    b.cache.evict_sampled(torch.zeros((a.L, 1, w.num_kv_heads, stride), device="cuda"))
    for l in range(a.L):
        for h in range(w.num_kv_heads):
            for x, y in zip(a.export(l, 0, h), b.export(l, 0, h)):
                assert np.array_equal(x, y)
    c = Loaded(w)
    with pytest.raises(binding.FkvError) as e:
        c.cache.evict_sampled(torch.zeros((a.L, 1, w.num_kv_heads, 8), device="cuda"))
    assert e.value.code == -1


# ------------------------------------------------------------------ the library stays inside its workspace
def test_nothing_is_written_outside_the_workspace():
    # A caller-owned buffer with guard zones before and after the workspace: a whole protocol run (prefill,
    # decode steps with maintained features, deterministic and sampled evictions, staged calls, export) must
    # leave every guard byte as it was.
    w = small(2, num_layers=2, max_len=700)
    guard = 1 << 20
    cfg_probe = binding.from_workload(w, 2, max_tokens=max(w.lens) + 300, feature_window=32)
    need = cfg_probe.workspace_bytes
    cfg_probe.close()
    buf = torch.full((guard + need + 512 + guard,), 0xA5, dtype=torch.uint8, device="cuda")
    mid = buf[guard:guard + need + 512]
    cache = binding.from_workload(w, 2, max_tokens=max(w.lens) + 300, feature_window=32, workspace=mid)
    lo, hi = guard + cache.workspace_offset, guard + cache.workspace_offset + need
    for l in range(2):
        W1, b1, W2, b2 = wl.scorer_params(w, l)
        cache.load_scorers(l, W1, b1, W2, b2)
        K, V, A, pos = wl.layer_inputs(w, l, 0)
        cache.prefill(l, 0, K.cuda(), V.cuda(), A.cuda(), pos.cuda())
    for step in range(40):
        ks = torch.stack([wl.new_kv(w, l, step)[0] for l in range(2)]).cuda()
        vs = torch.stack([wl.new_kv(w, l, step)[1] for l in range(2)]).cuda()
        qs = torch.stack([wl.queries(w, l, step) for l in range(2)]).cuda()
        cache.decode_step(ks, vs, qs)
        if step == 19:
            cache.evict()
    n = cache.lengths(0)[0]
    stride = 2 * max(1, n - w.budgets[0])
    noise = torch.stack([wl.gumbel_noise(w, l, stride, device="cuda") for l in range(2)])
    cache.evict_sampled(noise)
    cache.score(0)
    cache.export_head(1, 0, 0)
    torch.cuda.synchronize()
    assert cache.device_status()[0] == 0
    assert bool((buf[:lo] == 0xA5).all()) and bool((buf[hi:] == 0xA5).all())
