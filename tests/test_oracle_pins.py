"""Pins for the CPU oracle: what the paper and the mathematics fix, not the oracle itself.

Each part of the oracle is held against something of a different make:
closed forms, library routines the step reduces to, brute force over tiny
inputs, and the paper's own identity and error bound for renormalised
attention (Appendix A).
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2602_03203_b200 import workloads as wl
from util import bits, bits_to_f64, f32_to_bits, npf

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_facts.txt")


def _facts():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=", 1) if "(" not in line else line.rsplit("=", 1)
            out[k.strip()] = float(v)
    return out


# ----------------------------------------------------------------- shapes the paper prints
def test_paper_shapes_and_footprint():
    f = _facts()
    assert wl.FEATS_PER_HEAD == f["feats_per_head"]
    assert wl.config(1).x_dim == f["x_dim(g=4,D=64)"]
    assert wl.config(3).x_dim == f["x_dim(g=4,D=128)"]
    assert wl.config(4).x_dim == f["x_dim(g=7,D=128)"]
    w = wl.config(3)
    assert w.scorer_hidden == f["scorer_hidden"] and wl.CHUNK == f["eviction_length"]
    kv_bytes = w.num_layers * w.num_kv_heads * w.head_dim * 2 * 2 * w.lens[0]
    assert abs(kv_bytes / 2 ** 30 - f["kv_bytes_qwen3_4b_32k_gib"]) < 0.01


# ----------------------------------------------------------------- scorer
def _rand_segment(n, D, F, H, seed):
    rng = np.random.default_rng(seed)
    K = f32_to_bits(rng.standard_normal((n, D)).astype(np.float32))
    V = f32_to_bits(rng.standard_normal((n, D)).astype(np.float32))
    A = rng.random((n, F)).astype(np.float32) * 3
    W1 = (rng.standard_normal((2 * D + F, H)) * 0.2).astype(np.float32)
    b1 = (rng.standard_normal(H) * 0.2).astype(np.float32)
    W2 = rng.standard_normal(H).astype(np.float32)
    b2 = np.float32(0.3)
    return K, V, A, W1, b1, W2, b2


@pytest.mark.parametrize("act,fn", [
    (oracle.RELU, torch.relu),
    (oracle.SILU, torch.nn.functional.silu),
    (oracle.GELU_TANH, lambda z: torch.nn.functional.gelu(z, approximate="tanh")),
    (oracle.SIGMOID, torch.sigmoid),
])
def test_score_reduces_to_two_library_matmuls(act, fn):
    # Appendix B.1: phi = sigma(x W1 + b1) W2 + b2 is two affine maps around a pointwise
    # function; non-square shapes (x_dim 152/29, H 16/5) catch a transposed operand.
    for (n, D, F, H) in [(37, 64, 24, 16), (9, 8, 13, 5)]:
        K, V, A, W1, b1, W2, b2 = _rand_segment(n, D, F, H, 1)
        x = np.concatenate([bits_to_f64(K), bits_to_f64(V), A.astype(np.float64)], axis=1)
        z = torch.from_numpy(x @ W1.astype(np.float64) + b1.astype(np.float64))
        ref = (fn(z).numpy() @ W2.astype(np.float64) + float(b2)).astype(np.float32)
        got = oracle.score(K, V, A, W1, b1, W2, b2, act)
        np.testing.assert_allclose(got, ref, rtol=0, atol=2e-6)


def test_score_closed_forms():
    n, D, F, H = 11, 16, 12, 16
    K, V, A, W1, b1, W2, b2 = _rand_segment(n, D, F, H, 2)
    # W1 = 0: every pair scores relu(b1).W2 + b2.
    const = float(np.maximum(b1.astype(np.float64), 0) @ W2.astype(np.float64) + b2)
    got = oracle.score(K, V, A, np.zeros_like(W1), b1, W2, b2)
    np.testing.assert_allclose(got, np.full(n, const, np.float32), atol=1e-7)
    # One-hot W1 rows read back a single input channel, which fixes the order k | v | a.
    Kf, Vf = bits_to_f64(K), bits_to_f64(V)
    for row, column in [(3, Kf[:, 3]), (D + 5, Vf[:, 5]), (2 * D + 7, A[:, 7].astype(np.float64))]:
        W1h = np.zeros_like(W1)
        W1h[row, 2] = 1.0
        W2h = np.zeros_like(W2)
        W2h[2] = 1.0
        got = oracle.score(K, V, A, W1h, np.zeros_like(b1), W2h, 0.0)
        np.testing.assert_allclose(got, np.maximum(column, 0).astype(np.float32), atol=1e-7)
    # With every pre-activation positive ReLU is the identity and phi is affine in x.
    big = np.full_like(b1, 1e3)
    got = oracle.score(K, V, A, W1, big, W2, b2)
    x = np.concatenate([Kf, Vf, A.astype(np.float64)], axis=1)
    ref = (x @ W1.astype(np.float64) + big) @ W2.astype(np.float64) + float(b2)
    np.testing.assert_allclose(got, ref.astype(np.float32), rtol=1e-6)


def test_score_triple_loop_brute_force():
    n, D, F, H = 4, 3, 2, 3
    K, V, A, W1, b1, W2, b2 = _rand_segment(n, D, F, H, 3)
    Kf, Vf = bits_to_f64(K), bits_to_f64(V)
    for i in range(n):
        x = list(Kf[i]) + list(Vf[i]) + [float(a) for a in A[i]]
        phi = float(b2)
        for j in range(H):
            z = float(b1[j])
            for c in range(len(x)):
                z += x[c] * float(W1[c][j])
            phi += max(z, 0.0) * float(W2[j])
        assert abs(oracle.score(K, V, A, W1, b1, W2, b2)[i] - phi) < 1e-6


# ----------------------------------------------------------------- selection
def _canon(s):
    s = float(s)
    if math.isnan(s):
        return -math.inf
    return 0.0 if s == 0.0 else s


def _brute_select(phi, B, R):
    n = len(phi)
    if n <= B:
        return list(range(n))
    r = min(R, B)
    m = n - r
    order = sorted(range(m), key=lambda i: (-_canon(phi[i]), i))
    return sorted(order[: B - r]) + list(range(m, n))


def test_select_against_full_sort():
    rng = np.random.default_rng(5)
    for trial in range(200):
        n = int(rng.integers(1, 80))
        B = int(rng.integers(1, 90))
        R = int(rng.integers(0, 20))
        phi = rng.standard_normal(n).astype(np.float32)
        if trial % 3 == 0:  # many exact ties
            phi = np.round(phi * 2) / 2
        if trial % 7 == 0:
            phi[rng.integers(0, n)] = np.nan
            phi[rng.integers(0, n)] = -0.0
            phi[rng.integers(0, n)] = np.inf
            phi[rng.integers(0, n)] = -np.inf
        got = oracle.select(phi, B, R)
        assert got.tolist() == _brute_select(phi, B, R), (n, B, R)


def test_select_exhaustive_subsets_tiny():
    # For n <= 7: among all subsets of the competing slots of the right size, the kept one
    # is the unique subset no outsider of which beats a member under (score desc, slot asc).
    rng = np.random.default_rng(6)
    for n in range(2, 8):
        for B in range(1, n):
            for R in (0, 1, 2):
                phi = np.round(rng.standard_normal(n) * 1.5).astype(np.float32)  # ties on purpose
                r = min(R, B)
                m, k = n - r, B - r
                beats = lambda a, b: (phi[a] > phi[b]) or (phi[a] == phi[b] and a < b)
                winners = [set(S) for S in itertools.combinations(range(m), k)
                           if not any(beats(o, i) for i in S for o in range(m) if o not in S)]
                assert len(winners) == 1
                expect = sorted(winners[0]) + list(range(m, n))
                assert oracle.select(phi, B, R).tolist() == expect


def test_select_invariants_and_special_cases():
    rng = np.random.default_rng(7)
    n, B, R = 500, 200, 32
    phi = rng.standard_normal(n).astype(np.float32)
    kept = oracle.select(phi, B, R)
    assert len(kept) == min(B, n)                                # Section 3.1: back to the budget
    assert np.all(np.diff(kept) > 0)                             # ascending, no repeats
    assert kept[-R:].tolist() == list(range(n - R, n))           # the recent window always stays
    comp = kept[kept < n - R]
    evicted = np.setdiff1d(np.arange(n - R), comp)
    assert phi[evicted].max() <= phi[comp].min()                 # lowest scores are the ones evicted
    # n <= B keeps everything; all-equal scores keep the earliest slots plus the window.
    assert oracle.select(phi[:150], B, R).tolist() == list(range(150))
    assert oracle.select(np.ones(n, np.float32), B, R).tolist() == list(range(B - R)) + list(range(n - R, n))
    # R >= B keeps exactly the last B.
    assert oracle.select(phi, 50, 80).tolist() == list(range(n - 50, n))
    # -0 ties with +0 (lower slot wins); NaN is evicted before any number.
    assert oracle.select(np.array([0.0, -0.0, 0.0], np.float32), 2, 0).tolist() == [0, 1]
    assert oracle.select(np.array([np.nan, -1e30, np.nan, -np.inf], np.float32), 1, 0).tolist() == [1]
    assert oracle.select(np.array([np.nan, np.nan, -np.inf], np.float32), 2, 0).tolist() == [0, 1]


# ----------------------------------------------------------------- compaction
def test_compact_rows_positions_idempotence():
    K, V, A, W1, b1, W2, b2 = _rand_segment(300, 16, 12, 16, 8)
    pos = np.cumsum(np.random.default_rng(8).integers(1, 5, 300)).astype(np.int32)
    phi = oracle.score(K, V, A, W1, b1, W2, b2)
    kept = oracle.select(phi, 100, 10)
    K2, V2, A2, pos2 = oracle.compact(K, V, A, pos, kept)
    assert np.array_equal(K2, K[kept]) and np.array_equal(V2, V[kept])
    assert np.array_equal(A2, A[kept]) and np.array_equal(pos2, pos[kept])
    assert np.all(np.diff(pos2) > 0)
    # Evicting again at the budget changes nothing.
    phi2 = oracle.score(K2, V2, A2, W1, b1, W2, b2)
    np.testing.assert_array_equal(phi2, phi[kept])               # scores do not depend on the slot
    assert oracle.select(phi2, 100, 10).tolist() == list(range(100))


# ----------------------------------------------------------------- attention
def test_attend_matches_library_sdpa():
    rng = np.random.default_rng(9)
    for (n, g, D) in [(257, 4, 64), (33, 7, 128), (1, 4, 16)]:
        q = f32_to_bits(rng.standard_normal((g, D)).astype(np.float32))
        K = f32_to_bits(rng.standard_normal((n, D)).astype(np.float32) * 1.5)
        V = f32_to_bits(rng.standard_normal((n, D)).astype(np.float32))
        tq = torch.from_numpy(bits_to_f64(q)).view(1, g, 1, D)
        tk = torch.from_numpy(bits_to_f64(K)).view(1, 1, n, D).expand(1, g, n, D)
        tv = torch.from_numpy(bits_to_f64(V)).view(1, 1, n, D).expand(1, g, n, D)
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).view(g, D).numpy()
        out_b, out64 = oracle.attend(q, K, V)
        np.testing.assert_allclose(out64, ref, atol=1e-12)
        assert np.array_equal(out_b, f32_to_bits(ref.astype(np.float32)))
        # an explicit scale is honoured
        ref2 = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=0.37).view(g, D).numpy()
        np.testing.assert_allclose(oracle.attend(q, K, V, 0.37)[1], ref2, atol=1e-12)


def test_attend_closed_forms():
    rng = np.random.default_rng(10)
    g, D = 4, 32
    q = f32_to_bits(rng.standard_normal((g, D)).astype(np.float32))
    V = f32_to_bits(rng.standard_normal((50, D)).astype(np.float32))
    k1 = f32_to_bits(rng.standard_normal((1, D)).astype(np.float32))
    # one retained pair: o = v_0
    assert np.array_equal(oracle.attend(q, k1, V[:1])[0], np.broadcast_to(V[:1], (g, D)))
    # identical keys: uniform weights, o = mean(v)
    out64 = oracle.attend(q, np.repeat(k1, 50, axis=0), V)[1]
    np.testing.assert_allclose(out64, np.broadcast_to(bits_to_f64(V).mean(0), (g, D)), atol=1e-13)


def test_renormalisation_identity_and_error_bound():
    # Appendix A: with evicted mass eps, a_hat_i = a_i / (1 - eps) on the retained set,
    # and ||o - o_hat||_2 <= 2 C eps with C = max ||v_i||_2 - for ANY retained set.
    rng = np.random.default_rng(11)
    n, g, D = 400, 4, 64
    q = f32_to_bits(rng.standard_normal((g, D)).astype(np.float32))
    K = f32_to_bits(rng.standard_normal((n, D)).astype(np.float32))
    V = f32_to_bits(rng.standard_normal((n, D)).astype(np.float32))
    qf, Kf, Vf = bits_to_f64(q), bits_to_f64(K), bits_to_f64(V)
    s = qf @ Kf.T / math.sqrt(D)
    a = np.exp(s - s.max(1, keepdims=True))
    a /= a.sum(1, keepdims=True)                     # full-cache attention weights
    o_full = oracle.attend(q, K, V)[1]
    np.testing.assert_allclose(o_full, a @ Vf, atol=1e-12)
    C = np.linalg.norm(Vf, axis=1).max()
    for frac in (0.9, 0.5, 0.1):
        kept = np.sort(rng.choice(n, int(n * frac), replace=False))
        eps = 1.0 - a[:, kept].sum(1)
        o_hat = oracle.attend(q, K[kept], V[kept])[1]
        np.testing.assert_allclose(o_hat, (a[:, kept] / (1 - eps)[:, None]) @ Vf[kept], atol=1e-12)
        assert np.all(np.linalg.norm(o_full - o_hat, axis=1) <= 2 * C * eps + 1e-12)


# ----------------------------------------------------------------- the batch drivers add nothing
def test_batch_drivers_equal_single_segment_calls():
    w = wl.shrink(wl.config(4), num_layers=1, max_len=300, batch=3)
    Ks, Vs, As, Ps, ns, Bs, W1s, b1s, W2s, b2s = [], [], [], [], [], [], [], [], [], []
    W1, b1, W2, b2 = [npf(t) for t in wl.scorer_params(w, 0)]
    for s in range(w.batch):
        K, V, A, pos = wl.layer_inputs(w, 0, s)
        for h in range(w.num_kv_heads):
            Ks.append(bits(K[h])); Vs.append(bits(V[h])); As.append(npf(A[h])); Ps.append(npf(pos))
            ns.append(w.lens[s]); Bs.append(w.budgets[s])
            W1s.append(W1[h]); b1s.append(b1[h]); W2s.append(W2[h]); b2s.append(b2[h])
    off = np.concatenate([[0], np.cumsum(ns)[:-1]]).astype(np.int64)
    phi, kept, nkept, K2, V2, A2, pos2 = oracle.evict_batch(
        np.concatenate(Ks), np.concatenate(Vs), np.concatenate(As), np.concatenate(Ps), off, ns, Bs, 5,
        np.stack(W1s), np.stack(b1s), np.stack(W2s), np.array(b2s))
    q = bits(wl.queries(w, 0))
    qs = []
    for i in range(len(ns)):
        p1 = oracle.score(Ks[i], Vs[i], As[i], W1s[i], b1s[i], W2s[i], b2s[i])
        k1 = oracle.select(p1, Bs[i], 5)
        o = int(off[i])
        assert np.array_equal(phi[o:o + ns[i]], p1) and nkept[i] == len(k1)
        assert np.array_equal(kept[o:o + nkept[i]], k1)
        c = oracle.compact(Ks[i], Vs[i], As[i], Ps[i], k1)
        assert np.array_equal(K2[o:o + nkept[i]], c[0]) and np.array_equal(pos2[o:o + nkept[i]], c[3])
        assert np.array_equal(V2[o:o + nkept[i]], c[1]) and np.array_equal(A2[o:o + nkept[i]], c[2])
        s, h = divmod(i, w.num_kv_heads)
        qs.append(q[s, h * w.group_size:(h + 1) * w.group_size])
    out = oracle.attend_batch(np.stack(qs), K2, V2, off, nkept)
    for i in range(len(ns)):
        o = int(off[i])
        assert np.array_equal(out[i], oracle.attend(qs[i], K2[o:o + nkept[i]], V2[o:o + nkept[i]])[0])


# ---------------------------------------------------------------- sampled eviction action (Section 3.1, Eq. 2; App. B.2)
def _random_scores(rng, n, kind):
    x = rng.standard_normal(n).astype(np.float32)
    if kind == "ties":
        x = (np.round(x * 3) / 3).astype(np.float32)
    if kind == "special":
        for val in (np.nan, -0.0, 0.0, np.inf, -np.inf):
            x[rng.integers(0, n, max(1, n // 20))] = val
    return x


@pytest.mark.parametrize("kind", ["normal", "ties", "special"])
def test_sampled_zero_noise_is_the_deterministic_rule(kind):
    # With no perturbation the E largest -phi among the candidates are the E lowest scores:
    # the action reduces to plain Top-K (the ablation's "Top-K" row), which is pinned above.
    rng = np.random.default_rng(5)
    for _ in range(60):
        n = int(rng.integers(2, 300)); B = int(rng.integers(1, n + 2)); R = int(rng.integers(0, 40))
        phi = _random_scores(rng, n, kind)
        kept, cand = oracle.select_sampled(phi, B, R, np.zeros(2 * n, np.float32))
        assert np.array_equal(kept, oracle.select(phi, B, R))


def test_sampled_invariants_and_candidate_set():
    rng = np.random.default_rng(6)
    for _ in range(100):
        n = int(rng.integers(3, 400)); B = int(rng.integers(1, n)); R = int(rng.integers(0, 30))
        phi = _random_scores(rng, n, "ties" if _ % 2 else "normal")
        noise = rng.gumbel(size=2 * n).astype(np.float32)
        kept, cand = oracle.select_sampled(phi, B, R, noise)
        r = min(R, B); m = n - r; E = n - B; C = min(2 * E, m)
        assert len(kept) == B and np.all(np.diff(kept) > 0)
        assert kept[B - r:].tolist() == list(range(m, n))                       # the recent pairs stay
        evicted = np.setdiff1d(np.arange(m), kept)
        assert len(evicted) == E and np.all(np.isin(evicted, cand))              # only candidates are evicted
        # candidates are the C lowest scores (ties: the higher slot is the lower-ranked pair) - brute force
        canon = np.where(np.isnan(phi[:m]), -np.inf, phi[:m]) + 0.0
        order = sorted(range(m), key=lambda i: (canon[i], -i))
        assert sorted(order[:C]) == cand.tolist()
        # every non-candidate scores at least as high as every candidate
        if C < m:
            assert canon[np.setdiff1d(np.arange(m), cand)].min() >= canon[cand].max()


def test_sampled_noise_decides_inside_the_candidate_set():
    phi = np.array([0.9, 0.10, 0.8, 0.11, 0.12, 0.13, 0.7, 0.95], np.float32)    # n = 8, B = 6: E = 2, 4 candidates
    kept, cand = oracle.select_sampled(phi, 6, 0, np.zeros(4, np.float32))
    assert cand.tolist() == [1, 3, 4, 5] and kept.tolist() == [0, 2, 4, 5, 6, 7]
    noise = np.array([-50.0, 0.0, 0.0, 50.0], np.float32)                         # rank 0 (slot 1) never, rank 3 (slot 5) surely
    kept, _ = oracle.select_sampled(phi, 6, 0, noise)
    assert 1 in kept and 5 not in kept and 3 not in kept                          # slot 3 is the lowest of the rest
    # a pair outside the candidate set is never evicted, whatever the noise
    for seed in range(50):
        kept, _ = oracle.select_sampled(phi, 6, 0, np.random.default_rng(seed).gumbel(size=4).astype(np.float32) * 100)
        assert all(s in kept for s in (0, 2, 6, 7))


def test_sampled_matches_multinomial_without_replacement():
    # The paper draws E pairs from Multinomial(softmax(-phi)) over the candidates.  Sequential draws
    # without replacement have a closed form for every evicted SET (sum over the orders of
    # p_a / 1 * p_b / (1 - p_a) ...); the Gumbel-perturbed selection must reproduce those
    # probabilities.  A wrong sign of phi, a softmax over the wrong set, or drawing with replacement fails.
    import itertools
    phi = np.array([0.3, 2.0, -0.4, 0.9, 0.1, 1.5, 3.0], np.float32)   # n = 7, B = 5, R = 1: m = 6, E = 2, C = 4
    B, R, E = 5, 1, 2
    _, cand = oracle.select_sampled(phi, B, R, np.zeros(4, np.float32))
    assert cand.tolist() == [0, 2, 3, 4]
    logits = -phi[cand].astype(np.float64)
    p = np.exp(logits - logits.max()); p /= p.sum()
    exact = {}
    for a, b in itertools.permutations(range(4), 2):
        key = frozenset((int(cand[a]), int(cand[b])))
        exact[key] = exact.get(key, 0.0) + p[a] * p[b] / (1.0 - p[a])
    assert abs(sum(exact.values()) - 1.0) < 1e-12
    rng = np.random.default_rng(7)
    N = 40000
    counts = {k: 0 for k in exact}
    for _ in range(N):
        kept, _c = oracle.select_sampled(phi, B, R, rng.gumbel(size=4).astype(np.float32))
        ev = frozenset(int(x) for x in np.setdiff1d(np.arange(6), kept))
        counts[ev] += 1
    for k, pe in exact.items():
        sigma = np.sqrt(pe * (1 - pe) / N)
        assert abs(counts[k] / N - pe) < 5 * sigma + 1e-4, (sorted(k), counts[k] / N, pe)


# ---------------------------------------------------------------- attention features (Appendix B.1)
def _rand_bits(rng, shape, scale=1.0):
    return f32_to_bits((rng.standard_normal(shape) * scale).astype(np.float32))


def test_features_uniform_attention_closed_form():
    # Identical keys: every query spreads 1 / nvalid[t] over the pairs it saw, so every sum is known.
    rng = np.random.default_rng(11)
    n0, nq, g, D = 20, 40, 3, 16
    K = np.repeat(_rand_bits(rng, (1, D)), n0 + nq, axis=0)
    q = _rand_bits(rng, (nq, g, D))
    nvalid = np.arange(n0 + 1, n0 + nq + 1, dtype=np.int32)          # one pair appended per query
    A0 = np.zeros((n0 + nq, 6 * g), np.float32)
    A0[:n0] = rng.random((n0, 6 * g)).astype(np.float32)
    A1 = oracle.features(K, q, nvalid, A0)
    for i in (0, 5, n0 - 1, n0, n0 + 7, n0 + nq - 1):
        seen = [t for t in range(nq) if i < nvalid[t]]                # queries that could see pair i
        for j in range(g):
            row = A1[i, 6 * j:6 * j + 6]
            for k, w in enumerate((8, 16, 32)):
                expect = sum(1.0 / nvalid[t] for t in seen if nq - 1 - t < w) / w
                assert abs(row[k] - expect) < 1e-6
            chunk = sum(1.0 / nvalid[t] for t in seen) / nq
            assert abs(row[3] - chunk) < 1e-6
            assert abs(row[4] - (A0[i, 6 * j + 4] + chunk)) < 1e-6
            assert abs(row[5] - (0.9 * A0[i, 6 * j + 5] + chunk)) < 1e-6
    # a pair appended at the last step was seen by one query only: window-8 feature = (1/n)/8
    assert abs(A1[n0 + nq - 1, 0] - 1.0 / (n0 + nq) / 8) < 1e-7


def test_features_against_library_softmax_and_one_hot():
    rng = np.random.default_rng(12)
    n, nq, g, D = 50, 24, 2, 32
    Kb, qb = _rand_bits(rng, (n, D)), _rand_bits(rng, (nq, g, D))
    nvalid = np.full(nq, n, np.int32)
    A1 = oracle.features(Kb, qb, nvalid, np.zeros((n, 6 * g), np.float32), scale=0.3)
    Kf = torch.from_numpy(bits_to_f64(Kb)); qf = torch.from_numpy(bits_to_f64(qb))
    P = torch.softmax(torch.einsum("tjd,nd->jtn", qf, Kf) * 0.3, dim=-1).numpy()     # [g][nq][n], library softmax
    for j in range(g):
        assert np.allclose(A1[:, 6 * j + 0], P[j, -8:].sum(0) / 8, atol=1e-6)
        assert np.allclose(A1[:, 6 * j + 1], P[j, -16:].sum(0) / 16, atol=1e-6)
        assert np.allclose(A1[:, 6 * j + 2], P[j].sum(0) / 32, atol=1e-6)             # only 24 queries, still / 32
        assert np.allclose(A1[:, 6 * j + 3], P[j].mean(0), atol=1e-6)
    # a query far along one key puts all its mass there
    Kone = np.zeros((4, D), np.float32); Kone[2, 0] = 50.0
    qone = np.zeros((1, 1, D), np.float32); qone[0, 0, 0] = 50.0
    A2 = oracle.features(f32_to_bits(Kone), f32_to_bits(qone), np.array([4], np.int32), np.zeros((4, 6), np.float32),
                         scale=1.0)
    assert np.allclose(A2[2], [1 / 8, 1 / 16, 1 / 32, 1.0, 1.0, 1.0]) and np.allclose(A2[[0, 1, 3]], 0.0)


def test_features_chunks_accumulate_and_decay():
    rng = np.random.default_rng(13)
    n, g, D = 30, 2, 16
    Kb = _rand_bits(rng, (n, D))
    nv = np.full(10, n, np.int32)
    q1, q2 = _rand_bits(rng, (10, g, D)), _rand_bits(rng, (10, g, D))
    Z = np.zeros((n, 6 * g), np.float32)
    A1 = oracle.features(Kb, q1, nv, Z)
    A2 = oracle.features(Kb, q2, nv, A1)
    c1, c2 = oracle.features(Kb, q1, nv, Z)[:, 3::6], oracle.features(Kb, q2, nv, Z)[:, 3::6]
    assert np.allclose(A2[:, 4::6], c1 + c2, atol=1e-6)                 # direct sum over chunks
    assert np.allclose(A2[:, 5::6], 0.9 * c1 + c2, atol=1e-6)           # per-chunk decay 0.9
    assert np.allclose(A2[:, 3::6], c2, atol=1e-7)                      # window features belong to the last chunk only
    assert np.allclose(A2[:, 3::6].sum(0), 1.0, atol=1e-5)              # mean of probability rows still sums to 1


# ---------------------------------------------------------------- baseline scores (Appendix E.2: H2O, SnapKV)
def test_feature_column_scores():
    rng = np.random.default_rng(21)
    n, g = 40, 4
    A = rng.random((n, 6 * g)).astype(np.float32)
    for col in range(6):
        phi = oracle.score_feature(A, g, col)
        assert np.allclose(phi, A.reshape(n, g, 6)[:, :, col].astype(np.float64).mean(1), rtol=1e-6)
    # one head only: the column itself; a head-major layout mistake (6 heads x g columns) fails here
    A1 = np.zeros((3, 6 * g), np.float32); A1[1, 2 * 6 + 4] = 8.0          # head 2, direct-sum column
    assert oracle.score_feature(A1, g, oracle.H2O_COLUMN).tolist() == [0.0, 2.0, 0.0]
    assert oracle.score_feature(A1, g, oracle.SNAPKV_COLUMN).tolist() == [0.0, 0.0, 0.0]
    # H2O keeps the pairs with the highest cumulative attention: selection on that column
    cum = np.array([5, 1, 4, 2, 3], np.float32)
    A2 = np.zeros((5, 6), np.float32); A2[:, 4] = cum
    assert oracle.select(oracle.score_feature(A2, 1, oracle.H2O_COLUMN), 3, 0).tolist() == [0, 2, 4]


# ---------------------------------------------------------------- R-KV baseline (Appendix E.2; weights 0.1 / 0.9)
def test_rkv_paper_weights_are_the_defaults():
    f = _facts()
    import inspect
    sig = inspect.signature(oracle.score_rkv)
    assert sig.parameters["lambda_a"].default == f["rkv_weight_attention"]
    assert sig.parameters["lambda_s"].default == f["rkv_weight_similarity"]


def test_rkv_against_library_cosine_matrix():
    # Random bf16 keys of a non-square shape: the full cosine matrix from a library matmul in fp64, its
    # diagonal struck out, row maxima (a transposed operand, a missing norm or a kept diagonal fails).
    rng = np.random.default_rng(31)
    n, D, g = 57, 64, 3
    Kb = f32_to_bits(rng.standard_normal((n, D)) * rng.lognormal(0, 1, (1, D)))
    A = rng.random((n, 6 * g)).astype(np.float32)
    K = bits_to_f64(Kb)
    Kn = K / np.linalg.norm(K, axis=1, keepdims=True)
    C = Kn @ Kn.T
    np.fill_diagonal(C, -np.inf)
    snap = A.reshape(n, g, 6)[:, :, 0].astype(np.float64).mean(1)
    for la, ls in [(0.1, 0.9), (1.0, 0.0), (0.0, 1.0), (0.3, 2.0)]:
        phi = oracle.score_rkv(Kb, A, g, la, ls)
        assert np.allclose(phi, la * snap - ls * C.max(1), rtol=0, atol=2e-7)
    rows = np.array([5, 0, 56, 5], np.int32)                       # the sampled form gives the same values
    assert np.array_equal(oracle.score_rkv(Kb, A, g, rows=rows), oracle.score_rkv(Kb, A, g)[rows])


def test_rkv_closed_forms():
    g, D = 2, 64
    # identical keys: every pair has a twin, similarity 1 for all
    Kb = np.tile(f32_to_bits(np.linspace(-1, 2, D)[None]), (9, 1))
    Z = np.zeros((9, 6 * g), np.float32)
    assert np.allclose(oracle.score_rkv(Kb, Z, g, 0.0, 1.0), -1.0, atol=1e-7)
    # mutually orthogonal keys (scaled unit vectors): similarity 0 for all, whatever the norms
    E = np.zeros((5, D)); E[np.arange(5), [3, 9, 17, 40, 63]] = [1.0, -2.0, 0.5, 4.0, 8.0]
    assert np.array_equal(oracle.score_rkv(f32_to_bits(E), Z[:5], g, 0.0, 1.0), np.zeros(5, np.float32))
    # opposite keys: cosine -1; with a third, unrelated key the maximum picks the larger one (0)
    O = np.zeros((2, D)); O[0, 0] = 1.0; O[1, 0] = -3.0
    assert np.allclose(oracle.score_rkv(f32_to_bits(O), Z[:2], g, 0.0, 1.0), 1.0)      # phi = -(-1)
    O3 = np.vstack([O, np.eye(1, D, 7)])
    assert np.allclose(oracle.score_rkv(f32_to_bits(O3), Z[:3], g, 0.0, 1.0), 0.0)
    # a single pair has no other pair; a zero key has cosine 0 with everything
    assert oracle.score_rkv(f32_to_bits(np.ones((1, D))), Z[:1], g, 0.0, 1.0).tolist() == [0.0]
    Zk = np.zeros((3, D)); Zk[1] = 1.0; Zk[2] = 1.0
    assert np.allclose(oracle.score_rkv(f32_to_bits(Zk), Z[:3], g, 0.0, 1.0), [0.0, -1.0, -1.0])
    # weight of the similarity term -> 0: the SnapKV score, bit for bit, and so the same kept set
    rng = np.random.default_rng(32)
    A = rng.random((40, 6 * g)).astype(np.float32)
    Kr = f32_to_bits(rng.standard_normal((40, D)))
    assert np.array_equal(oracle.score_rkv(Kr, A, g, 1.0, 0.0), oracle.score_feature(A, g, oracle.SNAPKV_COLUMN))
    # the sign: of two pairs with equal attention the one with a near-duplicate elsewhere scores lower
    Kd = rng.standard_normal((6, D)); Kd[4] = Kd[1] * 1.001
    phi = oracle.score_rkv(f32_to_bits(Kd), np.ones((6, 6 * g), np.float32), g)
    assert phi[1] < phi[0] and phi[4] < phi[0] and set(oracle.select(phi, 4, 0).tolist()) == {0, 2, 3, 5}


# ---------------------------------------------------------------- Golden Eviction labels (Section 3.2, Eq. 3-5)
def _golden_brute(A, B, L):
    """Independent statement with numpy slicing and Python sets (not the oracle's loops)."""
    g, T, _ = A.shape
    M = math.ceil((T - B) / L) - 1
    blocks = np.zeros((M, T))
    for t in range(1, M + 1):
        rows = A[:, B + t * L:min(T, B + (t + 1) * L), :].astype(np.float64)
        blocks[t - 1] = rows.sum(axis=(0, 1)) / (g * L)
    alpha = np.maximum.accumulate(blocks[::-1], axis=0)[::-1]
    cache, kept = list(range(B)), []
    for t in range(1, M + 1):
        a32 = alpha[t - 1].astype(np.float32)
        best = sorted(cache, key=lambda i: (-a32[i], i))[:B - L]
        kept.append(sorted(best))
        cache = sorted(best) + list(range(B + (t - 1) * L, B + t * L))
    return alpha, np.array(kept, np.int32)


def test_golden_against_brute_force_and_invariants():
    for seed, (g, T, B, L) in enumerate([(2, 96, 32, 8), (4, 130, 40, 16), (1, 64, 24, 8), (3, 77, 30, 10)]):
        A = wl.causal_attention(seed, g, T).numpy()
        alpha, kept = oracle.golden(A, B, L)
        M = math.ceil((T - B) / L) - 1                                   # the paper's count of eviction steps
        assert alpha.shape == (M, T) and kept.shape == (M, B - L)
        a_ref, k_ref = _golden_brute(A, B, L)
        assert np.allclose(alpha, a_ref, rtol=1e-6, atol=1e-9) and np.array_equal(kept, k_ref)
        assert np.all(alpha[:-1] >= alpha[1:])                            # a maximum over fewer future blocks
        cache = set(range(B))
        for t in range(M):
            assert np.all(np.diff(kept[t]) > 0) and set(kept[t].tolist()) <= cache   # evictions are irreversible
            cache = set(kept[t].tolist()) | set(range(B + t * L, B + (t + 1) * L))


def test_golden_closed_forms():
    # Every query puts 60 % of its attention on key 5 and spreads the rest evenly over what it can see:
    # key 5 has the top future score at every step and is always retained; the others tie, so the
    # lowest positions survive.
    g, T, B, L = 2, 80, 24, 8
    A = np.zeros((g, T, T), np.float32)
    for r in range(T):
        if r >= 5:
            A[:, r, :r + 1] = 0.4 / r if r > 0 else 0.0
            A[:, r, 5] = 0.6
        else:
            A[:, r, :r + 1] = 1.0 / (r + 1)
    alpha, kept = oracle.golden(A, B, L)
    M = math.ceil((T - B) / L) - 1
    assert M == 6
    assert np.all(np.argmax(alpha, axis=1) == 5) and np.allclose(alpha[:, 5], 0.6)
    for t in range(M):
        assert 5 in kept[t]
    # block t averages 0.4 / r over its rows: decreasing in t, so the future score IS the block score
    t = 2
    rows = np.arange(B + t * L, B + (t + 1) * L)
    assert np.isclose(alpha[t - 1, 0], np.mean(0.4 / rows), rtol=1e-5)
    # the last block is zero-padded to L rows when T is not on a block boundary
    A2 = A[:, :76, :76]
    alpha2, _ = oracle.golden(A2, B, L)
    rows = np.arange(B + 6 * L, 76)
    assert np.isclose(alpha2[5, 0], np.sum(0.4 / rows) / L, rtol=1e-5)
