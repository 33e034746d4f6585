"""Test plumbing: put one workload into a CUDA cache and keep the same bytes for the oracle."""
from __future__ import annotations

import numpy as np
import torch

from paper_2602_03203_b200 import binding, workloads as wl
from util import bits, npf


class Loaded:
    """A workload resident in a ``binding.Cache`` plus host copies of every input tensor."""

    def __init__(self, w: wl.Workload, num_layers=None, max_tokens=None, num_pages=0, gen_device="cpu"):
        self.w = w
        self.L = num_layers or w.num_layers
        self.cache = binding.from_workload(w, self.L, num_pages=num_pages, max_tokens=max_tokens)
        self.scorer = {}   # layer -> (W1, b1, W2, b2) numpy, per head on axis 0
        self.seg = {}      # (layer, seq) -> dict(K, V bits [Hkv][n][D]; A [Hkv][n][F]; pos [n])
        for l in range(self.L):
            W1, b1, W2, b2 = wl.scorer_params(w, l, gen_device)
            self.cache.load_scorers(l, W1, b1, W2, b2)
            self.scorer[l] = tuple(npf(t) for t in (W1, b1, W2, b2))
            for s in range(w.batch):
                K, V, A, pos = wl.layer_inputs(w, l, s, gen_device)
                self.cache.prefill(l, s, K.cuda(), V.cuda(), A.cuda(), pos.cuda())
                self.seg[(l, s)] = dict(K=bits(K), V=bits(V), A=npf(A), pos=npf(pos))
        torch.cuda.synchronize()

    def head(self, layer, seq, h):
        d = self.seg[(layer, seq)]
        return d["K"][h], d["V"][h], d["A"][h], d["pos"]

    def weights(self, layer, h):
        W1, b1, W2, b2 = self.scorer[layer]
        return W1[h], b1[h], W2[h], float(b2[h])

    def export(self, layer, seq, h):
        k, v, a, p = self.cache.export_head(layer, seq, h)
        return bits(k), bits(v), npf(a), npf(p)


def kept_set_within_band(phi_oracle: np.ndarray, kept_oracle: np.ndarray, kept_gpu: np.ndarray, n: int, B: int, R: int,
                         tol: float) -> bool:
    """End-to-end rule: the two kept sets may differ only at competing slots whose oracle
    score lies within `tol` of the oracle's (B - r)-th best score."""
    if n <= B:
        return np.array_equal(kept_oracle, kept_gpu)
    r = min(R, B)
    m, k = n - r, B - r
    if k == 0:
        return np.array_equal(kept_oracle, kept_gpu)
    comp = np.where(np.isnan(phi_oracle[:m]), -np.inf, phi_oracle[:m])
    kth = np.sort(comp)[::-1][k - 1]
    diff = np.setxor1d(kept_oracle, kept_gpu)
    return bool(np.all(diff < m) and np.all(np.abs(comp[diff] - kth) <= tol))
