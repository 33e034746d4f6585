"""Golden Eviction label builder (Section 3.2, Eq. 3-5) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_03203_b200 import binding, workloads as wl
from util import npf

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("g,T,B,L", [(2, 96, 32, 8), (4, 1000, 256, 64), (7, 777, 300, 50), (1, 2048, 1024, 128),
                                     (4, 4096, 2048, 256), (2, 300, 280, 16)])
def test_golden_matches_oracle(g, T, B, L):
    A = wl.causal_attention(T + g, g, T)
    alpha_g, kept_g = binding.golden_eviction(A.cuda(), B, L)
    alpha_o, kept_o = oracle.golden(A.numpy(), B, L)
    assert alpha_g.shape == alpha_o.shape
    # block averages: fp32 sums of up to g L probabilities against fp64
    assert np.allclose(npf(alpha_g), alpha_o, rtol=2e-6 * np.sqrt(g * L) + 1e-6, atol=1e-9)
    # the retained sets, bit for bit, from the SAME future scores (the GPU's own)
    assert np.array_equal(npf(kept_g), oracle.golden_select(npf(alpha_g), B, L))
    # and end to end: the two traces agree except where future scores are within rounding of the cut
    if not np.array_equal(npf(kept_g), kept_o):
        for t in range(len(kept_o)):
            diff = np.setxor1d(npf(kept_g)[t], kept_o[t])
            if len(diff):
                cut = np.sort(alpha_o[t][kept_o[t]])[0]
                assert np.all(np.abs(alpha_o[t][diff] - cut) <= 1e-5 * max(cut, 1e-9) + 1e-9)
                break   # later steps follow different caches


def test_golden_select_ties_and_errors():
    rng = np.random.default_rng(3)
    T, B, L = 500, 128, 32
    M = binding.lib().fkv_golden_steps(T, B, L)
    alpha = np.sort((np.round(rng.random((M, T)) * 8) / 8).astype(np.float32), axis=0)[::-1].copy()   # heavy ties
    kept = binding.golden_select(torch.from_numpy(alpha).cuda(), B, L)
    assert np.array_equal(npf(kept), oracle.golden_select(alpha, B, L))
    assert binding.lib().fkv_golden_steps(100, 50, 50) == -1          # L must be below B
    assert binding.lib().fkv_golden_steps(100, 90, 10) == 0           # no block after the first eviction position
