"""Seeded synthetic inputs for the eviction + decode-attention path.

This module only draws random tensors (shapes, value distributions, sparsity
of spikes and duplicates).  It contains none of the method's arithmetic: no
scorer, no selection, no attention.  Both the CPU oracle's tests and the CUDA
path's tests/bench take their inputs from here, so the two sides always see
byte-identical tensors.

All tensors are produced with ``torch`` on the device that is asked for; a
given (workload, layer, seq, device type) always gives the same bytes.  A test
generates once and hands the same bytes to both sides.

Shapes follow the reasoning-model decodes the paper evaluates (Section 4.1:
Qwen3-4B, DeepSeek-R1-Distill-Qwen-7B; Appendix E: an 8B model) and the
feature width 6g + 2D of Appendix B.1.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Tuple

import torch

# Tensor ids that key the per-tensor random streams.
_T_K, _T_V, _T_FEAT, _T_SCALE, _T_W, _T_Q, _T_NEW, _T_LEN, _T_SPIKE, _T_DUP, _T_NOISE = range(11)

FEATS_PER_HEAD = 6  # Appendix B.1: windows 8/16/32/L, cumulative sum, decayed sum
CHUNK = 256         # Section 4.1: eviction length L = 256 (one "chunk" of queries)
DECAY = 0.9         # Appendix B.1: per-chunk decay of the decayed cumulative sum


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    num_layers: int
    num_kv_heads: int
    group_size: int          # g: query heads per KV head
    head_dim: int            # D
    lens: Tuple[int, ...]    # cached tokens per sequence before the eviction
    budgets: Tuple[int, ...]  # B per sequence
    recent_keep: int         # R: most-recent pairs that are never evicted
    seed: int
    k_dist: str              # "normal" | "channel_lognormal" | "spikes" | "dups"
    page_size: int = 16
    scorer_hidden: int = 16  # Section 4.1: hidden width of the scorer
    activation: int = 0      # 0 = ReLU

    @property
    def batch(self) -> int:
        return len(self.lens)

    @property
    def num_q_heads(self) -> int:
        return self.num_kv_heads * self.group_size

    @property
    def feat_dim(self) -> int:
        return FEATS_PER_HEAD * self.group_size

    @property
    def x_dim(self) -> int:
        return 2 * self.head_dim + self.feat_dim


def _seed(w: Workload, tensor_id: int, layer: int = 0, seq: int = 0, step: int = 0) -> int:
    # A fixed mixing of the coordinates into one 63-bit seed.
    x = (w.seed + 1) * 0x9E3779B97F4A7C15
    for v in (tensor_id, layer, seq, step):
        x = (x ^ (v + 0x632BE59BD9B4E019)) * 0xD6E8FEB86659FD93 & 0xFFFFFFFFFFFFFFFF
        x ^= x >> 32
    return x & 0x7FFFFFFFFFFFFFFF


def _gen(w: Workload, device, tensor_id: int, layer: int = 0, seq: int = 0, step: int = 0) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_seed(w, tensor_id, layer, seq, step))
    return g


def _config4_lens(seed: int) -> Tuple[int, ...]:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 7919 + 17)
    return tuple(int(x) for x in torch.randint(4096, 32768 + 1, (16,), generator=g))


def config(idx: int, budget: int | None = None) -> Workload:
    """The five benchmark configurations (1-based): tiny, Qwen3-4B at 8K and 32K, 7B batched, 8B long-decode."""
    if idx == 1:
        return Workload("cfg1_tiny", 1, 2, 4, 64, (512,), (budget or 256,), 0, 0, "normal")
    if idx == 2:
        return Workload("cfg2_qwen3_4b_8k", 36, 8, 4, 128, (8192 + 128,), (budget or 4096,), 128, 1,
                        "channel_lognormal")
    if idx == 3:
        return Workload("cfg3_qwen3_4b_32k", 36, 8, 4, 128, (32768,), (budget or 8192,), 0, 2,
                        "channel_lognormal")
    if idx == 4:
        lens = _config4_lens(3)
        return Workload("cfg4_7b_batch16_varlen", 28, 4, 7, 128, lens, tuple(n // 2 for n in lens), 0, 3, "spikes")
    if idx == 5:
        return Workload("cfg5_8b_batch8_64k", 32, 8, 4, 128, (65536,) * 8, (budget or 16384,) * 8, 0, 4, "dups")
    raise ValueError(f"no config {idx}")


def shrink(w: Workload, num_layers: int | None = None, max_len: int | None = None, batch: int | None = None) -> Workload:
    """A smaller case with the same per-segment structure (for oracle-speed tests)."""
    lens = w.lens[: batch or len(w.lens)]
    budgets = w.budgets[: len(lens)]
    if max_len is not None:
        scale = [min(1.0, max_len / n) for n in lens]
        budgets = tuple(max(1, int(b * s)) for b, s in zip(budgets, scale))
        lens = tuple(max(1, int(n * s)) for n, s in zip(lens, scale))
    return dataclasses.replace(w, name=w.name + "_small", num_layers=num_layers or w.num_layers, lens=lens,
                               budgets=budgets)


def scorer_params(w: Workload, layer: int, device="cpu"):
    """Random-init scorer of one layer: W1 [Hkv][2D+6g][H], b1 [Hkv][H], W2 [Hkv][H], b2 [Hkv], fp32.

    U(-1/sqrt(fan_in), +1/sqrt(fan_in)), plain fp32 as a trainer would hand
    them over.
    """
    g = _gen(w, device, _T_W, layer)
    Hk, X, H = w.num_kv_heads, w.x_dim, w.scorer_hidden
    b_in, b_hid = 1.0 / math.sqrt(X), 1.0 / math.sqrt(H)
    W1 = (torch.rand((Hk, X, H), generator=g, device=device) * 2 - 1) * b_in
    b1 = (torch.rand((Hk, H), generator=g, device=device) * 2 - 1) * b_in
    W2 = (torch.rand((Hk, H), generator=g, device=device) * 2 - 1) * b_hid
    b2 = (torch.rand((Hk,), generator=g, device=device) * 2 - 1) * b_hid
    return W1.contiguous(), b1.contiguous(), W2.contiguous(), b2.contiguous()


def _features(w: Workload, layer: int, seq: int, n: int, device) -> torch.Tensor:
    """Attention-feature rows [Hkv][n][6g], fp32, >= 0.

    Per query head a heavy-tailed attention mass over the n slots with mean 1
    (the probability relative to uniform attention); the four window columns
    are that mass times U(0.5, 1.5); the cumulative sum is the mass times the
    number of chunks seen, the decayed sum the mass times sum_j 0.9^j.
    """
    g = _gen(w, device, _T_FEAT, layer, seq)
    Hk, G = w.num_kv_heads, w.group_size
    e = torch.exp(torch.randn((Hk, n, G), generator=g, device=device))
    mass = e / e.mean(dim=1, keepdim=True)
    jitter = torch.rand((Hk, n, G, 4), generator=g, device=device) + 0.5
    chunks = max(1, n // CHUNK)
    geo = (1.0 - DECAY ** chunks) / (1.0 - DECAY)
    feat = torch.empty((Hk, n, G, FEATS_PER_HEAD), device=device, dtype=torch.float32)
    feat[..., 0:4] = mass.unsqueeze(-1) * jitter
    feat[..., 4] = mass * chunks
    feat[..., 5] = mass * geo
    return feat.reshape(Hk, n, G * FEATS_PER_HEAD).contiguous()


def layer_inputs(w: Workload, layer: int, seq: int, device="cpu"):
    """Dense cache content of one (layer, sequence) before the eviction.

    Returns K, V [Hkv][n][D] bf16, feat [Hkv][n][6g] fp32, pos [n] int32
    (strictly increasing original token positions).
    """
    n, Hk, D = w.lens[seq], w.num_kv_heads, w.head_dim
    K = torch.randn((Hk, n, D), generator=_gen(w, device, _T_K, layer, seq), device=device)
    V = torch.randn((Hk, n, D), generator=_gen(w, device, _T_V, layer, seq), device=device)
    feat = _features(w, layer, seq, n, device)
    if w.k_dist == "channel_lognormal":
        # One outlier scale per (layer, head, channel), shared by all sequences.
        s = torch.exp(torch.randn((Hk, 1, D), generator=_gen(w, device, _T_SCALE, layer), device=device))
        K = K * s
    elif w.k_dist == "spikes":
        # 5 % of the positions of a sequence (the same in every layer and head) carry 4x norm.
        gs = _gen(w, device, _T_SPIKE, 0, seq)
        spike = torch.rand((n,), generator=gs, device=device) < 0.05
        f = torch.where(spike, 4.0, 1.0).view(1, n, 1)
        K, V = K * f, V * f
    K, V = K.to(torch.bfloat16), V.to(torch.bfloat16)
    if w.k_dist == "dups":
        # 1 % of the slots are exact copies (K, V and feature rows) of another
        # slot of the same segment, so their scores tie bit for bit.
        gd = _gen(w, device, _T_DUP, layer, seq)
        ndup = max(1, n // 100)
        perm = torch.randperm(n, generator=gd, device=device)
        dst, pool = perm[:ndup], perm[ndup:]
        src = pool[torch.randint(0, pool.numel(), (ndup,), generator=gd, device=device)]
        K[:, dst], V[:, dst], feat[:, dst] = K[:, src], V[:, src], feat[:, src]
    pos = torch.arange(n, device=device, dtype=torch.int32)
    return K.contiguous(), V.contiguous(), feat.contiguous(), pos


def queries(w: Workload, layer: int, step: int = 0, device="cpu") -> torch.Tensor:
    """Decode queries q [batch][Hq][D] bf16 ~ N(0,1)."""
    g = _gen(w, device, _T_Q, layer, 0, step)
    return torch.randn((w.batch, w.num_q_heads, w.head_dim), generator=g, device=device).to(torch.bfloat16)


def new_kv(w: Workload, layer: int, step: int = 0, device="cpu"):
    """The (k, v) rows one decode step appends: [batch][Hkv][D] bf16 each."""
    g = _gen(w, device, _T_NEW, layer, 0, step)
    k = torch.randn((w.batch, w.num_kv_heads, w.head_dim), generator=g, device=device).to(torch.bfloat16)
    v = torch.randn((w.batch, w.num_kv_heads, w.head_dim), generator=g, device=device).to(torch.bfloat16)
    return k, v


def gumbel_noise(w: Workload, layer: int, stride: int, event: int = 0, device="cpu") -> torch.Tensor:
    """Standard Gumbel draws g = -log(-log u) for the sampled eviction action: [batch][Hkv][stride] fp32.

    Random INPUT of the method (it has no arithmetic of the method in it): both the CPU oracle and the
    CUDA path are handed the same values.
    """
    g = _gen(w, device, _T_NOISE, layer, 0, event)
    u = torch.rand((w.batch, w.num_kv_heads, stride), generator=g, device=device, dtype=torch.float64)
    u = u.clamp_(1e-12, 1.0 - 1e-12)
    return (-torch.log(-torch.log(u))).to(torch.float32).contiguous()


def causal_attention(seed: int, g: int, T: int, device="cpu", heavy: int = 8) -> torch.Tensor:
    """Synthetic causal attention probabilities [g][T][T] fp32 (rows sum to 1) for the Golden-Eviction
    label builder: random logits, a few "heavy hitter" key positions that many queries attend to, and a
    recency bias - the patterns the paper's Figure 1 describes.  Input data only."""
    gen = torch.Generator(device=device)
    gen.manual_seed(0x5EED0000 + seed)
    logits = torch.randn((g, T, T), generator=gen, device=device)
    hh = torch.randperm(T, generator=gen, device=device)[:heavy]
    logits[:, :, hh] += 3.0
    r = torch.arange(T, device=device)
    logits = logits - 0.002 * (r.view(1, T, 1) - r.view(1, 1, T)).clamp(min=0)
    logits = logits.masked_fill(r.view(1, 1, T) > r.view(1, T, 1), float("-inf"))
    return torch.softmax(logits, dim=-1).contiguous()


def segment_list(w: Workload) -> List[Tuple[int, int, int]]:
    """All (layer, seq, kv_head) segments of a workload."""
    return [(l, s, h) for l in range(w.num_layers) for s in range(w.batch) for h in range(w.num_kv_heads)]
