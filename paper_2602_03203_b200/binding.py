"""Thin ctypes binding of the C ABI in ``include/fkv.h``.

Argument marshalling only: every step of the path runs in the CUDA library.
torch is used for device memory and streams.  There is no CPU fallback: if the
library has not been built, or no CUDA device is present, calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfkv.so")
_lib = None

ALL_LAYERS = -1
ACT_RELU, ACT_SILU, ACT_GELU_TANH, ACT_SIGMOID = 0, 1, 2, 3
DEV_POOL_EXHAUSTED, DEV_CAPACITY, DEV_WAIT_TIMEOUT, DEV_BAD_INDEX = 1, 2, 4, 8
STATUS = {0: "FKV_OK", -1: "FKV_ERR_INVALID_ARG", -2: "FKV_ERR_WORKSPACE_TOO_SMALL", -3: "FKV_ERR_CAPACITY",
          -4: "FKV_ERR_CUDA", -5: "FKV_ERR_NOT_READY", -6: "FKV_ERR_DEVICE"}

EXPORTS = ["fkv_workspace_bytes", "fkv_init_cache", "fkv_destroy", "fkv_reset", "fkv_load_scorer", "fkv_set_budget",
           "fkv_prefill", "fkv_append", "fkv_set_features", "fkv_evict", "fkv_decode_attn", "fkv_score", "fkv_select",
           "fkv_compact", "fkv_score_stride", "fkv_export_head", "fkv_get_lengths", "fkv_device_status",
           "fkv_launch_count", "fkv_last_cuda_error", "fkv_sync_lengths", "fkv_set_timing", "fkv_get_evict_timing",
           "fkv_decode_step", "fkv_decode_attn_dense_noalloc", "fkv_append_decode_attn", "fkv_evict_sampled", "fkv_select_sampled", "fkv_update_features", "fkv_evict_by_feature", "fkv_golden_steps", "fkv_golden_eviction", "fkv_golden_select",
           "fkv_evict_rkv", "fkv_score_rkv"]


class FkvConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "num_layers", "num_kv_heads", "group_size", "head_dim", "max_batch", "page_size", "scorer_hidden",
        "activation", "budget", "recent_keep", "max_tokens_per_head", "num_pages", "feature_window")]


class FkvError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = f"{where}: {STATUS.get(code, code)}"
        if code == -4:
            msg += f" ({lib().fkv_last_cuda_error().decode()})"
        super().__init__(msg)


def lib():
    """The loaded CUDA library.  Raises if it has not been built (no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_03203_b200.build`")
        _lib = ctypes.CDLL(LIB_PATH)
        for name in EXPORTS:
            getattr(_lib, name).restype = ctypes.c_int
        _lib.fkv_last_cuda_error.restype = ctypes.c_char_p
        vp, i32, u64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint64, ctypes.c_float
        # Declared argument types for the per-token calls: plain ints and floats are converted by ctypes itself.
        _lib.fkv_append.argtypes = [vp, i32, vp, vp, vp, vp, vp]
        _lib.fkv_decode_attn.argtypes = [vp, i32, vp, vp, f32, vp]
        _lib.fkv_append_decode_attn.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, f32, vp]
        _lib.fkv_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, f32, vp]
        _lib.fkv_evict.argtypes = [vp, i32, vp]
    return _lib


def _check(code: int, where: str):
    if code != 0:
        raise FkvError(code, where)


def _ptr(t: Optional[torch.Tensor], dtype=None, device_type="cuda"):
    """Address of a contiguous tensor on the expected device (NULL for None)."""
    if t is None:
        return ctypes.c_void_p(0)
    if not t.is_contiguous() or t.is_cuda != (device_type == "cuda") or (dtype is not None and t.dtype is not dtype):
        raise ValueError(f"expected a contiguous {dtype} tensor on {device_type}, got {t.dtype} on {t.device}, "
                         f"contiguous={t.is_contiguous()}")
    return ctypes.c_void_p(t.data_ptr())


try:   # the raw handle of torch's current stream without building a Stream object (a hot-path saving)
    _raw_stream = torch._C._cuda_getCurrentRawStream
except AttributeError:   # pragma: no cover
    _raw_stream = None


def _mask(seq_mask, max_batch):
    """A Python integer with bit s set for every sequence that takes part (0 or None: all) as the host bit
    array the library reads: (array or None to keep alive, pointer)."""
    if not seq_mask:
        return None, ctypes.c_void_p(0)
    words = (max_batch + 63) // 64
    arr = (ctypes.c_uint64 * words)(*[(seq_mask >> (64 * i)) & 0xFFFFFFFFFFFFFFFF for i in range(words)])
    return arr, ctypes.cast(arr, ctypes.c_void_p)


def _stream():
    if _raw_stream is not None:
        return ctypes.c_void_p(_raw_stream(torch.cuda.current_device()))
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


class Cache:
    """One budgeted KV cache on the current CUDA device (see include/fkv.h for the semantics)."""

    def __init__(self, num_layers, num_kv_heads, group_size, head_dim, max_batch, budget, max_tokens_per_head,
                 recent_keep=0, activation=ACT_RELU, num_pages=0, page_size=16, scorer_hidden=16, feature_window=0,
                 workspace=None):
        if not torch.cuda.is_available():
            raise RuntimeError("fkv needs a CUDA device; there is no CPU path")
        self.cfg = FkvConfig(num_layers, num_kv_heads, group_size, head_dim, max_batch, page_size, scorer_hidden,
                             activation, budget, recent_keep, max_tokens_per_head, num_pages, feature_window)
        nbytes = ctypes.c_size_t(0)
        _check(lib().fkv_workspace_bytes(ctypes.byref(self.cfg), ctypes.byref(nbytes)), "fkv_workspace_bytes")
        self.workspace_bytes = nbytes.value
        # The caller may bring the workspace (a CUDA uint8 tensor of at least workspace_bytes + 255 bytes); the
        # library only ever touches [base, base + workspace_bytes) of it.
        if workspace is None:
            workspace = torch.empty(nbytes.value + 256, dtype=torch.uint8, device="cuda")
        if workspace.dtype != torch.uint8 or not workspace.is_cuda or not workspace.is_contiguous():
            raise ValueError("workspace must be a contiguous CUDA uint8 tensor")
        self.workspace = workspace
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        if base + nbytes.value > self.workspace.data_ptr() + self.workspace.numel():
            raise ValueError(f"workspace too small: {self.workspace.numel()} bytes, need {nbytes.value} + alignment")
        self.workspace_offset = base - self.workspace.data_ptr()
        self._h = ctypes.c_void_p(0)
        _check(lib().fkv_init_cache(ctypes.byref(self.cfg), ctypes.c_void_p(base), ctypes.c_size_t(nbytes.value),
                                    _stream(), ctypes.byref(self._h)), "fkv_init_cache")
        cap = ctypes.c_int32(0)
        _check(lib().fkv_score_stride(self._h, ctypes.byref(cap)), "fkv_score_stride")
        self.cap = cap.value
        self.feat_dim = 6 * group_size

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().fkv_destroy(self._h)
            self._h = ctypes.c_void_p(0)
            self.workspace = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- set-up
    def reset(self):
        _check(lib().fkv_reset(self._h, _stream()), "fkv_reset")

    def load_scorer(self, layer, kv_head, W1, b1, W2, b2):
        W1, b1, W2 = (x.detach().to("cpu", torch.float32).contiguous() for x in (W1, b1, W2))
        _check(lib().fkv_load_scorer(self._h, layer, kv_head, _ptr(W1, torch.float32, "cpu"),
                                     _ptr(b1, torch.float32, "cpu"), _ptr(W2, torch.float32, "cpu"),
                                     ctypes.c_float(float(b2)), _stream()), "fkv_load_scorer")

    def load_scorers(self, layer, W1, b1, W2, b2):
        """All KV heads of a layer: W1 [Hkv][2D+F][H], b1 [Hkv][H], W2 [Hkv][H], b2 [Hkv]."""
        W1, b1, W2, b2 = (x.detach().to("cpu", torch.float32) for x in (W1, b1, W2, b2))
        for h in range(self.cfg.num_kv_heads):
            self.load_scorer(layer, h, W1[h], b1[h], W2[h], float(b2[h]))

    def set_budget(self, seq, budget):
        _check(lib().fkv_set_budget(self._h, seq, int(budget), _stream()), "fkv_set_budget")

    def prefill(self, layer, seq, k, v, feat=None, pos=None):
        n = k.shape[1]
        _check(lib().fkv_prefill(self._h, layer, seq, _ptr(k, torch.bfloat16), _ptr(v, torch.bfloat16),
                                 _ptr(feat, torch.float32), _ptr(pos, torch.int32), n, _stream()), "fkv_prefill")

    def set_features(self, layer, seq, feat):
        _check(lib().fkv_set_features(self._h, layer, seq, _ptr(feat, torch.float32), _stream()), "fkv_set_features")

    # -- the four calls of the path
    def append(self, layer, k, v, pos=None, seq_mask=0):
        keep, m = _mask(seq_mask, self.cfg.max_batch)
        _check(lib().fkv_append(self._h, layer, _ptr(k, torch.bfloat16), _ptr(v, torch.bfloat16),
                                _ptr(pos, torch.int32), m, _stream()), "fkv_append")

    def evict(self, layer=ALL_LAYERS):
        _check(lib().fkv_evict(self._h, layer, _stream()), "fkv_evict")

    def evict_sampled(self, noise, layer=ALL_LAYERS):
        """The paper's sampled action; noise [layers of the call][batch][Hkv][stride] standard Gumbel draws."""
        _check(lib().fkv_evict_sampled(self._h, layer, _ptr(noise, torch.float32), int(noise.shape[-1]), _stream()),
               "fkv_evict_sampled")

    def evict_by_feature(self, column, layer=ALL_LAYERS):
        """Baseline eviction: score = one feature column (4: H2O cumulative attention, 0: SnapKV last-8 window)."""
        _check(lib().fkv_evict_by_feature(self._h, layer, int(column), _stream()), "fkv_evict_by_feature")

    def evict_rkv(self, layer=ALL_LAYERS, lambda_attn=0.1, lambda_sim=0.9):
        """Baseline eviction by the R-KV score: lambda_attn * window attention - lambda_sim * max cosine to another key."""
        _check(lib().fkv_evict_rkv(self._h, layer, ctypes.c_float(lambda_attn), ctypes.c_float(lambda_sim), _stream()),
               "fkv_evict_rkv")

    def score_rkv(self, layer, lambda_attn=0.1, lambda_sim=0.9, out=None):
        if out is None:
            out = torch.zeros((self.cfg.max_batch, self.cfg.num_kv_heads, self.cap), dtype=torch.float32, device="cuda")
        _check(lib().fkv_score_rkv(self._h, layer, ctypes.c_float(lambda_attn), ctypes.c_float(lambda_sim),
                                   _ptr(out, torch.float32), _stream()), "fkv_score_rkv")
        return out

    def decode_attn(self, layer, q, out=None, scale=0.0):
        if out is None:
            out = torch.empty_like(q)
        _check(lib().fkv_decode_attn(self._h, layer, _ptr(q, torch.bfloat16), _ptr(out, torch.bfloat16), scale,
                                     _stream()), "fkv_decode_attn")
        return out

    def append_decode_attn(self, layer, k, v, q, out=None, pos=None, seq_mask=0, scale=0.0):
        """append(k, v) then decode_attn(q) on one layer, as one launch."""
        if out is None:
            out = torch.empty_like(q)
        keep, m = _mask(seq_mask, self.cfg.max_batch)
        _check(lib().fkv_append_decode_attn(self._h, layer, _ptr(k, torch.bfloat16), _ptr(v, torch.bfloat16),
                                            _ptr(pos, torch.int32), m, _ptr(q, torch.bfloat16),
                                            _ptr(out, torch.bfloat16), scale, _stream()), "fkv_append_decode_attn")
        return out

    def bound_append_decode_attn(self, layer, k, v, q, out, pos=None, seq_mask=0, scale=0.0):
        """The same call with its arguments checked and marshalled once: returns a function of no arguments that
        enqueues append + attention on `layer` over these (fixed) tensors on the stream current at THIS call, and
        raises on a non-zero status.  For decode loops that reuse their k / v / q / out buffers, where the
        per-call conversion of ten arguments costs more host time than the kernel takes."""
        fn = lib().fkv_append_decode_attn
        mask_arr, m = _mask(seq_mask, self.cfg.max_batch)
        args = (self._h, layer, _ptr(k, torch.bfloat16), _ptr(v, torch.bfloat16), _ptr(pos, torch.int32), m,
                _ptr(q, torch.bfloat16), _ptr(out, torch.bfloat16), scale, _stream())
        keep = (k, v, q, out, pos, mask_arr)   # the tensors stay alive as long as the function does

        def call(_fn=fn, _args=args, _keep=keep):
            code = _fn(*_args)
            if code:
                raise FkvError(code, "fkv_append_decode_attn")
        return call

    def decode_step(self, k, v, q, out=None, pos=None, scale=0.0):
        """One token through all layers: k, v [L][batch][Hkv][D]; q, out [L][batch][Hq][D]."""
        if out is None:
            out = torch.empty_like(q)
        _check(lib().fkv_decode_step(self._h, _ptr(k, torch.bfloat16), _ptr(v, torch.bfloat16), _ptr(pos, torch.int32),
                                     _ptr(q, torch.bfloat16), _ptr(out, torch.bfloat16), scale, _stream()),
               "fkv_decode_step")
        return out

    # -- staged entry points
    def score(self, layer, out=None):
        if out is None:
            out = torch.zeros((self.cfg.max_batch, self.cfg.num_kv_heads, self.cap), dtype=torch.float32, device="cuda")
        _check(lib().fkv_score(self._h, layer, _ptr(out, torch.float32), _stream()), "fkv_score")
        return out

    def select(self, layer, scores):
        idx = torch.full((self.cfg.max_batch, self.cfg.num_kv_heads, self.cap), -1, dtype=torch.int32, device="cuda")
        cnt = torch.zeros((self.cfg.max_batch, self.cfg.num_kv_heads), dtype=torch.int32, device="cuda")
        _check(lib().fkv_select(self._h, layer, _ptr(scores, torch.float32), _ptr(idx, torch.int32),
                                _ptr(cnt, torch.int32), _stream()), "fkv_select")
        return idx, cnt

    def select_sampled(self, layer, scores, noise):
        idx = torch.full((self.cfg.max_batch, self.cfg.num_kv_heads, self.cap), -1, dtype=torch.int32, device="cuda")
        cnt = torch.zeros((self.cfg.max_batch, self.cfg.num_kv_heads), dtype=torch.int32, device="cuda")
        _check(lib().fkv_select_sampled(self._h, layer, _ptr(scores, torch.float32), _ptr(noise, torch.float32),
                                        int(noise.shape[-1]), _ptr(idx, torch.int32), _ptr(cnt, torch.int32), _stream()),
               "fkv_select_sampled")
        return idx, cnt

    def update_features(self, layer):
        _check(lib().fkv_update_features(self._h, layer, _stream()), "fkv_update_features")

    def compact(self, layer, idx, cnt):
        _check(lib().fkv_compact(self._h, layer, _ptr(idx, torch.int32), _ptr(cnt, torch.int32), _stream()),
               "fkv_compact")

    def export_head(self, layer, seq, kv_head):
        n = self.lengths(layer)[seq]
        D, F = self.cfg.head_dim, self.feat_dim
        k = torch.empty((n, D), dtype=torch.bfloat16, device="cuda")
        v = torch.empty((n, D), dtype=torch.bfloat16, device="cuda")
        feat = torch.empty((n, F), dtype=torch.float32, device="cuda")
        pos = torch.empty((n,), dtype=torch.int32, device="cuda")
        _check(lib().fkv_export_head(self._h, layer, seq, kv_head, _ptr(k), _ptr(v), _ptr(feat), _ptr(pos), _stream()),
               "fkv_export_head")
        return k, v, feat, pos

    def lengths(self, layer):
        arr = (ctypes.c_int32 * self.cfg.max_batch)()
        _check(lib().fkv_get_lengths(self._h, layer, arr), "fkv_get_lengths")
        return list(arr)

    def device_status(self):
        """(status bits, free pages); syncs the stream and clears the bits."""
        bits, free = ctypes.c_uint32(0), ctypes.c_int32(0)
        code = lib().fkv_device_status(self._h, ctypes.byref(bits), ctypes.byref(free), _stream())
        if code not in (0, -6):
            raise FkvError(code, "fkv_device_status")
        return bits.value, free.value

    def sync_lengths(self):
        _check(lib().fkv_sync_lengths(self._h, _stream()), "fkv_sync_lengths")

    def snapshot(self) -> torch.Tensor:
        """A copy of the whole workspace (cache content, page tables, lengths, scorers)."""
        torch.cuda.current_stream().synchronize()
        return self.workspace.clone()

    def restore(self, snap: torch.Tensor):
        """Put a snapshot back (device-to-device copy) and refresh the host mirror of the lengths."""
        self.workspace.copy_(snap)
        self.sync_lengths()

    def set_timing(self, on: bool):
        _check(lib().fkv_set_timing(self._h, int(on)), "fkv_set_timing")

    def evict_timing(self):
        """Milliseconds of the last timed fkv_evict: dict plan/score/select/compact/commit/features."""
        arr = (ctypes.c_float * 6)()
        _check(lib().fkv_get_evict_timing(self._h, arr), "fkv_get_evict_timing")
        return dict(zip(("plan", "score", "select", "compact", "commit", "features"), (float(x) for x in arr)))

    def launch_count(self):
        n = ctypes.c_uint64(0)
        _check(lib().fkv_launch_count(self._h, ctypes.byref(n)), "fkv_launch_count")
        return n.value


def decode_attn_dense_noalloc(q, k, v, group_size, out=None, scale=0.0):
    """Decode attention over dense K/V with no allocation inside the library.

    For callers that cannot give the library a workspace (a frozen memory pool, a host
    process that owns all of HBM): q [Hkv*g][D], k, v [Hkv][n][D], all bf16 on the device.
    The split-K partials sit in a fixed array inside the library; calls must not overlap
    on the GPU.  Returns out [Hkv*g][D] (pass `out` to avoid torch allocating it).
    """
    Hkv, n, D = k.shape
    if out is None:
        out = torch.empty_like(q)
    code = lib().fkv_decode_attn_dense_noalloc(_ptr(q, torch.bfloat16), _ptr(k, torch.bfloat16),
                                               _ptr(v, torch.bfloat16), n, Hkv, group_size, D, ctypes.c_float(scale),
                                               _ptr(out, torch.bfloat16), _stream())
    _check(code, "fkv_decode_attn_dense_noalloc")
    return out


def golden_eviction(attn, B, L):
    """Golden Eviction labels of one attention group: attn [g][T][T] fp32 on the device.
    Returns (alpha [M][T], kept [M][B - L])."""
    g, T, _ = attn.shape
    M = lib().fkv_golden_steps(T, int(B), int(L))
    if M < 0:
        raise FkvError(M, "fkv_golden_steps")
    alpha = torch.empty((M, T), dtype=torch.float32, device="cuda")
    kept = torch.empty((M, B - L), dtype=torch.int32, device="cuda")
    _check(lib().fkv_golden_eviction(_ptr(attn, torch.float32), g, T, int(B), int(L), _ptr(alpha, torch.float32),
                                     _ptr(kept, torch.int32), _stream()), "fkv_golden_eviction")
    return alpha, kept


def golden_select(alpha, B, L):
    M, T = alpha.shape
    kept = torch.empty((M, B - L), dtype=torch.int32, device="cuda")
    _check(lib().fkv_golden_select(_ptr(alpha, torch.float32), T, int(B), int(L), M, _ptr(kept, torch.int32), _stream()),
           "fkv_golden_select")
    return kept


def pages_for(w, num_layers=None, extra_tokens=256) -> int:
    """Pool pages that hold every sequence of `w` at its own length plus `extra_tokens`, and the
    fresh pages an all-layer eviction takes before it returns the old ones."""
    L = num_layers or w.num_layers
    per_head = sum(-(-(n + extra_tokens) // w.page_size) + -(-min(b, n) // w.page_size) + 1
                   for n, b in zip(w.lens, w.budgets))
    return L * w.num_kv_heads * per_head


def workspace_bytes_for(w, num_layers=None, num_pages=0, max_tokens=None) -> int:
    """Bytes of device workspace ``from_workload`` would allocate (no device access)."""
    cfg = FkvConfig(num_layers or w.num_layers, w.num_kv_heads, w.group_size, w.head_dim, w.batch, w.page_size,
                    w.scorer_hidden, w.activation, max(w.budgets), w.recent_keep,
                    max_tokens or (max(w.lens) + 256), num_pages, 0)
    nbytes = ctypes.c_size_t(0)
    _check(lib().fkv_workspace_bytes(ctypes.byref(cfg), ctypes.byref(nbytes)), "fkv_workspace_bytes")
    return nbytes.value


def from_workload(w, num_layers=None, num_pages=0, max_tokens=None, feature_window=0, workspace=None) -> Cache:
    """A cache shaped for a ``workloads.Workload`` with per-sequence budgets set."""
    L = num_layers or w.num_layers
    c = Cache(L, w.num_kv_heads, w.group_size, w.head_dim, w.batch, max(w.budgets),
              max_tokens or (max(w.lens) + 256), recent_keep=w.recent_keep, activation=w.activation,
              num_pages=num_pages, feature_window=feature_window, workspace=workspace)
    for s, b in enumerate(w.budgets):
        if b != max(w.budgets):
            c.set_budget(s, b)
    return c
