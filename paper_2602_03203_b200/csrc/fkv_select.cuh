// Kernel 2: per-segment top-k selection (Section 3.1, deterministic Top-K
// action): among slots [0, n - r) keep the k pairs with the highest scores,
// ties going to the lower slot; then the r most recent slots.  The kept slots
// are written in ascending order, which is the order compaction needs.
//
// Integer work on 4 bytes per pair, read from L2 right after the scorer wrote
// them.  One CTA per segment: a 4 x 8-bit most-significant-digit radix select
// finds the k-th largest key T and how many pairs equal to T are still needed;
// one ordered pass then emits {key > T} plus the first `need` slots with
// key == T, using block prefix sums - no atomics decide which tied pair stays.
#pragma once
#include "fkv_dev.cuh"

namespace fkv {

// Order-preserving key of a score: -0 -> +0, NaN -> -inf, then the usual
// sign-flip so that unsigned order equals float order.
__device__ __forceinline__ uint32_t score_key(float s) {
  if (s != s) s = -INFINITY;
  if (s == 0.f) s = 0.f;
  const uint32_t u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kSelThreads = 1024;

// scores/idx: row (seg - seg_base) * cap.  kept_count (optional): [seg - seg_base].
__global__ void __launch_bounds__(kSelThreads) k_select(Ctx c, const float *scores, int32_t *idx, int32_t *kept_count,
                                                         int seg_base) {
  __shared__ unsigned s_hist[256];
  __shared__ int s_scan[33];
  __shared__ unsigned s_digit, s_krem;
  __shared__ unsigned long long s_wsum[33];
  if ((int)blockIdx.x >= c.planhdr[PH_NWORK]) return;
  const int seg = c.work[blockIdx.x];
  const SegPlan p = c.plan[seg];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int m = p.n_old - p.r, k = p.k_sel;
  const float *sc = scores + (size_t)(seg - seg_base) * c.cap;
  int32_t *out = idx + (size_t)(seg - seg_base) * c.cap;
  if (kept_count && tid == 0) kept_count[seg - seg_base] = p.n_new;
  // The protected recent slots close the list.
  for (int j = tid; j < p.r; j += kSelThreads) out[k + j] = m + j;
  if (k <= 0) return;
  if (k >= m) {
    for (int j = tid; j < m; j += kSelThreads) out[j] = j;
    return;
  }

  // ---- radix select of the k-th largest key ----
  uint32_t prefix = 0, mask = 0;
  unsigned krem = (unsigned)k;
  const float4 *sc4 = reinterpret_cast<const float4 *>(sc);
  const int m4 = (m + 3) >> 2;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) s_hist[tid] = 0;
    __syncthreads();
    for (int i = tid; i < ((m4 + kSelThreads - 1) / kSelThreads) * kSelThreads; i += kSelThreads) {
      float4 x = i < m4 ? sc4[i] : make_float4(0, 0, 0, 0);
      const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t key = score_key(xs[e]);
        const bool valid = (i * 4 + e) < m && (key & mask) == prefix;
        // One shared-memory atomic per distinct digit in the warp.
        const unsigned digit = valid ? ((key >> shift) & 255u) : 0xffffffffu;
        const unsigned peers = __match_any_sync(0xffffffffu, digit);
        if (valid && lane == (__ffs(peers) - 1)) atomicAdd(&s_hist[digit], (unsigned)__popc(peers));
      }
    }
    __syncthreads();
    // Digit d is chosen when (#keys with a larger digit) < krem <= (that + hist[d]).
    {
      const int v = tid < 256 ? (int)s_hist[255 - tid] : 0;  // descending digits
      int tot;
      const int above = block_excl_scan(v, s_scan, tot);
      if (tid < 256 && (unsigned)above < krem && krem <= (unsigned)(above + v)) {
        s_digit = 255u - tid;
        s_krem = krem - (unsigned)above;
      }
    }
    __syncthreads();
    prefix |= s_digit << shift;
    mask |= 255u << shift;
    krem = s_krem;
    __syncthreads();
  }
  const uint32_t T = prefix;
  const unsigned need = krem;  // pairs with key == T still to keep, lowest slots first

  // ---- ordered emit ----
  unsigned run_gt = 0, run_eq = 0;
  for (int base = 0; base < m4; base += kSelThreads) {
    const int i = base + tid;
    float4 x = i < m4 ? sc4[i] : make_float4(0, 0, 0, 0);
    const float xs[4] = {x.x, x.y, x.z, x.w};
    unsigned gt[4], eq[4], cgt = 0, ceq = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint32_t key = score_key(xs[e]);
      const bool in = (i * 4 + e) < m;
      gt[e] = in && key > T; eq[e] = in && key == T;
      cgt += gt[e]; ceq += eq[e];
    }
    // Exclusive block scan of (cgt, ceq) packed in 64 bits.
    unsigned long long v = (unsigned long long)cgt | ((unsigned long long)ceq << 32), inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += t;
    }
    __syncthreads();
    if (lane == 31) s_wsum[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      unsigned long long w = s_wsum[lane], winc = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        unsigned long long t = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += t;
      }
      s_wsum[lane] = winc - w;
      if (lane == 31) s_wsum[32] = winc;
    }
    __syncthreads();
    const unsigned long long excl = s_wsum[warp] + inc - v, tot = s_wsum[32];
    unsigned bgt = run_gt + (unsigned)(excl & 0xffffffffu), beq = run_eq + (unsigned)(excl >> 32);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (gt[e]) out[bgt + min(beq, need)] = i * 4 + e;
      else if (eq[e] && beq < need) out[bgt + beq] = i * 4 + e;
      bgt += gt[e]; beq += eq[e];
    }
    run_gt += (unsigned)(tot & 0xffffffffu);
    run_eq += (unsigned)(tot >> 32);
  }
}

}  // namespace fkv
