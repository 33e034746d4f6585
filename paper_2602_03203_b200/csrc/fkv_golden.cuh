// Golden Eviction labels (Section 3.2, Eq. 3-5): the supervision targets of the scorer, built from the
// full attention matrix of one attention group.
//   block score   a~_t[i]     = average over the g heads and the L query rows of block t of A[h][r][i]
//                               (blocks start at the first eviction position B + L; the last is zero-padded)
//   future score  alpha[t][i] = max over j >= t of a~_j[i]
//   retained set  s_t         = the B - L cached pairs with the largest alpha[t][.] (ties: lower position)
// Three kernels: a streaming column reduction of A (HBM bound: every needed element of A is read once,
// coalesced along the key axis), a suffix maximum over the blocks, and a sequential selection - one CTA
// walks the M eviction steps, each a histogram select of the (B - L)-th largest key over the B cached
// pairs followed by an ordered compaction of the survivors with a block prefix sum.
#pragma once
#include "fkv_dev.cuh"
#include "fkv_select.cuh"

namespace fkv {

// grid (ceil(T / 256), M), 256 threads: thread = key column i, block t = blockIdx.y + 1.
__global__ void __launch_bounds__(256) k_golden_pool(const float *A, int g, int T, int B, int L, float *blocks) {
  const int i = blockIdx.x * 256 + threadIdx.x, t = blockIdx.y + 1;
  if (i >= T) return;
  const int r0 = B + t * L, r1 = min(T, r0 + L);
  float acc = 0.f;
  for (int h = 0; h < g; ++h) {
    const float *col = A + ((size_t)h * T + r0) * T + i;
    int r = r0;
    for (; r + 8 <= r1; r += 8, col += (size_t)8 * T) {   // eight loads in flight
      float x[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) x[u] = __ldg(col + (size_t)u * T);
#pragma unroll
      for (int u = 0; u < 8; ++u) acc += x[u];
    }
    for (; r < r1; ++r, col += T) acc += __ldg(col);
  }
  blocks[(size_t)(t - 1) * T + i] = acc / ((float)g * (float)L);
}

// grid ceil(T / 256): alpha[t][i] = max(block[t][i], alpha[t + 1][i]), in place, last block first.
__global__ void __launch_bounds__(256) k_golden_suffix_max(float *alpha, int T, int M) {
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= T) return;
  float run = -INFINITY;
  for (int t = M - 1; t >= 0; --t) {
    const float v = alpha[(size_t)t * T + i];
    run = v > run ? v : run;
    alpha[(size_t)t * T + i] = run;
  }
}

// One CTA of 1024 threads walks the M steps; dynamic shared memory: the cached positions [B].  Thread `tid` owns
// the consecutive cache entries [tid * per, tid * per + per) (per = ceil(B / 1024) <= 8) and keeps their score keys
// in registers.  Per step: the (B - L)-th largest key T is found with histogram passes over 2048 bins that follow
// the data (window [min, max], narrowed to the bin where the count from the top crosses B - L: at most three
// passes for 32-bit keys), then one ordered pass keeps {key > T} and the first `need` entries with key == T in
// cache order (= position order, the tie-break), placed by a block prefix sum.  kept: [M][B - L].
__global__ void __launch_bounds__(1024) k_golden_select(const float *alpha, int T, int B, int L, int M,
                                                         int32_t *kept) {
  extern __shared__ __align__(16) uint8_t gsm[];
  constexpr int kBins = 2048, kLogBins = 11, kPer = 8;
  __shared__ unsigned s_hist[kBins];
  __shared__ int s_scan[33];
  __shared__ unsigned s_red[64];
  __shared__ unsigned s_bin, s_krem;
  __shared__ unsigned long long s_wsum[33];
  int *cache = reinterpret_cast<int *>(gsm);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = (B + 1023) / 1024, j0 = min(B, tid * per), j1 = min(B, j0 + per), nm = j1 - j0;
  const int k = B - L;
  for (int j = tid; j < B; j += 1024) cache[j] = j;
  __syncthreads();
  for (int t = 1; t <= M; ++t) {
    const float *a = alpha + (size_t)(t - 1) * T;
    uint32_t key[kPer];
    int pos[kPer];
#pragma unroll
    for (int u = 0; u < kPer; ++u) {
      pos[u] = u < nm ? cache[j0 + u] : 0;
      key[u] = u < nm ? score_key(__ldg(a + pos[u])) : 0u;
    }
    // ---- key window ----
    uint32_t kmin = 0xffffffffu, kmax = 0u;
#pragma unroll
    for (int u = 0; u < kPer; ++u)
      if (u < nm) { kmin = min(kmin, key[u]); kmax = max(kmax, key[u]); }
    kmin = __reduce_min_sync(0xffffffffu, kmin);
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    if (lane == 0) { s_red[warp] = kmin; s_red[32 + warp] = kmax; }
    __syncthreads();
    kmin = __reduce_min_sync(0xffffffffu, s_red[lane]);
    kmax = __reduce_max_sync(0xffffffffu, s_red[32 + lane]);
    uint32_t Tk = kmin;
    unsigned need = (unsigned)k;
    if (kmin != kmax) {
      uint32_t lo = kmin, wmax = kmax - kmin;   // window: keys with key - lo <= wmax
      unsigned krem = (unsigned)k;
      int bits = 32 - __clz(wmax);
      for (;;) {
        const int shift = bits > kLogBins ? bits - kLogBins : 0;
        for (int b = tid; b < kBins; b += 1024) s_hist[b] = 0;
        __syncthreads();
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
          const uint32_t d = key[u] - lo;
          if (u < nm && key[u] >= lo && d <= wmax) atomicAdd(&s_hist[d >> shift], 1u);
        }
        __syncthreads();
        {   // bins in descending order, two per thread
          const unsigned v0 = s_hist[kBins - 1 - 2 * tid], v1 = s_hist[kBins - 2 - 2 * tid];
          int tot;
          const unsigned above = (unsigned)block_excl_scan((int)(v0 + v1), s_scan, tot);
          if (above < krem && krem <= above + v0) {
            s_bin = kBins - 1 - 2 * tid; s_krem = krem - above;
          } else if (above + v0 < krem && krem <= above + v0 + v1) {
            s_bin = kBins - 2 - 2 * tid; s_krem = krem - above - v0;
          }
        }
        __syncthreads();
        lo += s_bin << shift;
        krem = s_krem;
        __syncthreads();
        if (shift == 0) break;
        wmax = (1u << shift) - 1u;
        bits = shift;
      }
      Tk = lo;
      need = krem;   // entries with key == Tk still to keep, lowest cache index first
    }
    // ---- ordered emit: block prefix sums of (greater, equal) counts packed in 64 bits ----
    unsigned cgt = 0, ceq = 0;
#pragma unroll
    for (int u = 0; u < kPer; ++u) {
      cgt += (u < nm && key[u] > Tk);
      ceq += (u < nm && key[u] == Tk);
    }
    const unsigned long long v = (unsigned long long)cgt | ((unsigned long long)ceq << 32);
    unsigned long long inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long x = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += x;
    }
    if (lane == 31) s_wsum[warp] = inc;
    __syncthreads();   // also: every thread has read its cache entries
    if (warp == 0) {
      const unsigned long long w = s_wsum[lane];
      unsigned long long winc = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long x = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += x;
      }
      s_wsum[lane] = winc - w;
    }
    __syncthreads();
    const unsigned long long excl = s_wsum[warp] + inc - v;
    unsigned bgt = (unsigned)(excl & 0xffffffffu), beq = (unsigned)(excl >> 32);
    int32_t *out = kept + (size_t)(t - 1) * k;
#pragma unroll
    for (int u = 0; u < kPer; ++u) {
      const bool g = u < nm && key[u] > Tk, e = u < nm && key[u] == Tk;
      if (g || (e && beq < need)) {
        const int dst = (int)(bgt + min(beq, need));
        cache[dst] = pos[u];
        out[dst] = pos[u];
      }
      bgt += g; beq += e;
    }
    for (int j = tid; j < L; j += 1024) cache[k + j] = B + (t - 1) * L + j;   // they leave the recent window next
    __syncthreads();
  }
}

}  // namespace fkv
