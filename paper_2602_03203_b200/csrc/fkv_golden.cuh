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
  constexpr int kPer = 8;
  __shared__ SelShared<1024> sh;
  int *cache = reinterpret_cast<int *>(gsm);
  const int tid = threadIdx.x;
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
    // The (B - L)-th largest key and the ordered places: the selection kernel's own routines (one round, the keys in
    // registers), so that the tie-break rule lives in one place.
    uint32_t Tk;
    unsigned need;
    int nv = nm;
    sel_kth_key<1024, kPer>(sh, key, nv, 1, [](int) {}, SelAlone{}, (unsigned)k, Tk, need);
    unsigned long long total;
    const unsigned long long excl = sel_counts_before<1024, kPer>(sh, key, nv, Tk, total);   // its barriers: every thread has read its cache entries
    unsigned bgt = (unsigned)(excl & 0xffffffffu), beq = (unsigned)(excl >> 32);
    int32_t *out = kept + (size_t)(t - 1) * k;
#pragma unroll
    for (int u = 0; u < kPer; ++u) {
      const bool g = u < nm && key[u] > Tk, e = u < nm && key[u] == Tk;
      const int dst = sel_place(g, e, bgt, beq, need);
      if (dst >= 0) {
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
