// Golden Eviction labels (Section 3.2, Eq. 3-5): the supervision targets of the scorer, built from the
// full attention matrix of one attention group.
//   block score   a~_t[i]     = average over the g heads and the L query rows of block t of A[h][r][i]
//                               (blocks start at the first eviction position B + L; the last is zero-padded)
//   future score  alpha[t][i] = max over j >= t of a~_j[i]
//   retained set  s_t         = the B - L cached pairs with the largest alpha[t][.] (ties: lower position)
// Three kernels: a streaming column reduction of A (HBM bound: every needed element of A is read once,
// coalesced along the key axis), a suffix maximum over the blocks, and a sequential selection - one CTA
// walks the M eviction steps, ranking the B cached pairs with a bitonic sort of (score key, index) in
// shared memory and compacting the survivors in position order with a block prefix sum.
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

// One CTA of 1024 threads; dynamic shared memory: keys [P] 64-bit (P = power of two >= B), cached
// positions [B], flags [B].  kept: [M][B - L].
__global__ void __launch_bounds__(1024) k_golden_select(const float *alpha, int T, int B, int L, int M, int P,
                                                         int32_t *kept) {
  extern __shared__ __align__(16) uint8_t gsm[];
  __shared__ int s_scan[33];
  unsigned long long *keys = reinterpret_cast<unsigned long long *>(gsm);
  int *cache = reinterpret_cast<int *>(keys + P);
  int *flag = cache + B;
  const int tid = threadIdx.x;
  for (int j = tid; j < B; j += 1024) cache[j] = j;
  __syncthreads();
  for (int t = 1; t <= M; ++t) {
    const float *a = alpha + (size_t)(t - 1) * T;
    // (score key, inverted cache index): descending order = higher score first, then lower position
    for (int j = tid; j < P; j += 1024)
      keys[j] = j < B ? ((unsigned long long)score_key(a[cache[j]]) << 32) | (unsigned)(0xffffffffu - (unsigned)j) : 0ull;
    __syncthreads();
    for (int k = 2; k <= P; k <<= 1)
      for (int s = k >> 1; s > 0; s >>= 1) {
        for (int j = tid; j < P; j += 1024) {
          const int p = j ^ s;
          if (p > j) {
            const unsigned long long x = keys[j], y = keys[p];
            const bool desc = (j & k) == 0;
            if (desc ? x < y : x > y) { keys[j] = y; keys[p] = x; }
          }
        }
        __syncthreads();
      }
    for (int j = tid; j < B; j += 1024) flag[j] = 0;
    __syncthreads();
    for (int j = tid; j < B - L; j += 1024) flag[0xffffffffu - (unsigned)(keys[j] & 0xffffffffull)] = 1;
    __syncthreads();
    // Survivors in position order: thread owns a run of consecutive cache entries.
    const int per = (B + 1023) / 1024, j0 = tid * per, j1 = min(B, j0 + per);
    int cnt = 0;
    for (int j = j0; j < j1; ++j) cnt += flag[j];
    int tot;
    int off = block_excl_scan(cnt, s_scan, tot);
    int32_t *out = kept + (size_t)(t - 1) * (B - L);
    int mine[8];   // per <= 8 for B <= 8192
    int nm = 0;
    for (int j = j0; j < j1; ++j)
      if (flag[j]) mine[nm++] = cache[j];
    __syncthreads();   // every thread has read its cache entries
    for (int u = 0; u < nm; ++u) { cache[off + u] = mine[u]; out[off + u] = mine[u]; }
    for (int j = tid; j < L; j += 1024) cache[B - L + j] = B + (t - 1) * L + j;   // leave the recent window next
    __syncthreads();
  }
}

}  // namespace fkv
