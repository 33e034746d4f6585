// Kernel 2: per-segment top-k selection (Section 3.1, deterministic Top-K
// action): among slots [0, n - r) keep the k pairs with the highest scores,
// ties going to the lower slot; then the r most recent slots.  The kept slots
// are written in ascending order, which is the order compaction needs.
//
// Integer work on 4 bytes per pair, read from L2 right after the scorer wrote
// them.  One CTA per segment (a cluster of two for 32769 .. 65536 competing pairs): a histogram select finds the k-th largest key T
// and how many pairs equal to T are still needed; one ordered pass then emits
// {key > T} plus the first `need` slots with key == T, using block prefix
// sums - no atomics decide which tied pair stays.
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

constexpr int kSelThreads = 1024;   // the large variant: 1024 threads x 32 keys = one round of 32768
constexpr int kSelSmallThreads = 512, kSelSmallPerThread = 16;   // segments of <= 8192 competing pairs: two CTAs per SM
constexpr int kSelTinyThreads = 256, kSelTinyPerThread = 8;      // <= 2048 (budgets of 1K - 2K at large batch): many CTAs per SM

// Fresh page ids of one compacted segment: copied from the batch the planner
// reserved at the top of the free stack into the segment's row of pt_new.
__device__ __forceinline__ void fill_pt_new(const Ctx &c, int seg, const SegPlan &p) {
  if (!p.active) return;
  const int top0 = c.planhdr[PH_PUSH_START] + c.planhdr[PH_NEW_PAGES];  // stack top before the planner took them
  const int cnt = (p.n_new + kPage - 1) / kPage;
  int *dst = c.pt_new + (size_t)seg * c.max_pages;
  for (int j = threadIdx.x; j < cnt; j += blockDim.x) dst[j] = c.free_stack[top0 - 1 - (p.pad0 + j)];
}

// grid = segments of the call: pt_new rows when no selection kernel runs (fkv_compact).
__global__ void k_fill_pt_new(Ctx c, int seg0, int nseg) {
  if ((int)blockIdx.x < nseg) fill_pt_new(c, seg0 + blockIdx.x, c.plan[seg0 + blockIdx.x]);
}

// scores/idx: row (seg - seg_base) * cap.  kept_count (optional): [seg - seg_base].
//
// Every thread owns 32 consecutive slots per round of 32768 (so one block
// prefix sum orders a whole round).  SINGLE = the segment fits one round: the
// keys are loaded once and stay in registers for every pass.  Otherwise each
// pass streams the rounds again from L2, 8 loads in flight per thread.
//
// Selection of the k-th largest key T: a min/max pass fixes the key window;
// each histogram pass splits the current window into up to 2048 equal bins
// (so the bins follow the data, not fixed bit fields, and shared-memory
// atomics spread out), picks the bin where the count from the top crosses k,
// and narrows the window to it - at most three passes for 32-bit keys.
//
// MODE 1 is the first half of the sampled eviction action (Section 3.1, second equation; Appendix
// B.2): the same search run for the m - 2E best pairs (E = pairs to evict) tells which 2E pairs
// are the CANDIDATES (the lowest scores).  Instead of a slot list it writes a keep-priority per
// slot: +infinity for a pair outside the candidate set, score - g_j for the candidate of rank j in
// slot order, g_j the caller's standard Gumbel draw.  Keeping the best m - E priorities (a MODE 0
// pass over them) then evicts exactly the E candidates with the largest -score + g: E draws
// without replacement from softmax(-score) over the candidates.  prio may be the scores array.
constexpr int kSelRound = kSelThreads * 32;   // keys one CTA of the large variant holds in registers

// Score back from its ordering key (canonical: -0 came in as +0, NaN as -infinity).
__device__ __forceinline__ float key_score(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// ---- the selection machinery shared by the kernels that keep "the k best keys, ties to the lower index" ----
// Shared-memory scratch of one CTA of THREADS threads.
template <int THREADS>
struct SelShared {
  unsigned hist[2 * THREADS];
  int scan[33];
  unsigned red[64];
  unsigned bin, krem;
  unsigned long long wsum[33];
  unsigned long long xch[2];   // what a CTA pair tells each other: (min, max) of the keys; the first CTA's totals
};

// How the CTAs that share one segment's selection combine what each of them knows.  One CTA on its own: nothing to do.
struct SelAlone {
  template <int THREADS> __device__ __forceinline__ void minmax(SelShared<THREADS> &, uint32_t &, uint32_t &) const {}
  __device__ __forceinline__ void hist_ready() const {}
  template <int THREADS> __device__ __forceinline__ unsigned bin(const SelShared<THREADS> &sh, int b) const { return sh.hist[b]; }
  __device__ __forceinline__ void hist_read() const {}
};
// Two CTAs of one cluster, each with half of the segment's keys in registers: both see both halves' minimum and
// maximum and the sum of both histograms (read from the other CTA's shared memory), and so take the same decisions.
// Every thread of both CTAs makes every call (cluster barriers inside).
struct SelPair {
  uint32_t peer;   // the other CTA's rank in the cluster
  template <int THREADS> __device__ __forceinline__ void minmax(SelShared<THREADS> &sh, uint32_t &kmin, uint32_t &kmax) const {
    if (threadIdx.x == 0) sh.xch[0] = (unsigned long long)kmin | ((unsigned long long)kmax << 32);
    cluster_sync_all();
    const unsigned long long o = dsmem_ld_u64(dsmem_addr(smem_u32(&sh.xch[0]), peer));
    kmin = min(kmin, (uint32_t)(o & 0xffffffffu));
    kmax = max(kmax, (uint32_t)(o >> 32));
  }
  __device__ __forceinline__ void hist_ready() const { cluster_sync_all(); }   // both histograms are complete
  template <int THREADS> __device__ __forceinline__ unsigned bin(const SelShared<THREADS> &sh, int b) const {
    return sh.hist[b] + dsmem_ld_u32(dsmem_addr(smem_u32(&sh.hist[b]), peer));
  }
  __device__ __forceinline__ void hist_read() const { cluster_sync_all(); }    // ... and may be cleared again
};

// The k-th largest key T of the keys the CTA holds (0 < k < their number) and how many keys EQUAL to T
// are still to be kept once every key above T is.  Each thread holds up to PER keys of a round in
// key[0 .. nv); with several rounds, reload(round) brings a round's keys back (key and nv change).
// A min/max pass fixes the key window; each histogram pass splits the current window into up to
// 2 x THREADS equal bins (the bins follow the data, not fixed bit fields, so shared-memory atomics
// spread out), picks the bin where the count from the top crosses k and narrows the window to it -
// at most three passes for 32-bit keys.
template <int THREADS, int PER, class Reload, class Exch>
__device__ __forceinline__ void sel_kth_key(SelShared<THREADS> &sh, uint32_t (&key)[PER], int &nv, int rounds,
                                            Reload reload, const Exch &exch, unsigned k, uint32_t &T, unsigned &need) {
  constexpr int kBins = 2 * THREADS, NWARPS = THREADS / 32;
  constexpr int kLogBins = THREADS == 1024 ? 11 : THREADS == 512 ? 10 : 9;
  static_assert(THREADS == 1024 || THREADS == 512 || THREADS == 256, "bins = 2 x threads, a power of two");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t kmin = 0xffffffffu, kmax = 0u;
  for (int round = 0; round < rounds; ++round) {
    if (rounds > 1) reload(round);
#pragma unroll
    for (int j = 0; j < PER; ++j)
      if (j < nv) { kmin = min(kmin, key[j]); kmax = max(kmax, key[j]); }
  }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if (lane == 0) { sh.red[warp] = kmin; sh.red[32 + warp] = kmax; }
  __syncthreads();
  kmin = __reduce_min_sync(0xffffffffu, lane < NWARPS ? sh.red[lane] : 0xffffffffu);
  kmax = __reduce_max_sync(0xffffffffu, lane < NWARPS ? sh.red[32 + lane] : 0u);
  exch.minmax(sh, kmin, kmax);
  T = kmin;
  need = k;
  if (kmin == kmax) return;
  uint32_t lo = kmin, wmax = kmax - kmin;  // window: keys with key - lo <= wmax
  unsigned krem = k;
  int bits = 32 - __clz(wmax);
  for (;;) {
    const int shift = bits > kLogBins ? bits - kLogBins : 0;
    for (int b = tid; b < kBins; b += THREADS) sh.hist[b] = 0;
    __syncthreads();
    for (int round = 0; round < rounds; ++round) {
      if (rounds > 1) reload(round);
#pragma unroll
      for (int j = 0; j < PER; ++j) {
        const uint32_t d = key[j] - lo;
        if (j < nv && key[j] >= lo && d <= wmax) atomicAdd(&sh.hist[d >> shift], 1u);
      }
    }
    __syncthreads();
    exch.hist_ready();
    // Bins in descending order, two per thread: the top one is 2 THREADS - 1 - 2 tid.
    {
      const unsigned v0 = exch.bin(sh, kBins - 1 - 2 * tid), v1 = exch.bin(sh, kBins - 2 - 2 * tid);
      int tot;
      const unsigned above = (unsigned)block_excl_scan((int)(v0 + v1), sh.scan, tot);
      if (above < krem && krem <= above + v0) {
        sh.bin = kBins - 1 - 2 * tid; sh.krem = krem - above;
      } else if (above + v0 < krem && krem <= above + v0 + v1) {
        sh.bin = kBins - 2 - 2 * tid; sh.krem = krem - above - v0;
      }
    }
    __syncthreads();
    exch.hist_read();
    lo += sh.bin << shift;
    krem = sh.krem;
    __syncthreads();
    if (shift == 0) break;
    wmax = (1u << shift) - 1u;
    bits = shift;
  }
  T = lo;
  need = krem;  // keys equal to T still to keep, lowest index first
}

// How many keys above T (low word) and equal to T (high word) the threads BEFORE this one hold among the
// keys currently loaded, by one block prefix sum; total = the CTA's counts.  With these, thread order =
// index order decides which of the tied keys stay: no atomics do.
template <int THREADS, int PER>
__device__ __forceinline__ unsigned long long sel_counts_before(SelShared<THREADS> &sh, const uint32_t (&key)[PER], int nv,
                                                                uint32_t T, unsigned long long &total) {
  constexpr int NWARPS = THREADS / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned cgt = 0, ceq = 0;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    cgt += (j < nv && key[j] > T);
    ceq += (j < nv && key[j] == T);
  }
  unsigned long long v = (unsigned long long)cgt | ((unsigned long long)ceq << 32), inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();   // the scratch may still be read from the call before
  if (lane == 31) sh.wsum[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    unsigned long long w = lane < NWARPS ? sh.wsum[lane] : 0ull, winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      unsigned long long t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    sh.wsum[lane] = winc - w;
    if (lane == 31) sh.wsum[32] = winc;
  }
  __syncthreads();
  total = sh.wsum[32];
  return sh.wsum[warp] + inc - v;
}

// Place of a key in the kept list given the counts (above T, equal to T) of the keys before it: every key above
// T is kept, of those equal to T the first `need`; -1 if the key is not kept.
__device__ __forceinline__ int sel_place(bool greater, bool equal, unsigned bgt, unsigned beq, unsigned need) {
  if (greater) return (int)(bgt + min(beq, need));
  if (equal && beq < need) return (int)(bgt + beq);
  return -1;
}

// PAIR: two CTAs (one cluster, consecutive block indices) share a segment of up to 2 x THREADS x PER competing pairs:
// each holds one half of the keys in registers for every pass, the histograms are summed across the pair through
// distributed shared memory, and the second CTA's places start after the first one's counts.
template <bool SINGLE, int MODE, int THREADS, int PER, bool PAIR = false>
__global__ void __launch_bounds__(THREADS) k_select(Ctx c, const float *scores, int32_t *idx, int32_t *kept_count,
                                                         int seg_base, int fill_pages, float *prio,
                                                         const float *noise, int noise_stride, int noise_base) {
  constexpr int kSelPerThread = PER, kSelRound = THREADS * PER;
  __shared__ SelShared<THREADS> sh;
  static_assert(!PAIR || SINGLE, "a CTA of a pair keeps its half in registers");
  const int witem = PAIR ? blockIdx.x >> 1 : blockIdx.x, half = PAIR ? blockIdx.x & 1 : 0;
  if (witem >= c.planhdr[PH_NWORK]) return;   // (both CTAs of a pair)
  const int seg = c.work[witem];
  const SegPlan p = c.plan[seg];
  const int tid = threadIdx.x;
  if (fill_pages && half == 0) fill_pt_new(c, seg, p);
  const int m = p.n_old - p.r;
  const int k = MODE == 0 ? p.k_sel : max(0, m - 2 * (p.n_old - p.n_new));   // MODE 1: the non-candidates
  const float *sc = scores + (size_t)(seg - seg_base) * c.cap;
  int32_t *out = MODE == 0 ? idx + (size_t)(seg - seg_base) * c.cap : nullptr;
  float *pr = MODE == 1 ? prio + (size_t)(seg - seg_base) * c.cap : nullptr;
  const float *nz = MODE == 1 ? noise + (size_t)(seg - noise_base) * noise_stride : nullptr;
  // The cases that need no search (the first CTA of a pair writes them; both leave).
  if (MODE == 0) {
    if (kept_count && tid == 0 && half == 0) kept_count[seg - seg_base] = p.n_new;
    // The protected recent slots close the list.
    if (half == 0)
      for (int j = tid; j < p.r; j += THREADS) out[k + j] = m + j;
    if (k <= 0) return;
    if (k >= m) {
      if (half == 0)
        for (int j = tid; j < m; j += THREADS) out[j] = j;
      return;
    }
  } else {
    if (k <= 0) {   // every competing pair is a candidate: rank = slot
      if (half == 0)
        for (int j = tid; j < m; j += THREADS) pr[j] = key_score(score_key(sc[j])) - nz[j];
      return;
    }
    if (k >= m) {   // nothing to evict
      if (half == 0)
        for (int j = tid; j < m; j += THREADS) pr[j] = INFINITY;
      return;
    }
  }
  const int rounds = SINGLE ? 1 : (m + kSelRound - 1) / kSelRound;
  uint32_t key[kSelPerThread];
  int nv = 0;  // valid keys of this thread in the loaded round (they are its first nv)
  auto load_round = [&](int round) {
    const int base = round * kSelRound + tid * kSelPerThread;
    nv = min(max(m - base, 0), kSelPerThread);
    const float4 *src = reinterpret_cast<const float4 *>(sc + base);
    float4 x[kSelPerThread / 4];
#pragma unroll
    for (int q = 0; q < kSelPerThread / 4; ++q) x[q] = q * 4 < nv ? src[q] : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int q = 0; q < kSelPerThread / 4; ++q) {
      key[4 * q] = score_key(x[q].x); key[4 * q + 1] = score_key(x[q].y);
      key[4 * q + 2] = score_key(x[q].z); key[4 * q + 3] = score_key(x[q].w);
    }
  };
  if (SINGLE) load_round(half);   // (a CTA of a pair: its half of the keys)

  uint32_t T;
  unsigned need;
  if (PAIR) sel_kth_key<THREADS, PER>(sh, key, nv, rounds, load_round, SelPair{(uint32_t)(half ^ 1)}, (unsigned)k, T, need);
  else sel_kth_key<THREADS, PER>(sh, key, nv, rounds, load_round, SelAlone{}, (unsigned)k, T, need);

  // ---- ordered emit: one block prefix sum per round ----
  unsigned run_gt = 0, run_eq = 0;
  for (int round = 0; round < rounds; ++round) {
    if (!SINGLE) load_round(round);
    unsigned long long tot;
    const unsigned long long excl = sel_counts_before<THREADS, PER>(sh, key, nv, T, tot);
    if (PAIR) {   // the second CTA's places start after the first one's counts
      if (half == 0 && tid == 0) sh.xch[1] = tot;
      cluster_sync_all();
      if (half == 1) {
        const unsigned long long first = dsmem_ld_u64(dsmem_addr(smem_u32(&sh.xch[1]), 0));
        run_gt = (unsigned)(first & 0xffffffffu); run_eq = (unsigned)(first >> 32);
      }
      cluster_sync_all();   // the first CTA's shared memory has been read: it may leave
    }
    unsigned bgt = run_gt + (unsigned)(excl & 0xffffffffu), beq = run_eq + (unsigned)(excl >> 32);
    const int slot0 = (PAIR ? half : round) * kSelRound + tid * kSelPerThread;
#pragma unroll
    for (int j = 0; j < kSelPerThread; ++j) {
      const bool g = j < nv && key[j] > T, e = j < nv && key[j] == T;
      const int dst = sel_place(g, e, bgt, beq, need);
      if (MODE == 0) {
        if (dst >= 0) out[dst] = slot0 + j;
      } else if (j < nv) {
        const bool kept = dst >= 0;
        const int rank = slot0 + j - (int)(bgt + min(beq, need));   // candidates before this slot
        pr[slot0 + j] = kept ? INFINITY : key_score(key[j]) - nz[rank];
      }
      bgt += g; beq += e;
    }
    run_gt += (unsigned)(tot & 0xffffffffu);
    run_eq += (unsigned)(tot >> 32);
  }
}

}  // namespace fkv
