// Kernel 6: the attention features a_n of Appendix B.1, refreshed when an eviction closes a chunk.
//
// Per query head: recent-window attention for windows 8, 16, 32 and the update length, the sum of
// the chunk scores over chunks, and the same sum decayed by 0.9 per chunk.  Reading taken: a
// window feature is the MEAN over the last w decode queries of the softmax probability the head
// gave to the pair (0 for queries older than the pair); the chunk score is the window = update
// length feature; both cumulative features are updated before the scorer reads them.
//
// Nothing is accumulated during decoding.  Each decode launch that appends a token records its
// queries and, per query head, log2 of the softmax denominator (max included) and the number of
// pairs it saw.  Here the probabilities are RECOMPUTED for the whole chunk at once,
//     p[t][i] = 2^(scale <q_t, k_i> - M'_t),
// a dense contraction [128 pairs x D] . [D x queries] per tile and query head - the one step of
// this library that is compute-shaped, so it runs on the 5th-generation tensor cores, as a
// warp-specialised pipeline in one persistent CTA per SM (a contiguous range of 128-pair tiles):
//   - warps 2-3 copy the K rows of a tile into a ring of A stages, 16-byte asynchronous copies that
//     move the chunks verbatim (the page record's swizzle is the shared-memory swizzle);
//   - warp 0 copies a query head's record, which the decode launches wrote as a ready K-major
//     operand tile (row = ring slot), with one bulk copy per 64 channels into a ring of B stages,
//     and the head's softmax statistics into a small ring of their own.  When the records of all
//     g heads fit, they stay in shared memory for all tiles of a segment;
//   - warp 1 multiplies: one lane issues tcgen05.mma (kind::f16, bf16 x bf16 -> fp32, M = 128,
//     N = the padded query count, K = 16 per instruction) into one of four (two for more than 128
//     queries) accumulators in tensor memory; tcgen05.commit hands the accumulator to a reducing warpgroup and the stages back to
//     warp 0;
//   - three warpgroups (warps 4-15) reduce, taking the units of the four accumulators in turn (with
//     two accumulators there are four warpgroups, two share an accumulator and split the query
//     axis): a thread owns ONE pair (its tensor-memory
//     lane) and walks the query axis from the newest query back, 32 columns per tcgen05.ld: exp2,
//     add; the windows 8 / 16 / 32 are prefixes of that walk.  The six features of the head go
//     straight to the pair's meta row.
// While a head is reduced, the next one is multiplied and the one after copied.  Every wait is
// bounded; a role that gives up sets the status word and every role then drains to the common exit,
// where tensor memory is freed.
// The decode path pays 2 g D + 4 g bytes per token for the record instead of a read-modify-write
// of every pair's feature row per token.
#pragma once
#include "fkv_dev.cuh"
#include "fkv_score.cuh"

namespace fkv {

constexpr float kFeatDecay = 0.9f;   // Appendix B.1: per-chunk decay of the decayed sum
constexpr int kFeatPages = 8;        // pages (of 16 pairs) per tile: the M = 128 rows of the mma
constexpr int kFeatMaxQueries = 256; // N of one mma; two accumulators of that width fill tensor memory
// warp 0: records, warp 1: mma, warps 2-3: K rows (warp 2 owns tensor memory), then WGS reducing warpgroups: four when
// two of them share each of two accumulators (more than 128 queries), else three, which take the units of the four
// accumulators in turn - 512 threads leave each 128 registers, and the reductions then need no spills.
__host__ __device__ constexpr int feat_threads(int wgs) { return (4 + 4 * wgs) * 32; }
constexpr int kFeatMaxA = 4, kFeatMaxQ = 8, kFeatMaxS = 24;   // ring depths the barrier block has room for

struct FeatSmem {
  static constexpr size_t kBudget = 227 * 1024, kBars = 512, kPart = 2 * 128 * 16;   // barriers; the older halves' sums
  static __host__ __device__ int lq(int W) { return (W + 15) & ~15; }                        // rows of a query tile
  static __host__ __device__ size_t a_bytes(int D) { return (size_t)(D / 64) * 128 * 128; }   // [D/64][128 rows][128 B]
  static __host__ __device__ size_t q_bytes(int D, int W) { return (size_t)(D / 64) * lq(W) * 128; }
  // Statistics slots.  No barrier says that a slot may be overwritten; the depth does: a head's record is copied only
  // after an mma that used the record before it has completed, and that mma was issued only after every reduction
  // more than four units (the accumulators) back.  Resident records: a slot is reused after so many segments that
  // at least four units lie in between; streamed records: the B ring's depth + 4.
  static __host__ __device__ int stat_segs(int G) { return 2 + (3 + G) / G; }
  static __host__ __device__ int stat_slots(int G, int nq) { return nq == G ? stat_segs(G) * G : nq + 4; }
  // Ring depths: all g heads' records resident if that leaves two A stages, else two B stages streamed per tile.
  static __host__ void rings(int D, int G, int W, int &na, int &nq) {
    const size_t a = a_bytes(D), q = q_bytes(D, W), st = (size_t)lq(W) * 4;
    const size_t room = kBudget - 1024 - kBars - kPart;
    nq = (G * q + stat_segs(G) * G * st + 2 * a <= room) ? G : 2;
    const size_t left = room - nq * q - stat_slots(G, nq) * st;
    na = (int)(left / a);
    if (na > kFeatMaxA) na = kFeatMaxA;
  }
  // 1 KB alignment slack | A ring | B ring | statistics | barriers and the tensor-memory address.  Never less than
  // 120 KB: one CTA per SM, so the tensor-memory allocation never has to wait for another CTA.
  static __host__ __device__ size_t bytes(int D, int G, int W, int na, int nq) {
    const size_t need = 1024 + na * a_bytes(D) + nq * q_bytes(D, W) + (size_t)stat_slots(G, nq) * lq(W) * 4 + kPart + kBars;
    return need > 120 * 1024 ? need : 120 * 1024;
  }
};

// 2^x for x <= 0 (tiny results may flush to zero).
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- tcgen05 wrappers (5th-generation tensor cores, tensor memory) ----
// Shared-memory matrix descriptor of a K-major tile with 128-byte rows and the 128-byte swizzle:
// start address, stride between 8-row groups = 1024 bytes, descriptor version 1, layout 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3ffffu) >> 4) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, N and M of the instruction.
__device__ __forceinline__ uint32_t umma_idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {   // one full warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {    // the same warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same, with a word on the A operand's collector buffer: FILL keeps the A slice that this mma fetches, USE_LAST
// multiplies the kept slice again (another B, another accumulator) and lets it go - the slice is read from shared
// memory once for the two.
template <bool FILL>
__device__ __forceinline__ void umma_bf16_keep_a(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  if (FILL)
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16.collector::a::fill [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  else
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16.collector::a::lastuse [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {   // the barrier gets one arrival when the issued mmas are done
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// 32 consecutive fp32 columns of this thread's tensor-memory lane: the load is asynchronous, the registers hold
// the values only after tmem_ld_wait on the same array (which names them as operands, so that no use of them can
// be scheduled before it).
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}

// Bounded wait that polls with test_wait (returns at once) instead of try_wait (may suspend the thread for a
// hardware time slice): the roles of this kernel hand over every few hundred cycles.
__device__ __forceinline__ bool mbar_spin(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < (1u << 26); ++i) {
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}
// A whole warp waits on a phase parity, but only lane 0 polls the barrier word (sixteen reducing warps that all spin
// with 32 lanes each keep the shared-memory pipe busy for nothing); the others learn the outcome from a shuffle.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity) {
  bool ok = true;
  if ((threadIdx.x & 31) == 0) ok = mbar_spin(bar, parity);
  return __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
}

// The walk of one role over the CTA's tiles: which work item a tile is in and what that item's query record holds.
struct FeatWalk {
  int wi, tbeg, tend, seg, n, ls, head, cnt, Lc, Lq, oldest_seen, newest;
  bool ordered;   // ring not wrapped, whole 32-query chunks, and every query saw exactly one pair more than the one before
  float inv_Lc;
};
// A ring position and the phase bit of its barriers.  Kept by counting: the special-function pipe that an integer
// division needs is the one the reductions keep busy.
struct FeatRing {
  int i, ph;
  __device__ __forceinline__ void next(int n) { if (++i == n) { i = 0; ph ^= 1; } }
};
struct FeatTile {
  int pg0, np;
  bool fast, masked, first, last;
};
// Tile t of the flat tile list; false if its segment has no query on record (its stored features stand).
__device__ __forceinline__ bool feat_tile(const Ctx &c, int t, int t0, int t1, FeatWalk &w, FeatTile &x) {
  if (t >= w.tend) {
    while (t >= c.tile1_start[w.wi + 1]) ++w.wi;
    w.tbeg = c.tile1_start[w.wi]; w.tend = c.tile1_start[w.wi + 1];
    w.seg = c.work[w.wi];
    w.n = c.plan[w.seg].n_old;
    w.ls = w.seg / c.Hkv; w.head = w.seg % c.Hkv;
    w.cnt = c.hist_cnt[w.ls];
    w.Lc = min(w.cnt, c.hist_w);            // queries of the chunk that are on record
    w.Lq = (w.Lc + 15) & ~15;               // N of the mma
    w.oldest_seen = w.Lc ? c.hist_n[(size_t)w.ls * c.hist_w + (w.cnt - w.Lc) % c.hist_w] : 0;
    w.newest = w.Lc ? (w.cnt - 1) % c.hist_w : 0;   // ring slot of the most recent query
    w.inv_Lc = w.Lc ? 1.f / (float)w.Lc : 0.f;
    w.ordered = w.Lc > 0 && w.cnt <= c.hist_w && (w.Lc & 31) == 0 &&
                c.hist_n[(size_t)w.ls * c.hist_w + w.newest] - w.oldest_seen == w.Lc - 1;
  }
  if (w.Lc == 0) return false;
  x.pg0 = (t - w.tbeg) * kFeatPages;
  x.np = min(kFeatPages, (w.n + kPage - 1) / kPage - x.pg0);
  // No masks needed: every recorded query saw the whole tile (the oldest one saw the fewest pairs), the ring has
  // not wrapped (slot order = time order) and the record is whole 32-column chunks.
  x.fast = x.pg0 * kPage + kFeatPages * kPage <= w.oldest_seen && w.cnt <= c.hist_w && (w.Lc & 31) == 0;
  // Pairs appended during the chunk, but slot order = time order and query t saw the pairs below oldest_seen + t:
  // a pair counts from one column on, a threshold per thread.
  x.masked = !x.fast && w.ordered;
  x.first = t == w.tbeg || t == t0;         // first / last tile of its segment in this CTA's range
  x.last = t + 1 == w.tend || t + 1 == t1;
  return true;
}

// 32 columns [a0, a0 + 32) of one pair's row, newest first, every query valid: exp2 and add.
template <bool NEWEST>
__device__ __forceinline__ void feat_chunk(const uint32_t (&r)[32], const float *mp, float scale_log2, float &run,
                                           float &w8, float &w16) {
#pragma unroll
  for (int i = 28; i >= 0; i -= 4) {
    const float4 M4 = *reinterpret_cast<const float4 *>(mp + i);
    run += (ex2(fmaf(__uint_as_float(r[i + 3]), scale_log2, -M4.w)) + ex2(fmaf(__uint_as_float(r[i + 2]), scale_log2, -M4.z))) +
           (ex2(fmaf(__uint_as_float(r[i + 1]), scale_log2, -M4.y)) + ex2(fmaf(__uint_as_float(r[i]), scale_log2, -M4.x)));
    if (NEWEST && i == 24) w8 = run;
    if (NEWEST && i == 16) w16 = run;
  }
}

// The same for a pair that the queries before column `first` (relative to the chunk) did not see yet.
template <bool NEWEST>
__device__ __forceinline__ void feat_chunk_from(const uint32_t (&r)[32], const float *mp, float scale_log2, int first,
                                                float &run, float &w8, float &w16) {
#pragma unroll
  for (int i = 28; i >= 0; i -= 4) {
    const float4 M4 = *reinterpret_cast<const float4 *>(mp + i);
    const float p3 = i + 3 >= first ? ex2(fmaf(__uint_as_float(r[i + 3]), scale_log2, -M4.w)) : 0.f;
    const float p2 = i + 2 >= first ? ex2(fmaf(__uint_as_float(r[i + 2]), scale_log2, -M4.z)) : 0.f;
    const float p1 = i + 1 >= first ? ex2(fmaf(__uint_as_float(r[i + 1]), scale_log2, -M4.y)) : 0.f;
    const float p0 = i >= first ? ex2(fmaf(__uint_as_float(r[i]), scale_log2, -M4.x)) : 0.f;
    run += (p3 + p2) + (p1 + p0);
    if (NEWEST && i == 24) w8 = run;
    if (NEWEST && i == 16) w16 = run;
  }
}

template <int D, int WGS>
__global__ void __launch_bounds__(feat_threads(WGS), 1) k_features(Ctx c, float scale_log2, int NA, int NQ) {
  constexpr int HALVES = D / 64, ROWS = kFeatPages * kPage;   // 128 pairs
  extern __shared__ uint8_t smem_raw[];
  const int total = c.planhdr[PH_TILES1], nwork = c.planhdr[PH_NWORK];
  const int per = (total + (int)gridDim.x - 1) / (int)gridDim.x;
  const int t0 = blockIdx.x * per, t1 = min(t0 + per, total);
  if (t0 >= t1) return;                  // nothing allocated yet
  const int W = c.hist_w, Lw = c.hist_wp, G = c.G, Hq = c.Hkv * G;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const size_t abytes = FeatSmem::a_bytes(D), qbytes = (size_t)HALVES * Lw * 128;
  uint8_t *At = smem;                                    // [NA][HALVES][128][128 B]
  uint8_t *Qt = At + (size_t)NA * abytes;                // [NQ][HALVES][Lw][128 B]
  const bool resident = NQ == G;   // the g heads' records stay in their stages for all tiles of a segment
  const int NS = FeatSmem::stat_slots(G, NQ), SD = FeatSmem::stat_segs(G);
  float *St = reinterpret_cast<float *>(Qt + (size_t)NQ * qbytes);   // [NS][Lw]: log2 denominators of a head's queries
  float *Part = St + (size_t)NS * Lw;   // [2][128] x (sum, w8, w16, w32): the older half's sums when two warpgroups share an accumulator
  uint64_t *bars = reinterpret_cast<uint64_t *>(Part + 2 * ROWS * 4);
  uint64_t *a_full = bars, *a_empty = a_full + kFeatMaxA, *q_full = a_empty + kFeatMaxA, *q_empty = q_full + kFeatMaxQ;
  uint64_t *acc_full = q_empty + kFeatMaxQ, *acc_empty = acc_full + 4, *part_full = acc_empty + 4, *s_full = part_full + 2;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(s_full + kFeatMaxS);

  // Tensor memory: NB accumulators (four if they fit, so that the multiplies run ahead of the reductions), each a
  // power of two >= 32 columns with one fp32 column per query.
  uint32_t ncols = 32;
  while ((int)ncols < Lw) ncols <<= 1;
  const int NB = ncols <= 128 ? 4 : 2, lgNB = ncols <= 128 ? 2 : 1;
  if (warp == 2) tmem_alloc(smem_u32(tmem_slot), NB * ncols);
  if (threadIdx.x == 0) {
    for (int s = 0; s < NA; ++s) { mbar_init(smem_u32(&a_full[s]), 64); mbar_init(smem_u32(&a_empty[s]), 1); }
    for (int s = 0; s < NS; ++s) mbar_init(smem_u32(&s_full[s]), 1);
    for (int s = 0; s < NQ; ++s) { mbar_init(smem_u32(&q_full[s]), 1); mbar_init(smem_u32(&q_empty[s]), 1); }
    for (int b = 0; b < NB; ++b) { mbar_init(smem_u32(&acc_full[b]), 1); mbar_init(smem_u32(&acc_empty[b]), NB == 2 ? 8 : 4); }
    for (int b = 0; b < 2; ++b) mbar_init(smem_u32(&part_full[b]), 128);
    fence_barrier_init();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  FeatWalk w;
  w.wi = find_work(c.tile1_start, nwork, t0);
  w.tend = -1;
  FeatTile x;

  if (warp == 0) {
    // ---------------- copies the query records and their statistics ----------------
    int segs = -1;
    FeatRing sseg{SD - 1, 1}, qr{0, 0}, sr{0, 0};   // resident: segment slot of the statistics; streamed: B and statistics rings
    bool ok = true;
    for (int t = t0; t < t1 && ok; ++t) {
      if (!feat_tile(c, t, t0, t1, w, x)) continue;
      if (x.first) { ++segs; sseg.next(SD); }
      if (!resident || x.first) {
        for (int j = 0; j < G; ++j) {
          const int sq = resident ? j : qr.i, pq = resident ? segs & 1 : qr.ph;
          const int ss = resident ? sseg.i * G + j : sr.i;
          if (!resident) { qr.next(NQ); sr.next(NS); }
          const size_t qhead = (size_t)w.ls * Hq + w.head * G + j;
          if (!mbar_wait_warp(smem_u32(&q_empty[sq]), pq ^ 1)) { set_status(c, kDevWaitTimeout); ok = false; break; }
          if (lane == 0) {
            mbar_arrive_expect_tx(smem_u32(&q_full[sq]), (uint32_t)(HALVES * w.Lq * 128));
            mbar_arrive_expect_tx(smem_u32(&s_full[ss]), (uint32_t)(w.Lq * 4));
          }
          __syncwarp();
          if (lane < HALVES)
            bulk_g2s(smem_u32(Qt + (size_t)sq * qbytes + (size_t)lane * Lw * 128),
                     c.hist_q + hist_q_off(qhead, lane * 8, 0, Lw, D), (uint32_t)(w.Lq * 128), smem_u32(&q_full[sq]));
          else if (lane == HALVES)
            bulk_g2s(smem_u32(St + (size_t)ss * Lw), c.hist_mp + qhead * Lw, (uint32_t)(w.Lq * 4), smem_u32(&s_full[ss]));
        }
      }
    }
  } else if (warp == 2 || warp == 3) {
    // ---------------- copy the K rows: thread = one 16-byte chunk column of rows R0, R0 + 4, ... ----------------
    constexpr int NCH = D / 8, RSTEP = 64 / NCH;
    const int p = threadIdx.x - 64, ch = p % NCH, R0 = p / NCH;
    const uint32_t dcol = (uint32_t)((ch >> 3) * ROWS * 128 + (ch & 7) * 16);
    FeatRing ar{0, 0};
    for (int t = t0; t < t1; ++t) {
      if (!feat_tile(c, t, t0, t1, w, x)) continue;
      const int sa = ar.i, pa = ar.ph;
      const int *ptrow = c.pt + (size_t)w.seg * c.max_pages + x.pg0;
      int pid[kFeatPages];
#pragma unroll
      for (int pg = 0; pg < kFeatPages; ++pg) pid[pg] = ptrow[min(pg, x.np - 1)];   // one round trip, under the wait
      if (!mbar_wait_warp(smem_u32(&a_empty[sa]), pa ^ 1)) { set_status(c, kDevWaitTimeout); break; }
      const uint32_t dst0 = smem_u32(At + (size_t)sa * abytes) + dcol;
#pragma unroll
      for (int pg = 0; pg < kFeatPages; ++pg) {
        if (pg < x.np) {
          const uint8_t *page = c.pool + (size_t)pid[pg] * c.page_bytes + ch * 16;
#pragma unroll
          for (int k = 0; k < kPage / RSTEP; ++k) {
            const int r = R0 + k * RSTEP;
            cp_async16(dst0 + (uint32_t)((pg * kPage + r) * 128), page + r * 4 * D);
          }
        }
      }
      cp_async_wait_all();       // this thread's chunks have landed ...
      fence_proxy_async();       // ... and are visible to the tensor core's reads of shared memory
      mbar_arrive(smem_u32(&a_full[sa]));
      ar.next(NA);
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- multiplies (one thread: it issues every mma and commit itself) ----------------
    int segs = -1, u = 0;
    FeatRing ar{0, 0}, qr{0, 0};
    bool ok = true;
    for (int t = t0; t < t1 && ok; ++t) {
      if (!feat_tile(c, t, t0, t1, w, x)) continue;
      const int sa = ar.i, pa = ar.ph;
      if (!mbar_spin(smem_u32(&a_full[sa]), pa)) { set_status(c, kDevWaitTimeout); break; }
      if (x.first) ++segs;
      const uint32_t idesc = umma_idesc_bf16(ROWS, w.Lq);
      const uint64_t ad0 = umma_desc_sw128(smem_u32(At + (size_t)sa * abytes));
      const uint32_t qhalf16 = (uint32_t)(Lw * 128) >> 4;   // a 64-channel half of a record's tile, in 16-byte units
      // Two heads at a time when two accumulators are to be had: their k-steps alternate, so that an mma never has
      // to wait for the one before it on the same accumulator.
      for (int j = 0; j < G && ok; j += 2) {
        const int nh = min(2, G - j);
        int sq[2] = {0, 0}, bb[2] = {0, 0};
        for (int h = 0; h < nh && ok; ++h) {
          const int pq = resident ? segs & 1 : qr.ph;
          sq[h] = resident ? j + h : qr.i;
          if (!resident) qr.next(NQ);
          if (!resident || x.first)
            if (!mbar_spin(smem_u32(&q_full[sq[h]]), pq)) { set_status(c, kDevWaitTimeout); ok = false; break; }
          bb[h] = (u + h) & (NB - 1);
          if (!mbar_spin(smem_u32(&acc_empty[bb[h]]), (((u + h) >> lgNB) & 1) ^ 1)) { set_status(c, kDevWaitTimeout); ok = false; }
        }
        if (!ok) break;
        tc_fence_after();
        {
          // This thread's instruction count is on the critical path (it shares its scheduler with four reducing
          // warps): descriptors are built once and advanced by adding to their address field (16-byte units).
          const uint64_t bd0 = umma_desc_sw128(smem_u32(Qt + (size_t)sq[0] * qbytes));
          const uint64_t bd1 = umma_desc_sw128(smem_u32(Qt + (size_t)sq[1] * qbytes));
          const uint32_t d0 = tmem_base + (uint32_t)bb[0] * ncols, d1 = tmem_base + (uint32_t)bb[1] * ncols;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {        // K = 16 channels per instruction: 32 bytes inside the swizzled row
            const uint64_t ad = ad0 + (uint64_t)(((ks >> 2) * ROWS * 128 + (ks & 3) * 32) >> 4);
            const uint64_t kb = (uint64_t)((ks >> 2) * qhalf16 + (ks & 3) * 2);
            if (nh == 2) {
              umma_bf16_keep_a<true>(d0, ad, bd0 + kb, idesc, ks > 0);
              umma_bf16_keep_a<false>(d1, ad, bd1 + kb, idesc, ks > 0);
            } else {
              umma_bf16(d0, ad, bd0 + kb, idesc, ks > 0);
            }
          }
          for (int h = 0; h < nh; ++h) {
            umma_commit(smem_u32(&acc_full[bb[h]]));                              // the accumulator is complete
            if (!resident || x.last) umma_commit(smem_u32(&q_empty[sq[h]]));      // the record's stage has been read
          }
          if (j + nh == G) umma_commit(smem_u32(&a_empty[sa]));                   // ... and so has the tile's
        }
        u += nh;
      }
      ar.next(NA);
    }
  } else if (warp == 1) {
    // the other lanes of the mma warp have nothing to do
  } else if (warp >= 4) {
    // ---------------- reduce: thread = one pair of the tile (its tensor-memory lane).  Four accumulators: warpgroup
    // e owns accumulator e.  Two (more than 128 queries): warpgroups e and e + 2 share accumulator e; the first walks
    // the newer half of the query axis and owns the result, the second the older half, whose sums it hands over
    // through shared memory.
    const int wg = (warp - 4) >> 2, e = wg & (NB - 1), half = wg >> lgNB, quarter = warp & 3;
    const bool shared_acc = NB == 2;
    const int R = quarter * 32 + lane;
    const uint32_t trow0 = tmem_base + ((uint32_t)(quarter * 32) << 16);
    int u = 0, u3 = 0;
    FeatRing sseg{SD - 1, 1}, sr{0, 0};
    bool ok = true;
    for (int t = t0; t < t1 && ok; ++t) {
      if (!feat_tile(c, t, t0, t1, w, x)) continue;
      if (x.first) sseg.next(SD);
      const int slot = x.pg0 * kPage + R;
      const bool live = half == 0 && slot < w.n;
      float *frow = nullptr;
      if (live)
        frow = reinterpret_cast<float *>(c.pool + (size_t)c.pt[(size_t)w.seg * c.max_pages + x.pg0 + R / kPage] * c.page_bytes +
                                         c.off_f) + (R % kPage) * (c.F + 1);
      // 32-column chunks, counted from the newest: this warpgroup's are [k0, k1)
      const int nch = ((w.Lq + 31) & ~31) >> 5, top = (nch - 1) << 5;   // (Lq = Lc on the two ordered paths)
      const int k0 = half == 0 ? 0 : (nch + 1) >> 1, k1 = (shared_acc && half == 0) ? (nch + 1) >> 1 : nch;
      for (int j = 0; j < G; ++j, ++u) {
        const int ss = resident ? sseg.i * G + j : sr.i, sp = resident ? sseg.ph : sr.ph;   // the head's statistics
        if (!resident) sr.next(NS);
        const int b = u & (NB - 1);
        if (WGS == 3) {   // three warpgroups: every third unit, whatever its accumulator
          const bool mine = u3 == wg;
          if (++u3 == 3) u3 = 0;
          if (!mine) continue;
        } else if (b != e) {
          continue;
        }
        // The cumulative features to update: asked for here, used after the walk.
        float old_sum = 0.f, old_dec = 0.f;
        if (live) { old_sum = __ldcg(frow + j * 6 + 4); old_dec = __ldcg(frow + j * 6 + 5); }
        const float *mp = St + (size_t)ss * Lw;
        const uint32_t ph = (uint32_t)(u >> lgNB) & 1;
        if (!mbar_wait_warp(smem_u32(&s_full[ss]), sp) || !mbar_wait_warp(smem_u32(&acc_full[b]), ph)) {
          set_status(c, kDevWaitTimeout); ok = false; break;
        }
        tc_fence_after();
        const uint32_t trow = trow0 + (uint32_t)b * ncols;
        float run = 0.f, w8 = 0.f, w16 = 0.f, w32 = 0.f;
        if (x.fast) {
          // Columns are in time order and all valid: walk from the newest chunk back.
          for (int k = k0; k < k1; ++k) {
            const int a0 = top - (k << 5);
            uint32_t v[32];
            tmem_ld32_issue(trow + (uint32_t)a0, v);
            tmem_ld_wait(v);
            if (k == 0) {
              feat_chunk<true>(v, mp + a0, scale_log2, run, w8, w16);
              w32 = run;
            } else {
              feat_chunk<false>(v, mp + a0, scale_log2, run, w8, w16);
            }
          }
        } else if (x.masked) {
          // Time order, but the pair is younger than some of the queries: it counts from column c0 on.  Chunks
          // older than the warp's first pair's threshold (the smallest of the warp) hold nothing for any lane.
          const int c0 = min(max(slot + 1 - w.oldest_seen, 0), w.Lc);
          const int c0_warp = __shfl_sync(0xffffffffu, c0, 0);
          for (int k = k0; k < k1; ++k) {
            const int a0 = top - (k << 5);
            if (a0 + 32 <= c0_warp) break;
            uint32_t v[32];
            tmem_ld32_issue(trow + (uint32_t)a0, v);
            tmem_ld_wait(v);
            if (k == 0) {
              feat_chunk_from<true>(v, mp + a0, scale_log2, c0 - a0, run, w8, w16);
              w32 = run;
            } else {
              feat_chunk_from<false>(v, mp + a0, scale_log2, c0 - a0, run, w8, w16);
            }
          }
        } else {
          // General case: a query counts for the pair if it is on record and saw it; its age decides the windows.
          const int *hn = c.hist_n + (size_t)w.ls * W;
          const int newest = w.newest;
          for (int k = k0; k < k1; ++k) {
            const int a0 = top - (k << 5);
            uint32_t v[32];
            tmem_ld32_issue(trow + (uint32_t)a0, v);
            tmem_ld_wait(v);
#pragma unroll
            for (int i = 31; i >= 0; --i) {
              const int col = a0 + i;
              const bool on = col < w.Lc;                 // a recorded query (beyond: padding of the tile)
              const int seen = on ? __ldg(hn + col) : 0;
              const float m = on ? mp[col] : 0.f;
              const int age = newest - col + (col > newest ? W : 0);
              const float p = slot < seen ? ex2(fmaf(__uint_as_float(v[i]), scale_log2, -m)) : 0.f;
              run += p;
              w8 += age < 8 ? p : 0.f;
              w16 += age < 16 ? p : 0.f;
              w32 += age < 32 ? p : 0.f;
            }
          }
        }
        tc_fence_before();
        if (shared_acc) {
          float4 *mine = reinterpret_cast<float4 *>(Part) + (size_t)b * ROWS + R;
          if (half == 1) {
            *mine = make_float4(run, w8, w16, w32);
            mbar_arrive(smem_u32(&part_full[b]));   // every thread: its own sums are written
          } else {
            if (!mbar_wait_warp(smem_u32(&part_full[b]), ph)) { set_status(c, kDevWaitTimeout); ok = false; break; }
            const float4 o = *mine;                 // read before this warpgroup lets the accumulator go: the next
            run += o.x; w8 += o.y; w16 += o.z; w32 += o.w;   // sums land here only after the next mma into it
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&acc_empty[b]));   // this warp's share of the accumulator has been read
        if (live) {
          float *f = frow + j * 6;
          const float chunk = run * w.inv_Lc;
          f[0] = w8 * (1.f / 8.f); f[1] = w16 * (1.f / 16.f); f[2] = w32 * (1.f / 32.f);
          f[3] = chunk;
          f[4] = old_sum + chunk;
          f[5] = fmaf(kFeatDecay, old_dec, chunk);
        }
      }
    }
  }
  // ---- common exit: every role has drained; the warp that allocated tensor memory frees it ----
  tc_fence_before();
  __syncthreads();
  if (warp == 2) tmem_dealloc(tmem_base, NB * ncols);
}

}  // namespace fkv
