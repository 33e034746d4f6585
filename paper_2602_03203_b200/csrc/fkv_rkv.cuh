// R-KV baseline score (Appendix E.2): window attention and token-to-token similarity, weighed 0.1 / 0.9.
//
// The paper gives the two weights and no formula.  Reading taken (the library's own):
//     phi_i = lambda_a * a_i - lambda_s * s_i,
//     a_i = the SnapKV score (window-8 attention feature, mean over the g query heads),
//     s_i = max over the OTHER pairs j of the segment of cos(k_i, k_j)   (0 with a zero key or a single pair):
// a pair is redundant when some other pair carries nearly the same key, and redundancy lowers importance.
//
// The maximum does not reduce to anything cheaper than the n x n products <k_i, k_j>: this is a dense
// contraction, 2 n^2 D flops per segment (275 GFLOP at n = 32768, D = 128) against 2 n D bytes of keys that stay
// in L2 - compute-bound, so it runs on the 5th-generation tensor cores.  Nothing of the n x n matrix is ever
// stored: a CTA holds 256 rows (two M = 128 operand tiles) in shared memory, streams the segment's keys past
// them 256 at a time, and reduces every 128 x 256 block of products in the epilogue that reads it from tensor
// memory.
//
// One persistent CTA per SM over a contiguous range of the plan's 128-pair tiles, taken two at a time:
//   warp 0      tensor copies (TMA) of K rows out of page records: one copy = the 16 rows x 64 channels of one page
//               (the tensor map sees the page pool as [page][row][64-channel half][64 channels]), 2 KB that land as
//               16 rows of a K-major operand tile - the page record's swizzle is the shared-memory swizzle.  A lane
//               per copy: the unit's 256 rows once, then the column tiles into a ring, with their reciprocal norms;
//   warp 1      one lane issues tcgen05.mma (bf16 x bf16 -> fp32, M = 128, N = 256, K = 16 per instruction: wide
//               accumulators mean few hand-overs per product, and the hand-over round trip is what tensor memory's
//               room for two of them cannot hide) into one of the two 256-column accumulators and hands them on
//               with tcgen05.commit;
//   warps 4-11  reduce: warp = 32 rows (its tensor-memory lanes) x 128 of the 256 columns; a thread scales the
//               products by the column's reciprocal norm and keeps the running maximum of its row, the next 32
//               columns on their way from tensor memory meanwhile; the diagonal and the columns past the segment's
//               end are masked in the tiles that have them.  The two column halves of a row meet at the unit's end.
// Reciprocal norms and the attention term come from a small kernel that runs before (one thread per pair).
// Every wait is bounded; tensor memory is freed at the common exit.
#pragma once
#include <cuda.h>
#include "fkv_dev.cuh"
#include "fkv_features.cuh"

namespace fkv {

constexpr int kRkvStages = 2;                 // column tiles (256 keys) in the ring
constexpr int kRkvCols = 256;                 // keys per column tile = N of the mma
constexpr int kRkvNormSlots = kRkvStages + 2; // the copies run at most kRkvStages ahead of the mma, the mma at most one tile ahead of the reduction
constexpr int kRkvXch = 4;                    // hand-over slots of the row maxima (by unit)
constexpr int kRkvParts = 2;                  // reducing warps per 32 rows: each takes 256 / kRkvParts columns of an accumulator
constexpr int kRkvThreads = (4 + 4 * kRkvParts) * 32;

struct RkvSmem {
  static __host__ __device__ size_t tile(int D) { return (size_t)(D / 64) * 128 * 128; }   // 128 rows: [D/64][128][128 B]
  // 1 KB alignment slack | A (two tiles) | B ring (two tiles' worth a stage) | reciprocal norms | row maxima | barriers
  static __host__ __device__ size_t bytes(int D) {
    return 1024 + (2 + 2 * kRkvStages) * tile(D) + (size_t)kRkvNormSlots * kRkvCols * 4 + (size_t)kRkvXch * (kRkvParts - 1) * 256 * 4 + 256;
  }
};

// The largest of three (one instruction).
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// 16 rows x 64 columns of an accumulator: thread t = 4 g + q of the warp gets, for each group e of 8 columns, rows g and
// g + 8 of the 16 at columns 8 e + 2 q and 8 e + 2 q + 1 (registers 4 e, 4 e + 1 and 4 e + 2, 4 e + 3).  A thread thus
// meets only 16 of the 64 columns, and only their reciprocal norms have to reach its registers: with a row per thread
// (the 32x32b shape) every thread needs every column's norm, and those broadcast loads - 512 bytes into the register
// file per instruction - kept the shared-memory data path busier than anything else in the kernel.
__device__ __forceinline__ void tmem_ld16x64_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.16x256b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr)
               : "memory");
}

// One warp's share of one accumulator: its 32 rows (tensor-memory lanes from tacc's) x CW columns from tacc's, scaled by
// the columns' reciprocal norms rj[0 .. CW) and folded into the running maxima m[2 s + i] of the thread's rows
// 16 s + g + 8 i (s = 0, 1: the two loads of 16 rows; q = lane & 3 picks the columns).  `plain`: no column is the
// row's own pair or past the segment's end (valid columns; col0 = pair index of column 0, row0 = of the warp's row 0).
template <int CW>
__device__ __forceinline__ void rkv_reduce_item(uint32_t tacc, const float *rj, bool plain, int valid, int col0, int row0,
                                                int lane, float (&m)[4]) {
  const int g = lane >> 2, q = lane & 3;
  uint32_t va[32], vb[32];
  auto fold = [&](const uint32_t (&v)[32], int cb, int s2, const float2 (&nn)[8]) {
    if (plain) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float2 pa = __fmul2_rn(make_float2(__uint_as_float(v[4 * e]), __uint_as_float(v[4 * e + 1])), nn[e]);
        const float2 pb = __fmul2_rn(make_float2(__uint_as_float(v[4 * e + 2]), __uint_as_float(v[4 * e + 3])), nn[e]);
        m[s2] = max3(m[s2], pa.x, pa.y);
        m[s2 + 1] = max3(m[s2 + 1], pb.x, pb.y);
      }
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const int col = cb * 64 + 8 * e + 2 * q + (x & 1), row = row0 + 8 * s2 + g + 8 * (x >> 1);
          const float nx = (x & 1) ? nn[e].y : nn[e].x;
          if (col < valid && col0 + col != row) m[s2 + (x >> 1)] = fmaxf(m[s2 + (x >> 1)], __uint_as_float(v[4 * e + x]) * nx);
        }
      }
    }
  };
  tmem_ld16x64_issue(tacc, va);
  tmem_ld16x64_issue(tacc + (16u << 16), vb);
#pragma unroll
  for (int cb = 0; cb < CW / 64; ++cb) {
    float2 nn[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) nn[e] = *reinterpret_cast<const float2 *>(rj + cb * 64 + 8 * e + 2 * q);
    tmem_ld_wait(va);       // both loads: the wait is for every load of the thread
    tmem_ld_wait(vb);
    fold(va, cb, 0, nn);
    if (cb + 1 < CW / 64) tmem_ld16x64_issue(tacc + (uint32_t)(cb * 64 + 64), va);
    fold(vb, cb, 2, nn);
    if (cb + 1 < CW / 64) tmem_ld16x64_issue(tacc + (16u << 16) + (uint32_t)(cb * 64 + 64), vb);
  }
}
// The four lanes that share a row (q = 0 .. 3) pool their maxima: afterwards every lane holds the four rows' maxima.
__device__ __forceinline__ void rkv_pool_rows(float (&m)[4]) {
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    m[r] = fmaxf(m[r], __shfl_xor_sync(0xffffffffu, m[r], 1));
    m[r] = fmaxf(m[r], __shfl_xor_sync(0xffffffffu, m[r], 2));
  }
}

// One page's K rows, channels 64 q .. 64 q + 63, to 16 consecutive 128-byte rows of an operand tile.
__device__ __forceinline__ void tma_page_k(uint32_t dst, const CUtensorMap *tm, int q, int page, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(0), "r"(q), "r"(0), "r"(page), "r"(bar)
      : "memory");
}

// Before the contraction: thread = pair.  rn[seg * cap + slot] = 1 / |k| (0 for a zero key), and the attention term
// (feature `column` averaged over the g heads, summed in head order and divided in fp32) into
// out[(seg - seg_base) * cap + slot].  grid (work items, 128-pair tiles).
template <int D>
__global__ void __launch_bounds__(128) k_rkv_prepare(Ctx c, float *out, float *rn, int seg_base, int column) {
  if ((int)blockIdx.x >= c.planhdr[PH_NWORK]) return;
  const int seg = c.work[blockIdx.x];
  const int n = c.plan[seg].n_old;
  const int slot = blockIdx.y * 128 + threadIdx.x;
  if (slot >= n) return;
  const uint8_t *page = c.pool + (size_t)c.pt[(size_t)seg * c.max_pages + slot / kPage] * c.page_bytes;
  const uint4 *krow = reinterpret_cast<const uint4 *>(page + (slot % kPage) * 4 * D);   // the chunks' order does not matter here
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < D / 8; ++i) {
    const uint4 u = krow[i];
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float lo = __uint_as_float(w[j] << 16), hi = __uint_as_float(w[j] & 0xffff0000u);
      ss = fmaf(lo, lo, ss);
      ss = fmaf(hi, hi, ss);
    }
  }
  rn[(size_t)seg * c.cap + slot] = ss > 0.f ? 1.f / sqrtf(ss) : 0.f;
  const float *f = meta_row(c, page, slot % kPage) + column;
  float acc = 0.f;
  for (int j = 0; j < c.G; ++j) acc = acc + f[j * 6];
  out[(size_t)(seg - seg_base) * c.cap + slot] = acc / (float)c.G;
}

// The CTA's walk over its tiles [t0, t1): units of up to two consecutive tiles of one segment.
struct RkvWalk {
  int wi, tbeg, tend, seg, n;
};
struct RkvUnit {
  int row0, halves, ntj;   // first row, 128-row halves in use (1 or 2), 256-key column tiles of the segment
};
__device__ __forceinline__ int rkv_unit(const Ctx &c, int t, int t1, RkvWalk &w, RkvUnit &u) {   // returns tiles taken
  if (t >= w.tend) {
    while (t >= c.tile1_start[w.wi + 1]) ++w.wi;
    w.tbeg = c.tile1_start[w.wi]; w.tend = c.tile1_start[w.wi + 1];
    w.seg = c.work[w.wi];
    w.n = c.plan[w.seg].n_old;
  }
  u.row0 = (t - w.tbeg) * 128;
  u.halves = (t + 1 < w.tend && t + 1 < t1) ? 2 : 1;
  u.ntj = (w.n + kRkvCols - 1) / kRkvCols;
  return u.halves;
}


template <int D>
__global__ void __launch_bounds__(kRkvThreads, 1) k_rkv_score(Ctx c, const __grid_constant__ CUtensorMap tmk, float *out,
                                                              const float *rn, int seg_base, float lambda_a, float lambda_s) {
  constexpr int NQ = D / 64, NST = kRkvStages, NR = kRkvNormSlots, NC = kRkvCols;
  constexpr uint32_t PAGE_HALF = kPage * 128;   // bytes of one tensor copy
  extern __shared__ uint8_t smem_raw[];
  const int total = c.planhdr[PH_TILES1], nwork = c.planhdr[PH_NWORK];
  const int per = (total + (int)gridDim.x - 1) / (int)gridDim.x;
  const int t0 = blockIdx.x * per, t1 = min(t0 + per, total);
  if (t0 >= t1) return;                  // nothing allocated yet
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const size_t tb = RkvSmem::tile(D);
  uint8_t *At = smem;                                        // [2][D/64][128 rows][128 B]
  uint8_t *Bt = At + 2 * tb;                                 // [NST][D/64][256 rows][128 B]
  float *Rn = reinterpret_cast<float *>(Bt + NST * 2 * tb);  // [NR][256]
  float *Xch = Rn + NR * NC;                                 // [kRkvXch][kRkvParts - 1][2 halves][128 rows]
  uint64_t *bars = reinterpret_cast<uint64_t *>(Xch + kRkvXch * (kRkvParts - 1) * 256);
  uint64_t *a_full = bars, *a_empty = bars + 1, *b_full = bars + 2, *b_empty = b_full + NST;
  uint64_t *acc_full = b_empty + NST, *acc_empty = acc_full + 2, *x_full = acc_empty + 2;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(x_full + kRkvXch);

  if (warp == 0) tmem_alloc(smem_u32(tmem_slot), 512);   // two accumulators of 256 columns
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(a_full), 1); mbar_init(smem_u32(a_empty), 1);
    for (int s = 0; s < NST; ++s) { mbar_init(smem_u32(&b_full[s]), 1); mbar_init(smem_u32(&b_empty[s]), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&acc_full[b]), 1); mbar_init(smem_u32(&acc_empty[b]), 4 * kRkvParts); }
    for (int x = 0; x < kRkvXch; ++x) mbar_init(smem_u32(&x_full[x]), 4 * (kRkvParts - 1));
    fence_barrier_init();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  RkvWalk w;
  w.wi = find_work(c.tile1_start, nwork, t0);
  w.tend = -1;
  RkvUnit u;

  if (warp == 0) {
    // ---------------- copies: a lane per tensor copy (one page x one 64-channel half) ----------------
    FeatRing br{0, 0};
    int nu = 0, jr = 0;   // units so far (phase of the A barriers); ring slot of the next column tile's norms
    int armed_a = -1;                       // parity of the last phase armed on the barrier of the unit's rows
    uint32_t armed_b = 0, armed_par = 0;    // ... and of the column tiles' stages: bit s = stage s armed at all / its parity
    bool ok = true;
    for (int t = t0; t < t1 && ok;) {
      const int took = rkv_unit(c, t, t1, w, u);
      const int npg = (w.n + kPage - 1) / kPage;
      const int *ptrow = c.pt + (size_t)w.seg * c.max_pages;
      {
        // The unit's rows: lane = (half of the unit, page of the half, channel half).
        const int h = lane >> 4, pg = (lane >> 1) & 7, q = lane & 1;
        const int pa = u.row0 / kPage + h * 8 + pg;
        const bool on = h < u.halves && pa < npg && q < NQ;
        const int pid = on ? ptrow[pa] : 0;
        const int ncopies = __popc(__ballot_sync(0xffffffffu, on));
        if (!mbar_wait_warp(smem_u32(a_empty), (nu & 1) ^ 1)) { set_status(c, kDevWaitTimeout); break; }
        if (lane == 0) mbar_arrive_expect_tx(smem_u32(a_full), (uint32_t)ncopies * PAGE_HALF);
        armed_a = nu & 1;
        __syncwarp();
        if (on) tma_page_k(smem_u32(At + h * tb + (size_t)q * 128 * 128 + (size_t)pg * PAGE_HALF), &tmk, q, pid, smem_u32(a_full));
      }
      // Column tiles: lane = (channel half, page of the tile); the page id is read one tile before its copy.
      const int pg = lane & 15, q = lane >> 4;
      int pidn = (pg < npg && q < NQ) ? ptrow[pg] : 0;
      for (int j = 0; j < u.ntj; ++j) {
        const int pb = j * 16 + pg;
        const bool on = pb < npg && q < NQ;
        const int pid = pidn;
        if (j + 1 < u.ntj) pidn = (pb + 16 < npg && q < NQ) ? ptrow[pb + 16] : 0;
        const int ncopies = __popc(__ballot_sync(0xffffffffu, on));
        if (!mbar_wait_warp(smem_u32(&b_empty[br.i]), br.ph ^ 1)) { set_status(c, kDevWaitTimeout); ok = false; break; }
        const uint32_t nbytes = (uint32_t)min(NC, c.cap - j * NC) * 4u;   // reciprocal norms (entries past the segment's end are masked later)
        if (lane == 0) mbar_arrive_expect_tx(smem_u32(&b_full[br.i]), (uint32_t)ncopies * PAGE_HALF + nbytes);
        armed_b |= 1u << br.i;
        armed_par = (armed_par & ~(1u << br.i)) | ((uint32_t)br.ph << br.i);
        __syncwarp();
        if (on) tma_page_k(smem_u32(Bt + (size_t)br.i * 2 * tb + (size_t)q * NC * 128 + (size_t)pg * PAGE_HALF), &tmk, q, pid, smem_u32(&b_full[br.i]));
        if (lane == 0) bulk_g2s(smem_u32(Rn + jr * NC), rn + (size_t)w.seg * c.cap + (size_t)j * NC, nbytes, smem_u32(&b_full[br.i]));
        br.next(NST);
        if (++jr == NR) jr = 0;
      }
      ++nu;
      t += took;
    }
    // No copy may be in flight at the exit: every armed phase has completed (at once on the ordinary way out, where
    // the multiplies have waited for each of them).
    if (armed_a >= 0 && !mbar_wait_warp(smem_u32(a_full), (uint32_t)armed_a)) set_status(c, kDevWaitTimeout);
#pragma unroll
    for (int s = 0; s < NST; ++s)
      if (((armed_b >> s) & 1u) && !mbar_wait_warp(smem_u32(&b_full[s]), (armed_par >> s) & 1u)) set_status(c, kDevWaitTimeout);
  } else if (warp == 1 && lane == 0) {
    // ---------------- multiplies: one item = (column tile, half) = one accumulator ----------------
    const uint32_t idesc = umma_idesc_bf16(128, NC);
    FeatRing br{0, 0};
    int nu = 0, item = 0;
    bool ok = true;
    for (int t = t0; t < t1 && ok;) {
      const int took = rkv_unit(c, t, t1, w, u);
      if (!mbar_spin(smem_u32(a_full), nu & 1)) { set_status(c, kDevWaitTimeout); break; }
      for (int j = 0; j < u.ntj && ok; ++j) {
        if (!mbar_spin(smem_u32(&b_full[br.i]), br.ph)) { set_status(c, kDevWaitTimeout); ok = false; break; }
        const uint64_t bd0 = umma_desc_sw128(smem_u32(Bt + (size_t)br.i * 2 * tb));
        for (int h = 0; h < u.halves; ++h, ++item) {
          const int slot = item & 1;
          if (!mbar_spin(smem_u32(&acc_empty[slot]), ((item >> 1) & 1) ^ 1)) { set_status(c, kDevWaitTimeout); ok = false; break; }
          tc_fence_after();
          const uint64_t ad0 = umma_desc_sw128(smem_u32(At + h * tb));
          const uint32_t d = tmem_base + (uint32_t)slot * NC;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {        // K = 16 channels per instruction: 32 bytes inside the swizzled row
            const uint64_t offa = (uint64_t)(((ks >> 2) * 128 * 128 + (ks & 3) * 32) >> 4);
            const uint64_t offb = (uint64_t)(((ks >> 2) * NC * 128 + (ks & 3) * 32) >> 4);
            umma_bf16(d, ad0 + offa, bd0 + offb, idesc, ks > 0);
          }
          umma_commit(smem_u32(&acc_full[slot]));      // this accumulator is complete
        }
        if (ok) umma_commit(smem_u32(&b_empty[br.i])); // ... and the tile's stage has been read
        br.next(NST);
      }
      if (ok) umma_commit(smem_u32(a_empty));          // the unit's rows have been read
      ++nu;
      t += took;
    }
  } else if (warp >= 4) {
    // ---------------- reduce: warp = 32 rows (its tensor-memory lanes) x one part of the 256 columns ----------------
    constexpr int CW = NC / kRkvParts;   // this warp's columns of an accumulator
    const int quarter = warp & 3, part = (warp - 4) >> 2, g = lane >> 2, q = lane & 3;
    const int R = quarter * 32 + 16 * (q >> 1) + g + 8 * (q & 1);   // the row of the warp's 32 this lane answers for at a unit's end
    const uint32_t trow0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(part * CW);
    int item = 0, jr = 0, nu = 0;
    bool ok = true;
    for (int t = t0; t < t1 && ok;) {
      const int took = rkv_unit(c, t, t1, w, u);
      float m[2][4];   // running maxima of this thread's four rows (see rkv_reduce_item) in each half
#pragma unroll
      for (int i = 0; i < 8; ++i) m[i >> 2][i & 3] = -INFINITY;
      for (int j = 0; j < u.ntj && ok; ++j) {
        const float *rj = Rn + jr * NC + part * CW;
        const int col0 = j * NC + part * CW;                   // first column of this warp's share
        const int valid = max(0, min(CW, w.n - col0));         // columns of it that are pairs of the segment
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (h < u.halves) {
            const int slot = item & 1;
            if (!mbar_wait_warp(smem_u32(&acc_full[slot]), (item >> 1) & 1)) { set_status(c, kDevWaitTimeout); ok = false; break; }
            tc_fence_after();
            const int rowbase = u.row0 + h * 128;
            const bool plain = valid == CW && (col0 & ~127) != rowbase;   // no diagonal, no columns past the end
            if (valid > 0)
              rkv_reduce_item<CW>(trow0 + (uint32_t)(slot * NC), rj, plain, valid, col0, rowbase + quarter * 32, lane, m[h]);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&acc_empty[slot]));   // this warp's share of the accumulator has been read
            ++item;
          }
        }
        if (++jr == NR) jr = 0;
      }
      // A row's maximum: over the four lanes that share it, then over the column parts - the warps of the other
      // parts hand theirs over.
      float mine[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        rkv_pool_rows(m[h]);
        mine[h] = q == 0 ? m[h][0] : q == 1 ? m[h][1] : q == 2 ? m[h][2] : m[h][3];
      }
      float *xs = Xch + (nu & (kRkvXch - 1)) * (kRkvParts - 1) * 256;
      if (part > 0) {
        xs[(part - 1) * 256 + R] = mine[0];
        xs[(part - 1) * 256 + 128 + R] = mine[1];
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&x_full[nu & (kRkvXch - 1)]));
      } else if (ok) {
        if (!mbar_wait_warp(smem_u32(&x_full[nu & (kRkvXch - 1)]), (nu / kRkvXch) & 1)) { set_status(c, kDevWaitTimeout); break; }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int row = u.row0 + h * 128 + R;
          if (h < u.halves && row < w.n) {
            float mx = mine[h];
#pragma unroll
            for (int x = 0; x < kRkvParts - 1; ++x) mx = fmaxf(mx, xs[x * 256 + h * 128 + R]);
            const float sim = mx > -INFINITY ? __ldg(rn + (size_t)w.seg * c.cap + row) * mx : 0.f;   // a single pair has no other pair
            float *o = out + (size_t)(w.seg - seg_base) * c.cap + row;
            *o = lambda_a * *o - lambda_s * sim;
          }
        }
      }
      ++nu;
      t += took;
    }
  }
  // ---- common exit: every role has drained; the warp that allocated tensor memory frees it ----
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, 512);
}

// ================================================================ the same contraction by pairs of CTAs
// Two CTAs of a cluster (the two SMs of a pair) multiply as one: tcgen05.mma.cta_group::2 takes M = 256 rows - 128
// from each CTA's shared memory - against N = 256 keys - 128 from each CTA's shared memory - and leaves each CTA its
// own 128 rows of the products in its own tensor memory.  A CTA therefore copies only HALF of every column tile
// from L2 (the single-CTA kernel above waits for its copies more than for anything else), and its ring is four
// stages of 32 KB instead of two of 64.  A unit is up to four 128-pair tiles of one segment, dealt out in turn:
// tile k of the unit is half k / 2 of CTA k % 2.
//   warp 0 (both CTAs)   tensor copies of this CTA's rows and of its half of the column tiles; completion is counted
//                        on the FIRST CTA's barriers (the copies name the pair, so that they may signal the peer);
//                        the column tiles' reciprocal norms by 16-byte asynchronous copies on a barrier of this CTA;
//   warp 1 (first CTA)   one lane issues the mma for the pair and hands accumulators, stages and rows on to BOTH
//                        CTAs with one tcgen05.commit each (multicast to the pair);
//   warps 4-11 (both)    reduce this CTA's 128 x 256 accumulator as above; the accumulator is free when the sixteen
//                        warps of the pair have arrived on the first CTA's barrier (the peer's arrive remotely).
// Every wait is bounded; the pair meets at a cluster barrier before tensor memory is freed, so neither CTA leaves
// while the other still reads its shared memory or writes its tensor memory.
constexpr int kRkvPairStages = 4;
constexpr int kRkvPairNormSlots = kRkvPairStages + 2;

struct RkvPairSmem {
  // 1 KB alignment slack | A (two tiles) | B ring (one tile a stage) | reciprocal norms | row maxima | barriers
  static __host__ __device__ size_t bytes(int D) {
    return 1024 + (2 + kRkvPairStages) * RkvSmem::tile(D) + (size_t)kRkvPairNormSlots * kRkvCols * 4 +
           (size_t)kRkvXch * (kRkvParts - 1) * 256 * 4 + 512;
  }
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Arrivals on a barrier of another CTA of the cluster (addr: a shared::cluster address from dsmem_addr).  Relaxed:
// it says "my reads of the accumulator are over" - they are, tcgen05.wait::ld has returned - and publishes nothing
// this thread wrote; with release semantics at cluster scope the arrival held the warp for about a thousand cycles.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t addr) {
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t addr, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.release.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(addr), "r"(bytes) : "memory");
}
// tma_page_k for a CTA of a pair: the barrier may be the peer's.
__device__ __forceinline__ void tma_page_k_pair(uint32_t dst, const CUtensorMap *tm, int q, int page, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(0), "r"(q), "r"(0), "r"(page), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols) {   // one full warp of each CTA of the pair
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {    // the same warps
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// One arrival, when the pair's issued mmas are done, on the barrier at this offset in both CTAs of the pair.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar), "h"((uint16_t)3)
               : "memory");
}
// This thread's earlier 16-byte asynchronous copies, once complete, count as one arrival on the barrier.
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

struct RkvPairUnit {
  int row0, ntl, halves, ntj;   // first row, tiles of the unit (1 .. 4), halves the mma runs over, 256-key column tiles
};
__device__ __forceinline__ int rkv_pair_unit(const Ctx &c, int t, int t1, RkvWalk &w, RkvPairUnit &u) {   // returns tiles taken
  if (t >= w.tend) {
    while (t >= c.tile1_start[w.wi + 1]) ++w.wi;
    w.tbeg = c.tile1_start[w.wi]; w.tend = c.tile1_start[w.wi + 1];
    w.seg = c.work[w.wi];
    w.n = c.plan[w.seg].n_old;
  }
  u.row0 = (t - w.tbeg) * 128;
  u.ntl = min(4, min(w.tend, t1) - t);
  u.halves = (u.ntl + 1) >> 1;
  u.ntj = (w.n + kRkvCols - 1) / kRkvCols;
  return u.ntl;
}

template <int D>
__global__ void __launch_bounds__(kRkvThreads, 1) k_rkv_score_pair(Ctx c, const __grid_constant__ CUtensorMap tmk, float *out,
                                                                   const float *rn, int seg_base, float lambda_a, float lambda_s) {
  constexpr int NQ = D / 64, NST = kRkvPairStages, NR = kRkvPairNormSlots, NC = kRkvCols;
  constexpr uint32_t PAGE_HALF = kPage * 128;   // bytes of one tensor copy
  extern __shared__ uint8_t smem_raw[];
  const int rank = (int)cluster_ctarank();
  const int total = c.planhdr[PH_TILES1], nwork = c.planhdr[PH_NWORK];
  const int npairs = (int)gridDim.x >> 1, pair = (int)blockIdx.x >> 1;
  const int per = (total + npairs - 1) / npairs;
  const int t0 = pair * per, t1 = min(t0 + per, total);
  if (t0 >= t1) return;                  // both CTAs of the pair: nothing allocated yet, no barrier touched
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const size_t tb = RkvSmem::tile(D);
  uint8_t *At = smem;                                        // [2][D/64][128 rows][128 B]: this CTA's rows
  uint8_t *Bt = At + 2 * tb;                                 // [NST][D/64][128 rows][128 B]: this CTA's half of a column tile
  float *Rn = reinterpret_cast<float *>(Bt + NST * tb);      // [NR][256]
  float *Xch = Rn + NR * NC;                                 // [kRkvXch][kRkvParts - 1][2 halves][128 rows]
  uint64_t *bars = reinterpret_cast<uint64_t *>(Xch + kRkvXch * (kRkvParts - 1) * 256);
  uint64_t *a_full = bars, *a_empty = bars + 1, *b_full = bars + 2, *b_empty = b_full + NST;
  uint64_t *acc_full = b_empty + NST, *acc_empty = acc_full + 2, *x_full = acc_empty + 2, *n_full = x_full + kRkvXch;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(n_full + NR);

  if (warp == 0) tmem_alloc_pair(smem_u32(tmem_slot), 512);   // two accumulators of 256 columns in each CTA
  if (threadIdx.x == 0) {
    // a_full, b_full, acc_empty are used in the first CTA only: both CTAs arrive there.
    mbar_init(smem_u32(a_full), 2); mbar_init(smem_u32(a_empty), 1);
    for (int s = 0; s < NST; ++s) { mbar_init(smem_u32(&b_full[s]), 2); mbar_init(smem_u32(&b_empty[s]), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&acc_full[b]), 1); mbar_init(smem_u32(&acc_empty[b]), 2 * 4 * kRkvParts); }
    for (int x = 0; x < kRkvXch; ++x) mbar_init(smem_u32(&x_full[x]), 4 * (kRkvParts - 1));
    for (int i = 0; i < NR; ++i) mbar_init(smem_u32(&n_full[i]), 32);
    fence_barrier_init();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();        // the peer's barriers are initialised before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  RkvWalk w;
  w.wi = find_work(c.tile1_start, nwork, t0);
  w.tend = -1;
  RkvPairUnit u;

  if (warp == 0) {
    // ---------------- copies: a lane per tensor copy (one page x one 64-channel half) ----------------
    const uint32_t lead_a_full = dsmem_addr(smem_u32(a_full), 0);
    FeatRing br{0, 0};
    int nu = 0, jr = 0;   // units so far (phase of the A barriers); ring slot of the next column tile's norms
    bool ok = true;
    for (int t = t0; t < t1 && ok;) {
      const int took = rkv_pair_unit(c, t, t1, w, u);
      const int npg = (w.n + kPage - 1) / kPage;
      const int *ptrow = c.pt + (size_t)w.seg * c.max_pages;
      {
        // This CTA's rows: lane = (half, page of the half's tile, channel half); half h is tile 2 h + rank of the unit.
        const int h = lane >> 4, pg = (lane >> 1) & 7, q = lane & 1, k = 2 * h + rank;
        const int pa = u.row0 / kPage + k * 8 + pg;
        const bool on = k < u.ntl && pa < npg && q < NQ;
        const int pid = on ? ptrow[pa] : 0;
        const int ncopies = __popc(__ballot_sync(0xffffffffu, on));
        if (!mbar_wait_warp(smem_u32(a_empty), (nu & 1) ^ 1)) { set_status(c, kDevWaitTimeout); break; }
        if (lane == 0) mbar_arrive_expect_tx_cluster(lead_a_full, (uint32_t)ncopies * PAGE_HALF);
        __syncwarp();
        if (on) tma_page_k_pair(smem_u32(At + h * tb + (size_t)q * 128 * 128 + (size_t)pg * PAGE_HALF), &tmk, q, pid, lead_a_full);
      }
      // This CTA's half of the column tiles: lanes 0-15 = (channel half, page); the page id is read one tile before
      // its copy.  All lanes: 32 bytes of the tile's reciprocal norms.
      const int pg = lane & 7, q = (lane >> 3) & 1;
      const bool copier = lane < 16 && q < NQ;
      int pidn = (copier && rank * 8 + pg < npg) ? ptrow[rank * 8 + pg] : 0;
      for (int j = 0; j < u.ntj; ++j) {
        const int pb = j * 16 + rank * 8 + pg;
        const bool on = copier && pb < npg;
        const int pid = pidn;
        if (j + 1 < u.ntj) pidn = (copier && pb + 16 < npg) ? ptrow[pb + 16] : 0;
        const int ncopies = __popc(__ballot_sync(0xffffffffu, on));
        if (!mbar_wait_warp(smem_u32(&b_empty[br.i]), br.ph ^ 1)) { set_status(c, kDevWaitTimeout); ok = false; break; }
        const uint32_t lead_b_full = dsmem_addr(smem_u32(&b_full[br.i]), 0);
        if (lane == 0) mbar_arrive_expect_tx_cluster(lead_b_full, (uint32_t)ncopies * PAGE_HALF);
        __syncwarp();
        if (on) tma_page_k_pair(smem_u32(Bt + (size_t)br.i * tb + (size_t)q * 128 * 128 + (size_t)pg * PAGE_HALF), &tmk, q, pid, lead_b_full);
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const int col = j * NC + k * 128 + lane * 4;   // entries past the segment's end are masked later
          if (col < c.cap) cp_async16(smem_u32(Rn + jr * NC + k * 128 + lane * 4), rn + (size_t)w.seg * c.cap + col);
        }
        cp_async_arrive(smem_u32(&n_full[jr]));
        br.next(NST);
        if (++jr == NR) jr = 0;
      }
      ++nu;
      t += took;
    }
    // No copy may be in flight at the exit.  The tensor copies are waited for by the first CTA's multiplies (or, after
    // a failed wait, are complete long before the bounded waits of the other roles have run out and the pair has met
    // at the cluster barrier); the 16-byte copies here:
    cp_async_wait_all();
  } else if (warp == 1 && lane == 0 && rank == 0) {
    // ---------------- multiplies, for the pair: one item = (column tile, half) = one accumulator in each CTA ----------------
    const uint32_t idesc = umma_idesc_bf16(256, NC);
    FeatRing br{0, 0};
    int nu = 0, item = 0;
    bool ok = true;
    for (int t = t0; t < t1 && ok;) {
      const int took = rkv_pair_unit(c, t, t1, w, u);
      if (!mbar_spin(smem_u32(a_full), nu & 1)) { set_status(c, kDevWaitTimeout); break; }
      for (int j = 0; j < u.ntj && ok; ++j) {
        if (!mbar_spin(smem_u32(&b_full[br.i]), br.ph)) { set_status(c, kDevWaitTimeout); ok = false; break; }
        const uint64_t bd0 = umma_desc_sw128(smem_u32(Bt + (size_t)br.i * tb));
        for (int h = 0; h < u.halves; ++h, ++item) {
          const int slot = item & 1;
          if (!mbar_spin(smem_u32(&acc_empty[slot]), ((item >> 1) & 1) ^ 1)) { set_status(c, kDevWaitTimeout); ok = false; break; }
          tc_fence_after();
          const uint64_t ad0 = umma_desc_sw128(smem_u32(At + h * tb));
          const uint32_t d = tmem_base + (uint32_t)slot * NC;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {        // K = 16 channels per instruction: 32 bytes inside the swizzled row
            const uint64_t off = (uint64_t)(((ks >> 2) * 128 * 128 + (ks & 3) * 32) >> 4);
            umma_bf16_pair(d, ad0 + off, bd0 + off, idesc, ks > 0);
          }
          umma_commit_pair(smem_u32(&acc_full[slot]));      // this accumulator is complete, in both CTAs
        }
        if (ok) umma_commit_pair(smem_u32(&b_empty[br.i])); // ... and both halves of the tile's stage have been read
        br.next(NST);
      }
      if (ok) umma_commit_pair(smem_u32(a_empty));          // the unit's rows have been read
      ++nu;
      t += took;
    }
  } else if (warp >= 4) {
    // ---------------- reduce: warp = 32 of this CTA's rows (its tensor-memory lanes) x one part of the 256 columns ----------------
    constexpr int CW = NC / kRkvParts;   // this warp's columns of an accumulator
    const int quarter = warp & 3, part = (warp - 4) >> 2, g = lane >> 2, q = lane & 3;
    const int R = quarter * 32 + 16 * (q >> 1) + g + 8 * (q & 1);   // the row of the warp's 32 this lane answers for at a unit's end
    const uint32_t trow0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(part * CW);
    int item = 0, jr = 0, nu = 0, nuse = 0;   // nuse: times the norm ring has gone round
    bool ok = true;
    for (int t = t0; t < t1 && ok;) {
      const int took = rkv_pair_unit(c, t, t1, w, u);
      float m[2][4];   // running maxima of this thread's four rows (see rkv_reduce_item) in each half
#pragma unroll
      for (int i = 0; i < 8; ++i) m[i >> 2][i & 3] = -INFINITY;
      for (int j = 0; j < u.ntj && ok; ++j) {
        const float *rj = Rn + jr * NC + part * CW;
        const int col0 = j * NC + part * CW;                   // first column of this warp's share
        const int valid = max(0, min(CW, w.n - col0));         // columns of it that are pairs of the segment
        if (!mbar_wait_warp(smem_u32(&n_full[jr]), nuse & 1)) { set_status(c, kDevWaitTimeout); ok = false; break; }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (h < u.halves) {
            const int slot = item & 1;
            if (!mbar_wait_warp(smem_u32(&acc_full[slot]), (item >> 1) & 1)) { set_status(c, kDevWaitTimeout); ok = false; break; }
            tc_fence_after();
            const int k = 2 * h + rank, rowbase = u.row0 + k * 128;
            const bool plain = valid == CW && (col0 & ~127) != rowbase;   // no diagonal, no columns past the end
            if (valid > 0 && k < u.ntl)
              rkv_reduce_item<CW>(trow0 + (uint32_t)(slot * NC), rj, plain, valid, col0, rowbase + quarter * 32, lane, m[h]);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {   // this warp's share of the accumulator has been read
              if (rank == 0) mbar_arrive(smem_u32(&acc_empty[slot]));
              else mbar_arrive_cluster(dsmem_addr(smem_u32(&acc_empty[slot]), 0));
            }
            ++item;
          }
        }
        if (++jr == NR) { jr = 0; ++nuse; }
      }
      // A row's maximum: over the four lanes that share it, then over the column parts - the warps of the other
      // parts hand theirs over.
      float mine[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        rkv_pool_rows(m[h]);
        mine[h] = q == 0 ? m[h][0] : q == 1 ? m[h][1] : q == 2 ? m[h][2] : m[h][3];
      }
      float *xs = Xch + (nu & (kRkvXch - 1)) * (kRkvParts - 1) * 256;
      if (part > 0) {
        xs[(part - 1) * 256 + R] = mine[0];
        xs[(part - 1) * 256 + 128 + R] = mine[1];
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&x_full[nu & (kRkvXch - 1)]));
      } else if (ok) {
        if (!mbar_wait_warp(smem_u32(&x_full[nu & (kRkvXch - 1)]), (nu / kRkvXch) & 1)) { set_status(c, kDevWaitTimeout); break; }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int k = 2 * h + rank, row = u.row0 + k * 128 + R;
          if (k < u.ntl && row < w.n) {
            float mx = mine[h];
#pragma unroll
            for (int x = 0; x < kRkvParts - 1; ++x) mx = fmaxf(mx, xs[x * 256 + h * 128 + R]);
            const float sim = mx > -INFINITY ? __ldg(rn + (size_t)w.seg * c.cap + row) * mx : 0.f;   // a single pair has no other pair
            float *o = out + (size_t)(w.seg - seg_base) * c.cap + row;
            *o = lambda_a * *o - lambda_s * sim;
          }
        }
      }
      ++nu;
      t += took;
    }
  }
  // ---- common exit: every role of both CTAs has drained; the warps that allocated tensor memory free it ----
  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();
  if (warp == 0) tmem_dealloc_pair(tmem_base, 512);
}

}  // namespace fkv
