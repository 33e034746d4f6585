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
//   warp 1      one lane issues tcgen05.mma (bf16 x bf16 -> fp32, M = 128, N = 256, K = 16 per instruction: an
//               instruction takes about 130 cycles whatever its N up to 128, and 155 at N = 256) into one of the
//               two 256-column accumulators of tensor memory and hands them on with tcgen05.commit;
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
    // ---------------- reduce: warp = 32 rows (its tensor-memory lanes) x one half of the 256 columns ----------------
    constexpr int CW = NC / kRkvParts, NCHUNK = CW / 32;   // this warp's columns of an accumulator
    const int quarter = warp & 3, part = (warp - 4) >> 2, R = quarter * 32 + lane;
    const uint32_t trow0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(part * CW);
    int item = 0, jr = 0, nu = 0;
    bool ok = true;
    for (int t = t0; t < t1 && ok;) {
      const int took = rkv_unit(c, t, t1, w, u);
      float m[2] = {-INFINITY, -INFINITY};   // running maxima of this thread's row in each half of the unit
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
            const int row = u.row0 + h * 128 + R;
            const bool plain = valid == CW && (col0 & ~127) != u.row0 + h * 128;   // no diagonal, no columns past the end
            float mm = m[h];
            // 32 columns at a time, the next 32 on their way from tensor memory meanwhile.
            auto reduce32 = [&](const uint32_t (&v)[32], int c4) {
              if (plain) {
                float m1 = -INFINITY;
#pragma unroll
                for (int k = 0; k < 32; k += 4) {
                  const float4 r4 = *reinterpret_cast<const float4 *>(rj + c4 * 32 + k);
                  const float2 p0 = __fmul2_rn(make_float2(__uint_as_float(v[k]), __uint_as_float(v[k + 1])), make_float2(r4.x, r4.y));
                  const float2 p1 = __fmul2_rn(make_float2(__uint_as_float(v[k + 2]), __uint_as_float(v[k + 3])), make_float2(r4.z, r4.w));
                  mm = max3(mm, p0.x, p0.y);
                  m1 = max3(m1, p1.x, p1.y);
                }
                mm = fmaxf(mm, m1);
              } else {
#pragma unroll
                for (int k = 0; k < 32; ++k) {
                  const int col = c4 * 32 + k;
                  if (col < valid && col0 + col != row) mm = fmaxf(mm, __uint_as_float(v[k]) * rj[col]);
                }
              }
            };
            if (valid > 0) {
              const uint32_t tacc = trow0 + (uint32_t)(slot * NC);
              uint32_t va[32], vb[32];
              tmem_ld32_issue(tacc, va);
#pragma unroll
              for (int cc = 0; cc < NCHUNK; cc += 2) {
                tmem_ld_wait(va);
                tmem_ld32_issue(tacc + (uint32_t)(cc * 32 + 32), vb);
                reduce32(va, cc);
                tmem_ld_wait(vb);
                if (cc + 2 < NCHUNK) tmem_ld32_issue(tacc + (uint32_t)(cc * 32 + 64), va);
                reduce32(vb, cc + 1);
              }
            }
            m[h] = mm;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&acc_empty[slot]));   // this warp's share of the accumulator has been read
            ++item;
          }
        }
        if (++jr == NR) jr = 0;
      }
      // The column parts of a row meet: the warps of the other parts hand their maxima over.
      float *xs = Xch + (nu & (kRkvXch - 1)) * (kRkvParts - 1) * 256;
      if (part > 0) {
        xs[(part - 1) * 256 + R] = m[0];
        xs[(part - 1) * 256 + 128 + R] = m[1];
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&x_full[nu & (kRkvXch - 1)]));
      } else if (ok) {
        if (!mbar_wait_warp(smem_u32(&x_full[nu & (kRkvXch - 1)]), (nu / kRkvXch) & 1)) { set_status(c, kDevWaitTimeout); break; }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int row = u.row0 + h * 128 + R;
          if (h < u.halves && row < w.n) {
            float mx = m[h];
#pragma unroll
            for (int q = 0; q < kRkvParts - 1; ++q) mx = fmaxf(mx, xs[q * 256 + h * 128 + R]);
            const float s = mx > -INFINITY ? __ldg(rn + (size_t)w.seg * c.cap + row) * mx : 0.f;   // a single pair has no other pair
            float *o = out + (size_t)(w.seg - seg_base) * c.cap + row;
            *o = lambda_a * *o - lambda_s * s;
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

}  // namespace fkv
