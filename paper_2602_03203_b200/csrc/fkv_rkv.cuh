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
// them 128 at a time, and reduces every 128 x 128 block of products in the epilogue that reads it from tensor
// memory.
//
// One persistent CTA per SM over a contiguous range of the plan's 128-pair tiles, taken two at a time:
//   warps 0-3   copy K rows of page records into K-major operand tiles (16-byte asynchronous copies; the page
//               record's swizzle is the shared-memory swizzle), the CTA's 256 rows once, then the column tiles
//               into a ring, with the column tile's reciprocal norms;
//   warp 4      one lane issues tcgen05.mma (bf16 x bf16 -> fp32, M = N = 128, K = 16 per instruction) into one of
//               two pairs of accumulators in tensor memory and hands them on with tcgen05.commit;
//   warps 8-15  two warpgroups, one per 128 rows: a thread owns one row (its tensor-memory lane), scales the
//               products by the column's reciprocal norm and keeps the running maximum; the diagonal and the
//               columns past the segment's end are masked in the two tiles that have them.
// Reciprocal norms and the attention term come from a small kernel that runs before (one thread per pair).
// Every wait is bounded; tensor memory is freed at the common exit.
#pragma once
#include "fkv_dev.cuh"
#include "fkv_features.cuh"

namespace fkv {

constexpr int kRkvStages = 4;                 // column tiles in flight
constexpr int kRkvNormSlots = kRkvStages + 3; // the copies run at most kRkvStages ahead of the mma, the mma at most 2 ahead of the reduction
constexpr int kRkvThreads = 16 * 32;

struct RkvSmem {
  static __host__ __device__ size_t tile(int D) { return (size_t)(D / 64) * 128 * 128; }   // [D/64][128 rows][128 B]
  // 1 KB alignment slack | A (two tiles) | B ring | reciprocal norms | barriers
  static __host__ __device__ size_t bytes(int D) {
    return 1024 + (2 + kRkvStages) * tile(D) + (size_t)kRkvNormSlots * 128 * 4 + 256;
  }
};

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
  int row0, halves, ntj;   // first row, 128-row halves in use (1 or 2), column tiles of the segment
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
  u.ntj = (w.n + 127) / 128;
  return u.halves;
}

template <int D>
__global__ void __launch_bounds__(kRkvThreads, 1) k_rkv_score(Ctx c, float *out, const float *rn, int seg_base,
                                                              float lambda_a, float lambda_s) {
  constexpr int NCH = D / 8, RSTEP = 128 / NCH, NST = kRkvStages, NR = kRkvNormSlots;
  extern __shared__ uint8_t smem_raw[];
  const int total = c.planhdr[PH_TILES1], nwork = c.planhdr[PH_NWORK];
  const int per = (total + (int)gridDim.x - 1) / (int)gridDim.x;
  const int t0 = blockIdx.x * per, t1 = min(t0 + per, total);
  if (t0 >= t1) return;                  // nothing allocated yet
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const size_t tb = RkvSmem::tile(D);
  uint8_t *At = smem;                                    // [2][HALVES][128][128 B]
  uint8_t *Bt = At + 2 * tb;                             // [NST][HALVES][128][128 B]
  float *Rn = reinterpret_cast<float *>(Bt + NST * tb);  // [NR][128]
  uint64_t *bars = reinterpret_cast<uint64_t *>(Rn + NR * 128);
  uint64_t *a_full = bars, *a_empty = bars + 1, *b_full = bars + 2, *b_empty = b_full + NST;
  uint64_t *acc_full = b_empty + NST, *acc_empty = acc_full + 2;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);

  if (warp == 0) tmem_alloc(smem_u32(tmem_slot), 512);   // two pairs of 128-column accumulators
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(a_full), 128); mbar_init(smem_u32(a_empty), 1);
    for (int s = 0; s < NST; ++s) { mbar_init(smem_u32(&b_full[s]), 128); mbar_init(smem_u32(&b_empty[s]), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&acc_full[b]), 1); mbar_init(smem_u32(&acc_empty[b]), 8); }
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

  if (warp < 4) {
    // ---------------- copies: thread = one 16-byte chunk column of rows R0, R0 + RSTEP, ... of every page ----------------
    const int p = threadIdx.x, ch = p % NCH, R0 = p / NCH;
    const uint32_t dcol = (uint32_t)((ch >> 3) * 128 * 128 + (ch & 7) * 16);
    // One 128-row tile of the segment (its pages pg0 ..) into the operand tile at dst.
    auto copy_tile = [&](uint32_t dst, int pg0) {
      const int np = min(8, (w.n + kPage - 1) / kPage - pg0);
      const int *ptrow = c.pt + (size_t)w.seg * c.max_pages + pg0;
      int pid[8];
#pragma unroll
      for (int pg = 0; pg < 8; ++pg) pid[pg] = ptrow[min(pg, max(np - 1, 0))];
#pragma unroll
      for (int pg = 0; pg < 8; ++pg) {
        if (pg < np) {
          const uint8_t *page = c.pool + (size_t)pid[pg] * c.page_bytes + ch * 16;
#pragma unroll
          for (int k = 0; k < kPage / RSTEP; ++k) {
            const int r = R0 + k * RSTEP;
            cp_async16(dst + dcol + (uint32_t)((pg * kPage + r) * 128), page + r * 4 * D);
          }
        }
      }
    };
    // The column tiles are copied two ahead: the copies of tile j are issued before those of tile j - 2 are waited
    // for (a copy from L2 takes longer than the multiplies of a tile), and a tile is handed over - this thread's
    // copies complete, made visible to the tensor core's reads, one arrival - two tiles after it was asked for.
    FeatRing br{0, 0}, done{0, 0};
    int nu = 0, jr = 0;   // units so far (phase of the A barriers); ring slot of the next column tile's norms
    bool ok = true;
    auto hand_over = [&]() {
      fence_proxy_async();
      mbar_arrive(smem_u32(&b_full[done.i]));
      done.next(NST);
    };
    for (int t = t0; t < t1 && ok;) {
      const int took = rkv_unit(c, t, t1, w, u);
      if (!mbar_wait_warp(smem_u32(a_empty), (nu & 1) ^ 1)) { set_status(c, kDevWaitTimeout); break; }
      for (int h = 0; h < u.halves; ++h) copy_tile(smem_u32(At + h * tb), (u.row0 + h * 128) / kPage);
      cp_async_wait_all();
      fence_proxy_async();
      mbar_arrive(smem_u32(a_full));
      int inflight = 0;
      for (int j = 0; j < u.ntj; ++j) {
        if (!mbar_wait_warp(smem_u32(&b_empty[br.i]), br.ph ^ 1)) { set_status(c, kDevWaitTimeout); ok = false; break; }
        copy_tile(smem_u32(Bt + br.i * tb), j * 8);
        if (p < 32 && j * 128 + p * 4 < c.cap)   // this tile's reciprocal norms (entries past the segment's end are masked later)
          cp_async16(smem_u32(Rn + jr * 128 + p * 4), rn + (size_t)w.seg * c.cap + j * 128 + p * 4);
        cp_async_commit();
        br.next(NST);
        if (++jr == NR) jr = 0;
        if (++inflight == 3) {
          cp_async_wait_pending<2>();
          hand_over();
          --inflight;
        }
      }
      // The last tiles of the unit (on a failed wait too: nothing may be in flight at the exit).
      cp_async_wait_pending<0>();
      for (; inflight > 0 && ok; --inflight) hand_over();
      ++nu;
      t += took;
    }
  } else if (warp == 4 && lane == 0) {
    // ---------------- multiplies ----------------
    const uint32_t idesc = umma_idesc_bf16(128, 128);
    FeatRing br{0, 0};
    int nu = 0, uacc = 0;
    bool ok = true;
    for (int t = t0; t < t1 && ok;) {
      const int took = rkv_unit(c, t, t1, w, u);
      if (!mbar_spin(smem_u32(a_full), nu & 1)) { set_status(c, kDevWaitTimeout); break; }
      for (int j = 0; j < u.ntj; ++j, ++uacc) {
        const int b = uacc & 1;
        if (!mbar_spin(smem_u32(&b_full[br.i]), br.ph) || !mbar_spin(smem_u32(&acc_empty[b]), ((uacc >> 1) & 1) ^ 1)) {
          set_status(c, kDevWaitTimeout); ok = false; break;
        }
        tc_fence_after();
        const uint64_t bd0 = umma_desc_sw128(smem_u32(Bt + br.i * tb));
        for (int h = 0; h < u.halves; ++h) {
          const uint64_t ad0 = umma_desc_sw128(smem_u32(At + h * tb));
          const uint32_t d = tmem_base + (uint32_t)(b * 2 + h) * 128;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {        // K = 16 channels per instruction: 32 bytes inside the swizzled row
            const uint64_t off = (uint64_t)(((ks >> 2) * 128 * 128 + (ks & 3) * 32) >> 4);
            umma_bf16(d, ad0 + off, bd0 + off, idesc, ks > 0);
          }
        }
        umma_commit(smem_u32(&acc_full[b]));       // the accumulators of this column tile are complete
        umma_commit(smem_u32(&b_empty[br.i]));     // ... and its stage has been read
        br.next(NST);
      }
      if (ok) umma_commit(smem_u32(a_empty));      // the unit's rows have been read
      ++nu;
      t += took;
    }
  } else if (warp >= 8) {
    // ---------------- reduce: thread = one row of the unit (its tensor-memory lane) ----------------
    const int h = (warp - 8) >> 2, quarter = warp & 3, R = quarter * 32 + lane;
    const uint32_t trow0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)h * 128;
    int uacc = 0, jr = 0;
    bool ok = true;
    for (int t = t0; t < t1 && ok;) {
      const int took = rkv_unit(c, t, t1, w, u);
      const int row = u.row0 + h * 128 + R;
      const bool live = h < u.halves && row < w.n;
      const float rn_i = live ? __ldg(rn + (size_t)w.seg * c.cap + row) : 0.f;
      const int jdiag = (u.row0 + h * 128) >> 7;   // the column tile that holds this warpgroup's diagonal
      float m = -INFINITY;
      for (int j = 0; j < u.ntj; ++j, ++uacc) {
        const int b = uacc & 1;
        if (!mbar_wait_warp(smem_u32(&acc_full[b]), (uacc >> 1) & 1)) { set_status(c, kDevWaitTimeout); ok = false; break; }
        tc_fence_after();
        if (h < u.halves) {
          const float *rj = Rn + jr * 128;
          const int valid = min(128, w.n - j * 128);   // columns of this tile that are pairs of the segment
          const bool plain = j != jdiag && valid == 128;
#pragma unroll 1
          for (int c4 = 0; c4 < 4; ++c4) {
            uint32_t v[32];
            tmem_ld32_issue(trow0 + (uint32_t)(b * 256 + c4 * 32), v);
            tmem_ld_wait(v);
            if (plain) {
#pragma unroll
              for (int k = 0; k < 32; k += 4) {
                const float4 r4 = *reinterpret_cast<const float4 *>(rj + c4 * 32 + k);
                m = fmaxf(m, fmaxf(fmaxf(__uint_as_float(v[k]) * r4.x, __uint_as_float(v[k + 1]) * r4.y),
                                   fmaxf(__uint_as_float(v[k + 2]) * r4.z, __uint_as_float(v[k + 3]) * r4.w)));
              }
            } else {
#pragma unroll
              for (int k = 0; k < 32; ++k) {
                const int col = c4 * 32 + k;
                if (col < valid && j * 128 + col != row) m = fmaxf(m, __uint_as_float(v[k]) * rj[col]);
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&acc_empty[b]));   // this warp's share of the accumulators has been read
        if (++jr == NR) jr = 0;
      }
      if (live && ok) {
        const float s = m > -INFINITY ? rn_i * m : 0.f;        // a single pair has no other pair
        float *o = out + (size_t)(w.seg - seg_base) * c.cap + row;
        *o = lambda_a * *o - lambda_s * s;
      }
      t += took;
    }
  }
  // ---- common exit: every role has drained; the warp that allocated tensor memory frees it ----
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, 512);
}

}  // namespace fkv
