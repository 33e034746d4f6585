// Kernel 3: stable gather-compaction (Section 3.1, s' = s \ D).  Row j of the
// compacted segment is row idx[j] of the old one: K row, V row, feature row
// and position id move together from the old pages into fresh pages, so the
// gather never overwrites a row it still has to read.
//
// Roofline: HBM, 2 x (4D + 4F + 4) bytes per kept pair.  One CTA per (work item,
// tile of 64 output rows), the tiles of an item on consecutive CTAs.  The CTA first resolves index and page-table
// lookups for all its rows in one step, then every warp moves 8 rows: all
// loads first, then all stores, 16 bytes per lane for K and V and one or two
// 32-bit words per lane for the meta row (features + position, one run).
// The 16-byte chunks are re-swizzled for the new row index on the way.
#pragma once
#include "fkv_dev.cuh"

namespace fkv {

constexpr int kCompactRows = 64;  // output rows per CTA (four pages)
constexpr int kCompactRPW = 8;    // rows per warp, all loaded before any is stored

template <int D>
__global__ void __launch_bounds__(256) k_compact(Ctx c, const int32_t *idx, int seg_base, int tiles) {
  constexpr int NCH = D / 8;               // 16-byte chunks per K (or V) row
  static_assert(2 * NCH <= 32, "one chunk per lane");
  __shared__ long long s_src[kCompactRows];  // physical source slot (page * 16 + row) or -1
  __shared__ int s_dst[kCompactRows / kPage];
  const int wk = blockIdx.x / tiles;   // consecutive CTAs: consecutive row tiles of one work item
  if (wk >= c.planhdr[PH_NWORK]) return;
  const int seg = c.work[wk];
  const SegPlan p = c.plan[seg];
  if (!p.active) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int j0 = (blockIdx.x % tiles) * kCompactRows;
  if (j0 >= p.n_new) return;
  // Phase 1: one index and one page-table lookup per output row, all rows of the CTA at once.
  if (threadIdx.x < kCompactRows) {
    const int j = j0 + threadIdx.x;
    long long src = -1;
    if (j < p.n_new) {
      const int s = idx[(size_t)(seg - seg_base) * c.cap + j];
      if (s < 0 || s >= p.n_old) set_status(c, kDevBadIndex);
      else src = (long long)c.pt[(size_t)seg * c.max_pages + s / kPage] * kPage + s % kPage;
    }
    s_src[threadIdx.x] = src;
  } else if (threadIdx.x < kCompactRows + kCompactRows / kPage) {
    const int q = threadIdx.x - kCompactRows, pg = j0 / kPage + q;
    s_dst[q] = pg * kPage < p.n_new ? c.pt_new[(size_t)seg * c.max_pages + pg] : -1;
  }
  __syncthreads();
  // Phase 2: each warp moves 8 rows; lane = one 16-byte chunk of K (0..NCH-1) or V.
  const int MW = c.F + 1;   // words of a meta row (<= 49): lane and lane + 32
  const int isv = lane >= NCH, ch = isv ? lane - NCH : lane;
  const bool kvlane = lane < 2 * NCH;
  uint4 kv[kCompactRPW];
  uint32_t m0[kCompactRPW], m1[kCompactRPW];
  const int r0 = warp * kCompactRPW;
#pragma unroll
  for (int u = 0; u < kCompactRPW; ++u) {
    const long long src = s_src[r0 + u];
    if (src < 0) continue;
    const uint8_t *page = c.pool + (size_t)(src / kPage) * c.page_bytes;
    const int sr = (int)(src % kPage);
    if (kvlane) kv[u] = *reinterpret_cast<const uint4 *>(page + (isv ? c.off_v : 0) + kv_chunk_off(sr, ch, D));
    const uint32_t *mr = reinterpret_cast<const uint32_t *>(meta_row(c, page, sr));
    if (lane < MW) m0[u] = mr[lane];
    if (lane + 32 < MW) m1[u] = mr[lane + 32];
  }
#pragma unroll
  for (int u = 0; u < kCompactRPW; ++u) {
    if (s_src[r0 + u] < 0) continue;
    const int jr = r0 + u, dr = jr % kPage;
    uint8_t *page = c.pool + (size_t)s_dst[jr / kPage] * c.page_bytes;
    if (kvlane) *reinterpret_cast<uint4 *>(page + (isv ? c.off_v : 0) + kv_chunk_off(dr, ch, D)) = kv[u];
    uint32_t *mr = reinterpret_cast<uint32_t *>(meta_row(c, page, dr));
    if (lane < MW) mr[lane] = m0[u];
    if (lane + 32 < MW) mr[lane + 32] = m1[u];
  }
}

}  // namespace fkv
