// Kernel 3: stable gather-compaction (Section 3.1, s' = s \ D).  Row j of the
// compacted segment is row idx[j] of the old one: K row, V row, feature row
// and position id move together from the old pages into fresh pages, so the
// gather never overwrites a row it still has to read.
//
// Roofline: HBM, 2 x (4D + 4F + 4) bytes per kept pair.  grid (tiles of 32
// output rows, work list); a warp moves 4 rows: all loads first, then all
// stores, 16 bytes per lane for K and V.  The 16-byte chunks are re-swizzled
// for the new row index on the way.
#pragma once
#include "fkv_dev.cuh"

namespace fkv {

constexpr int kCompactRows = 32;  // output rows per CTA (two pages)

template <int D>
__global__ void __launch_bounds__(256) k_compact(Ctx c, const int32_t *idx, int seg_base) {
  constexpr int NCH = D / 8;               // 16-byte chunks per K (or V) row
  constexpr int QPL = (2 * NCH + 31) / 32;  // chunks per lane (1 for D = 128 and 64)
  if ((int)blockIdx.y >= c.planhdr[PH_NWORK]) return;
  const int seg = c.work[blockIdx.y];
  const SegPlan p = c.plan[seg];
  if (!p.active) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int j0 = blockIdx.x * kCompactRows + warp * 4;
  if (j0 >= p.n_new) return;
  const int32_t *ix = idx + (size_t)(seg - seg_base) * c.cap;
  const int *ptold = c.pt + (size_t)seg * c.max_pages, *ptnew = c.pt_new + (size_t)seg * c.max_pages;
  const int FH = c.F >> 1;  // 8-byte feature chunks per row

  const uint8_t *src[4];
  int sr[4];
  bool ok[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int j = j0 + u;
    ok[u] = j < p.n_new;
    int s = ok[u] ? ix[j] : 0;
    if (ok[u] && (s < 0 || s >= p.n_old)) {
      if (lane == 0) set_status(c, kDevBadIndex);
      ok[u] = false;
      s = 0;
    }
    sr[u] = s % kPage;
    src[u] = c.pool + (size_t)ptold[s / kPage] * c.page_bytes;
  }
  uint4 kv[4][QPL];
  float2 ft[4][2];
  int32_t ps[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    if (!ok[u]) continue;
#pragma unroll
    for (int q = 0; q < QPL; ++q) {
      const int ch2 = lane + q * 32;
      if (ch2 < 2 * NCH) {
        const int isv = ch2 >= NCH, ch = isv ? ch2 - NCH : ch2;
        kv[u][q] = *reinterpret_cast<const uint4 *>(src[u] + (isv ? c.off_v : 0) + kv_chunk_off(sr[u], ch));
      }
    }
    const float2 *f = reinterpret_cast<const float2 *>(src[u] + c.off_f) + sr[u] * FH;
#pragma unroll
    for (int q = 0; q < 2; ++q)
      if (lane + q * 32 < FH) ft[u][q] = f[lane + q * 32];
    if (lane == 31) ps[u] = reinterpret_cast<const int32_t *>(src[u] + c.off_p)[sr[u]];
  }
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    if (!ok[u]) continue;
    const int j = j0 + u, dr = j % kPage;
    uint8_t *dst = c.pool + (size_t)ptnew[j / kPage] * c.page_bytes;
#pragma unroll
    for (int q = 0; q < QPL; ++q) {
      const int ch2 = lane + q * 32;
      if (ch2 < 2 * NCH) {
        const int isv = ch2 >= NCH, ch = isv ? ch2 - NCH : ch2;
        *reinterpret_cast<uint4 *>(dst + (isv ? c.off_v : 0) + kv_chunk_off(dr, ch)) = kv[u][q];
      }
    }
    float2 *f = reinterpret_cast<float2 *>(dst + c.off_f) + dr * FH;
#pragma unroll
    for (int q = 0; q < 2; ++q)
      if (lane + q * 32 < FH) f[lane + q * 32] = ft[u][q];
    if (lane == 31) reinterpret_cast<int32_t *>(dst + c.off_p)[dr] = ps[u];
  }
}

}  // namespace fkv
