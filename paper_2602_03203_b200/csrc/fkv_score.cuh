// Kernel 1: the scorer of Appendix B.1,
//     phi_n = sigma(x_n W1 + b1) W2 + b2,   x_n = Concat(k_n, v_n, a_n),
// streamed over every pair of the segments on the work list.
//
// Roofline: HBM.  A pair is 4D + 4F bytes in and 4 bytes out, but 2(2D+F)H
// flops, which is more than the fp32 pipes can do at HBM speed, so the whole
// x W1 product runs on the tensor cores with fp32 accumulation and every
// operand carried at (nearly) fp32 precision by splitting it into parts the
// tensor cores multiply exactly:
//   k, v (bf16 data) x W1 rows (fp32): bf16 mma, the weight as rounding +
//       remainder (two bf16 values);
//   a (fp32 data) x W1 rows (fp32): tf32 mma, feature and weight each as a
//       truncation to tf32 + the remainder, three of the four cross products
//       (the fourth is below 2^-20 of the term).
//
// Structure: persistent CTAs, one per SM, each a contiguous range of tiles
// (NCW consecutive pages of one segment).  The pages of the range go round a
// ring of page slots in shared memory (as many as fit), each slot with its own
// mbarrier, and round the warps: whole page records (16 pairs: K, V, features
// + positions, one contiguous block) arrive from HBM by one bulk async copy
// per page, issued into a slot by the warp that has just scored the slot's
// previous page - no warp waits for another warp's progress, only for its own
// page to land, and no warp is set aside for copying (eight warps, two per
// scheduler, leave each thread 255 registers).  ldmatrix reads the pre-swizzled K and V rows as A fragments;
// the K/V rows of W1 sit in registers as B fragments, the feature rows in a
// per-warp shared-memory copy (also as B fragments).  Both are reloaded when
// the segment (and so the scorer) changes.
#pragma once
#include "fkv_dev.cuh"

namespace fkv {

__device__ __forceinline__ float activate(float z, int act) {
  switch (act) {
    case 0: return fmaxf(z, 0.f);
    case 1: return z / (1.f + __expf(-z));
    case 2: return 0.5f * z * (1.f + tanhf(0.7978845608028654f * (z + 0.044715f * z * z * z)));
    default: return 1.f / (1.f + __expf(-z));
  }
}

// Largest w with start[w] <= t, start[] ascending with start[0] = 0.
__device__ __forceinline__ int find_work(const int *start, int nwork, int t) {
  int lo = 0, hi = nwork - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (start[mid] <= t) lo = mid; else hi = mid - 1;
  }
  return lo;
}

struct ScoreSmem {
  static __host__ __device__ int pitch(int page_bytes) { return (page_bytes + 127) & ~127; }
  static __host__ __device__ int fk(int F) { return (F + 7) / 8; }   // 8-feature k-steps of the tf32 mma
  // slots [nslots][pitch] | per-warp feature weights [ncw][fk][32 lanes][8 words] | barriers
  static __host__ __device__ size_t bytes(int page_bytes, int F, int ncw, int nslots) {
    return (size_t)nslots * pitch(page_bytes) + (size_t)ncw * fk(F) * 1024 + (size_t)nslots * 8 + 128;
  }
};

// The pages a CTA scores, in order: its tile range [t0, t1) of the plan's tile list covers, for every work item
// (segment) it touches, a run of that segment's pages (the segment's last tile may be short).  v numbers the
// pages of the whole range from 0; the walk only moves forward.
struct PageWalk {
  int wi, v0, cnt;   // current work item, the number of its first page in the range, its pages in the range
  int p0, seg, n;    // that first page's index inside the segment, the segment, its length in pairs
};
__device__ __forceinline__ bool walk_to(const Ctx &c, PageWalk &w, int v, int t0, int t1, int nwork, int tile_pages) {
  while (v >= w.v0 + w.cnt) {
    w.v0 += w.cnt;
    w.cnt = 0;
    if (++w.wi >= nwork) return false;
    const int tbeg = c.tile1_start[w.wi];
    if (tbeg >= t1) return false;
    const int tend = c.tile1_start[w.wi + 1];
    w.seg = c.work[w.wi];
    w.n = c.plan[w.seg].n_old;
    w.p0 = (max(t0, tbeg) - tbeg) * tile_pages;
    w.cnt = max(0, min((min(t1, tend) - tbeg) * tile_pages, (w.n + kPage - 1) / kPage) - w.p0);
  }
  return true;
}

// Scores of the two rows (gid, gid + 8) this lane holds a quarter of: bias, activation, W2 dot, quad reduction.
template <int ACT>
__device__ __forceinline__ void score_rows(const float (&acc)[2][4], const float4 &b1, const float4 &w2, int act,
                                           float (&p)[2]) {
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const float z0 = acc[0][2 * r] + b1.x, z1 = acc[0][2 * r + 1] + b1.y;
    const float z2 = acc[1][2 * r] + b1.z, z3 = acc[1][2 * r + 1] + b1.w;
    float q;
    if (ACT == 0)
      q = fmaxf(z0, 0.f) * w2.x + fmaxf(z1, 0.f) * w2.y + fmaxf(z2, 0.f) * w2.z + fmaxf(z3, 0.f) * w2.w;
    else
      q = activate(z0, act) * w2.x + activate(z1, act) * w2.y + activate(z2, act) * w2.z + activate(z3, act) * w2.w;
    q += __shfl_xor_sync(0xffffffffu, q, 1);
    q += __shfl_xor_sync(0xffffffffu, q, 2);
    p[r] = q;
  }
}

// out[(seg - seg_base) * cap + slot] receives the score of each pair.  nslots = page slots of the ring.
template <int D, int NCW>
__global__ void __launch_bounds__(NCW * 32, 1) k_score(Ctx c, float *out, int seg_base, int nslots) {
  constexpr int KSH = D / 16;        // 16-channel k-steps per tensor (K, then V)
  extern __shared__ __align__(128) uint8_t smem[];
  const int pitch = ScoreSmem::pitch(c.page_bytes);
  float *wsm_all = reinterpret_cast<float *>(smem + (size_t)nslots * pitch);
  const int FK = ScoreSmem::fk(c.F);
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (size_t)nslots * pitch + (size_t)NCW * FK * 1024);  // full[]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  int *group_done = reinterpret_cast<int *>(&bars[nslots]);   // per group of NCW slots: warps that have scored their page
  if (threadIdx.x == 0) {
    for (int s = 0; s < nslots; ++s) mbar_init(smem_u32(&bars[s]), 1);
    fence_barrier_init();
    for (int s = 0; s < nslots / NCW; ++s) group_done[s] = 0;
  }
  __syncthreads();

  const int nwork = c.planhdr[PH_NWORK], total = c.planhdr[PH_TILES1];
  const int per = (total + gridDim.x - 1) / gridDim.x;
  const int t0 = blockIdx.x * per, t1 = min(t0 + per, total);
  if (t0 >= t1) return;
  const int wi0 = find_work(c.tile1_start, nwork, t0) - 1;

  // Page v of the CTA's range lives in ring slot v % nslots and is scored by warp v % NCW; nslots is a multiple
  // of NCW, so a slot always serves the same warp (its barrier carries one phase bit and is never more than one
  // phase ahead of its only waiter).  NCW consecutive pages - a page per warp - are a group, and a group's slots
  // are refilled TOGETHER: a warp that has scored its page counts itself off in the group's counter and goes on
  // to its next page at once; the warp that counts last issues the NCW copies of pages v + nslots, one per lane.
  // Eight consecutive pages asked for at once stream measurably better from HBM than the same copies
  // trickling out as each warp finishes, and no warp ever waits for another.  No "empty" barriers exist.
  PageWalk ahead = {wi0, 0, 0, 0, 0, 0};
  const uint64_t stream_once = l2_policy_evict_first();   // every page passes through L2 exactly once here
  auto fill = [&](int slot_i, int pid, uint32_t tie) {    // one bulk copy: the whole page record
    if (lane == 0) {
      const uint32_t bar = smem_u32(&bars[slot_i]);
      fence_proxy_async();   // the reads of the slot's previous page come before the copy engine's writes
      mbar_arrive_expect_tx(bar, (uint32_t)c.page_bytes);
      bulk_g2s_hint(smem_u32(smem + (size_t)slot_i * pitch) + tie, c.pool + (size_t)pid * c.page_bytes,
                    (uint32_t)c.page_bytes, bar, stream_once);
    }
  };
  for (int v = warp; v < nslots; v += NCW)
    if (walk_to(c, ahead, v, t0, t1, nwork, NCW))
      fill(v, c.pt[(size_t)ahead.seg * c.max_pages + ahead.p0 + (v - ahead.v0)], 0u);
  PageWalk refill = {wi0, 0, 0, 0, 0, 0};   // per lane: lane l (< NCW) looks up page l of the group to refill

  const int gid = lane >> 2, tig = lane & 3;
  // W1 (K rows, then V rows) as mma B fragments, both 8-wide halves of the 16 hidden units.  An fp32 weight is
  // carried as two bf16 values, its rounding (bw) and the rounding of what that left over (bl): the channels
  // are bf16 already, so both products are exact and the weight enters with about 2^-17 relative error.
  uint32_t bw[2 * KSH][4], bl[2 * KSH][4];
  uint4 *wsm = reinterpret_cast<uint4 *>(wsm_all + (size_t)warp * FK * 256);   // feature rows of W1: [FK][lane] x 2 uint4
  float4 b1 = make_float4(0.f, 0.f, 0.f, 0.f), w2 = b1;
  float b2 = 0.f;
  // ldmatrix row address pieces for this lane: matrix mi = lane / 8 covers rows (mi & 1) * 8 .. +8
  // and the low (mi < 2) or high 8 channels of a 16-channel step.
  const int lrow = ((lane >> 3) & 1) * 8 + (lane & 7), lhi = lane >> 4;
  // The scores are read back by the selection kernel right away: keep them in L2, so that no write
  // goes to DRAM in the middle of the read stream.
  const uint64_t keep = l2_policy_evict_last();

  PageWalk cur = {wi0, 0, 0, 0, 0, 0};
  int scorer = -1, seg_held = -1;    // (layer, head) whose weights the warp holds; the segment last seen
  int slot_i = warp, ph = 0;         // ring slot of page v and the parity of its barrier's current phase
  bool gave_up = false;
  for (int v = warp; walk_to(c, cur, v, t0, t1, nwork, NCW); v += NCW) {
    // The pages that will take this group's slots next, one per lane: looked up now by every warp of the group,
    // copied by the one that finishes last.
    const int vq = (v & ~(NCW - 1)) + nslots + (lane & (NCW - 1));
    const int pid_next = walk_to(c, refill, vq, t0, t1, nwork, NCW)
                             ? c.pt[(size_t)refill.seg * c.max_pages + refill.p0 + (vq - refill.v0)] : -1;
    const int seg = cur.seg, n = cur.n, pg = cur.p0 + (v - cur.v0);
    if (seg != seg_held) {           // the divisions below only when the segment changes
      seg_held = seg;
      const int spi = (seg / (c.batch * c.Hkv)) * c.Hkv + seg % c.Hkv;  // (layer, head)
      if (spi != scorer) {
      scorer = spi;
      const uint8_t *sp = c.sp + (size_t)spi * c.sp_stride;
      const uint4 *w = reinterpret_cast<const uint4 *>(sp);
#pragma unroll
      for (int k = 0; k < 2 * KSH; ++k) {
        uint4 x = __ldg(w + k * 32 + lane);
        bw[k][0] = x.x; bw[k][1] = x.y; bw[k][2] = x.z; bw[k][3] = x.w;
        x = __ldg(w + (2 * KSH + k) * 32 + lane);
        bl[k][0] = x.x; bl[k][1] = x.y; bl[k][2] = x.z; bl[k][3] = x.w;
      }
      __syncwarp();
      const uint4 *wf = reinterpret_cast<const uint4 *>(sp + c.sp_off_wf);
      for (int i = lane; i < FK * 64; i += 32) wsm[i] = __ldg(wf + i);
      b1 = __ldg(reinterpret_cast<const float4 *>(sp + c.sp_off_b1) + tig);
      w2 = __ldg(reinterpret_cast<const float4 *>(sp + c.sp_off_w2) + tig);
      b2 = __ldg(reinterpret_cast<const float *>(sp + c.sp_off_b2));
      __syncwarp();
      }
    }
    if (!mbar_wait(smem_u32(&bars[slot_i]), ph)) { set_status(c, kDevWaitTimeout); gave_up = true; break; }
    const uint8_t *page = smem + (size_t)slot_i * pitch;
    const uint32_t kbase = smem_u32(page), vbase = kbase + c.off_v;
    // Eight accumulators (four chains for each half of the hidden units), summed below in a fixed order, so that
    // consecutive mma are independent.  The feature columns come first: x = xt + xr (truncation to tf32 and the
    // remainder, both exact), w = wt + wr likewise (prepared by the host): xt wt + xr wt + xt wr.  This lane's
    // part of the A fragment: rows gid and gid + 8, feature columns 8 ks + tig and + 4.
    float ac[4][2][4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
      for (int h = 0; h < 2; ++h) ac[q][h][0] = ac[q][h][1] = ac[q][h][2] = ac[q][h][3] = 0.f;
    const float *f0 = meta_row(c, page, gid), *f1 = meta_row(c, page, gid + 8);
    for (int ks = 0; ks < FK; ++ks) {
      const int c0 = ks * 8 + tig, c1 = c0 + 4;
      float x[4];
      x[0] = c0 < c.F ? f0[c0] : 0.f; x[1] = c0 < c.F ? f1[c0] : 0.f;   // past F sits the position id: never read as a feature
      x[2] = c1 < c.F ? f0[c1] : 0.f; x[3] = c1 < c.F ? f1[c1] : 0.f;
      uint32_t xt[4], xr[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        xt[i] = __float_as_uint(x[i]) & 0xffffe000u;
        xr[i] = __float_as_uint(x[i] - __uint_as_float(xt[i])) & 0xffffe000u;
      }
      const uint4 wt = wsm[(ks * 32 + lane) * 2], wr = wsm[(ks * 32 + lane) * 2 + 1];
      mma_tf32(ac[0][0], xt[0], xt[1], xt[2], xt[3], wt.x, wt.y);
      mma_tf32(ac[0][1], xt[0], xt[1], xt[2], xt[3], wt.z, wt.w);
      mma_tf32(ac[1][0], xr[0], xr[1], xr[2], xr[3], wt.x, wt.y);
      mma_tf32(ac[1][1], xr[0], xr[1], xr[2], xr[3], wt.z, wt.w);
      mma_tf32(ac[2][0], xt[0], xt[1], xt[2], xt[3], wr.x, wr.y);
      mma_tf32(ac[2][1], xt[0], xt[1], xt[2], xt[3], wr.z, wr.w);
    }
    // K (chains 0: roundings, 1: remainders of the weights) and V (chains 2, 3).
#pragma unroll
    for (int kk = 0; kk < KSH; ++kk) {           // 16-channel step inside K and inside V
      const int ch = kk * 2 + lhi;               // 16-byte chunk this lane addresses
      uint32_t a[4], b[4];
      ldsm_x4(a, kbase + kv_chunk_off(lrow, ch, D));
      ldsm_x4(b, vbase + kv_chunk_off(lrow, ch, D));
      mma_bf16(ac[0][0], a[0], a[1], a[2], a[3], bw[kk][0], bw[kk][1]);
      mma_bf16(ac[0][1], a[0], a[1], a[2], a[3], bw[kk][2], bw[kk][3]);
      mma_bf16(ac[2][0], b[0], b[1], b[2], b[3], bw[KSH + kk][0], bw[KSH + kk][1]);
      mma_bf16(ac[2][1], b[0], b[1], b[2], b[3], bw[KSH + kk][2], bw[KSH + kk][3]);
      mma_bf16(ac[1][0], a[0], a[1], a[2], a[3], bl[kk][0], bl[kk][1]);
      mma_bf16(ac[1][1], a[0], a[1], a[2], a[3], bl[kk][2], bl[kk][3]);
      mma_bf16(ac[3][0], b[0], b[1], b[2], b[3], bl[KSH + kk][0], bl[KSH + kk][1]);
      mma_bf16(ac[3][1], b[0], b[1], b[2], b[3], bl[KSH + kk][2], bl[KSH + kk][3]);
    }
    float acc[2][4];
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[h][i] = (ac[0][h][i] + ac[1][h][i]) + (ac[2][h][i] + ac[3][h][i]);
    float p[2];
    if (c.act == 0) score_rows<0>(acc, b1, w2, 0, p);
    else score_rows<1>(acc, b1, w2, c.act, p);
    // Every lane of a quad holds both sums; lane l < 16 takes the score of row l (from quad l % 8), so
    // the page's sixteen scores leave as one 64-byte store.
    const float lo = __shfl_sync(0xffffffffu, p[0], (lane & 7) * 4), hi = __shfl_sync(0xffffffffu, p[1], (lane & 7) * 4);
    const float mine = lane < 8 ? lo : hi;
    const int slot = pg * kPage + lane;
    if (lane < kPage && slot < n) st_f32_hint(out + (size_t)(seg - seg_base) * c.cap + slot, mine + b2, keep);
    // The slot may be refilled once the count below is seen, and must not be before every read of the page has
    // returned: tie the counter's address to the score, which depends on every value read from the page, through
    // a zero the compiler cannot see through (the grid is one-dimensional).
    __syncwarp();
    const int sg = slot_i / NCW;
    int last = 0;
    if (lane == 0) {
      last = atomicAdd(group_done + sg + (__float_as_uint(mine) & (gridDim.y - 1)), 1) == NCW - 1;
      if (last) group_done[sg] = 0;   // the group's next pages are not even asked for yet: nobody counts before this
    }
    if (__shfl_sync(0xffffffffu, last, 0) && lane < NCW && pid_next >= 0) {
      const int s_ = sg * NCW + lane;
      const uint32_t bar = smem_u32(&bars[s_]);
      fence_proxy_async();   // the reads of the slots' previous pages come before the copy engine's writes
      mbar_arrive_expect_tx(bar, (uint32_t)c.page_bytes);
      bulk_g2s_hint(smem_u32(smem + (size_t)s_ * pitch), c.pool + (size_t)pid_next * c.page_bytes,
                    (uint32_t)c.page_bytes, bar, stream_once);
    }
    slot_i += NCW;
    if (slot_i >= nslots) { slot_i -= nslots; ph ^= 1; }
  }
  // After a wait that ran out the warp leaves early: give the copies it still has in flight (the pages it would
  // have scored next) one more bounded wait each, so that none lands in shared memory the CTA has given up.
  if (gave_up)
    for (int j = 1; j < nslots / NCW; ++j) {
      slot_i += NCW;
      if (slot_i >= nslots) { slot_i -= nslots; ph ^= 1; }
      mbar_wait(smem_u32(&bars[slot_i]), ph);
    }
}

// Baseline scores that need no learned scorer (Appendix E.2): one attention-feature column averaged
// over the g query heads of the KV head - H2O's cumulative attention (column 4), SnapKV's window of
// the final 8 tokens (column 0).  The heads are summed in order and divided by g in fp32.
// grid (work list, tiles of 128 pairs); thread = pair; reads only the meta rows (4F + 4 bytes per pair).
__global__ void __launch_bounds__(128) k_score_feature(Ctx c, float *out, int seg_base, int column) {
  if ((int)blockIdx.x >= c.planhdr[PH_NWORK]) return;
  const int seg = c.work[blockIdx.x];
  const int n = c.plan[seg].n_old;
  const int slot = blockIdx.y * 128 + threadIdx.x;
  if (slot >= n) return;
  const uint8_t *page = c.pool + (size_t)c.pt[(size_t)seg * c.max_pages + slot / kPage] * c.page_bytes;
  const float *f = meta_row(c, page, slot % kPage) + column;
  float acc = 0.f;
  for (int j = 0; j < c.G; ++j) acc = acc + f[j * 6];
  out[(size_t)(seg - seg_base) * c.cap + slot] = acc / (float)c.G;
}

}  // namespace fkv
