// Kernel 1: the scorer of Appendix B.1,
//     phi_n = sigma(x_n W1 + b1) W2 + b2,   x_n = Concat(k_n, v_n, a_n),
// streamed over every pair of the segments on the work list.
//
// Roofline: HBM.  A pair is 4D + 4F bytes in and 4 bytes out, but 2(2D+F)H
// flops, which is more than the fp32 pipes can do at HBM speed, so the
// [16 pairs x 2D] . [2D x 16] part runs as bf16 mma with fp32 accumulation;
// the F feature columns stay in fp32 FMAs (they are not bf16 data).
//
// Structure: persistent CTAs, one per SM, each a contiguous range of tiles
// (NCW consecutive pages of one segment).  A producer warp brings whole page
// records (16 pairs: K, V, features + positions, one contiguous block) from
// HBM into shared memory with one bulk async copy per page.  Consumer warp w
// takes page w of every tile and owns its own ring of page slots, each slot
// with its own full/empty mbarrier pair, fed by lane w of the producer - the
// warps never wait for one another.  ldmatrix reads the pre-swizzled K and V
// rows as A fragments; the bf16 rows of W1 sit in registers as B fragments
// and the fp32 feature rows in a per-warp shared-memory copy, both reloaded
// when the segment (and so the scorer) changes.
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
  // slots [spw * ncw][pitch] | per-warp feature weights [ncw][F * 16 floats] | barriers
  static __host__ __device__ size_t bytes(int page_bytes, int F, int ncw, int spw) {
    return (size_t)spw * ncw * pitch(page_bytes) + (size_t)ncw * F * 64 + (size_t)spw * ncw * 16 + 128;
  }
};

// Scores of the two rows (gid, gid + 8) this lane holds a quarter of: bias, activation, W2 dot, quad reduction.
template <int ACT>
__device__ __forceinline__ void score_rows(const float (&acc)[2][4], const float (&fz)[2][4], const float4 &b1,
                                           const float4 &w2, int act, float (&p)[2]) {
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const float z0 = acc[0][2 * r] + fz[r][0] + b1.x, z1 = acc[0][2 * r + 1] + fz[r][1] + b1.y;
    const float z2 = acc[1][2 * r] + fz[r][2] + b1.z, z3 = acc[1][2 * r + 1] + fz[r][3] + b1.w;
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

// out[(seg - seg_base) * cap + slot] receives the score of each pair.  spw = page slots per consumer warp.
template <int D, int NCW>
__global__ void __launch_bounds__((NCW + 1) * 32, 1) k_score(Ctx c, float *out, int seg_base, int spw) {
  constexpr int KSH = D / 16;        // 16-channel k-steps per tensor (K, then V)
  extern __shared__ __align__(128) uint8_t smem[];
  const int pitch = ScoreSmem::pitch(c.page_bytes);
  const int nslots = spw * NCW;
  float *wsm_all = reinterpret_cast<float *>(smem + (size_t)nslots * pitch);
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (size_t)nslots * pitch + (size_t)NCW * c.F * 64);  // full[], empty[]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2 * nslots; ++s) mbar_init(smem_u32(&bars[s]), 1);
    fence_barrier_init();
  }
  __syncthreads();

  const int nwork = c.planhdr[PH_NWORK], total = c.planhdr[PH_TILES1];
  const int per = (total + gridDim.x - 1) / gridDim.x;
  const int t0 = blockIdx.x * per, t1 = min(t0 + per, total);
  if (t0 >= t1) return;
  constexpr int TILE = NCW * kPage;
  int wi = find_work(c.tile1_start, nwork, t0);
  // The work item a warp is in: its tiles [tbeg, tend), its segment and length.  Reloaded only on a change.
  int tbeg = 0, tend = -1, seg = 0, n = 0;

  if (warp == NCW) {
    // ---------------- producer: lane w feeds consumer warp w ----------------
    if (lane >= NCW) return;
    int ks = 0, ph = 0;   // this lane's next slot (of its spw) and the phase of that slot's barriers
    auto lookup = [&](int t, int &pid) {   // page of tile t for this lane, or -1
      if (t >= tend) {
        while (t >= c.tile1_start[wi + 1]) ++wi;
        tbeg = c.tile1_start[wi]; tend = c.tile1_start[wi + 1];
        seg = c.work[wi];
        n = c.plan[seg].n_old;
      }
      const int pg = (t - tbeg) * NCW + lane;
      pid = pg * kPage < n ? c.pt[(size_t)seg * c.max_pages + pg] : -1;
    };
    const uint64_t stream_once = l2_policy_evict_first();   // every page passes through L2 exactly once here
    int pid, pid_next = -1;
    lookup(t0, pid);
    for (int t = t0; t < t1; ++t) {
      if (t + 1 < t1) lookup(t + 1, pid_next);   // in flight while this lane waits for its slot
      if (pid >= 0) {
        const int slot = lane + NCW * ks;
        if (!mbar_wait(smem_u32(&bars[nslots + slot]), ph ^ 1)) { set_status(c, kDevWaitTimeout); break; }
        mbar_arrive_expect_tx(smem_u32(&bars[slot]), (uint32_t)c.page_bytes);
        bulk_g2s_hint(smem_u32(smem + (size_t)slot * pitch), c.pool + (size_t)pid * c.page_bytes,
                      (uint32_t)c.page_bytes, smem_u32(&bars[slot]), stream_once);
        if (++ks == spw) { ks = 0; ph ^= 1; }
      }
      pid = pid_next;
    }
    return;
  }

  // ---------------- consumers: warp w owns page w of every tile ----------------
  const int gid = lane >> 2, tig = lane & 3;
  uint32_t bw[2 * KSH][4];  // W1 (K rows, then V rows) as mma B fragments: both 8-wide halves of the 16 hidden units
  float4 *wsm = reinterpret_cast<float4 *>(wsm_all + (size_t)warp * c.F * 16);   // feature rows of W1, [F][4 tig] float4
  float4 b1 = make_float4(0.f, 0.f, 0.f, 0.f), w2 = b1;
  float b2 = 0.f;
  // ldmatrix row address pieces for this lane: matrix mi = lane / 8 covers rows (mi & 1) * 8 .. +8
  // and the low (mi < 2) or high 8 channels of a 16-channel step.
  const int lrow = ((lane >> 3) & 1) * 8 + (lane & 7), lhi = lane >> 4;
  int ks = 0, ph = 0;
  // The scores are read back by the selection kernel right away: keep them in L2, so that no write
  // goes to DRAM in the middle of the read stream.
  const uint64_t keep = l2_policy_evict_last();

  for (int t = t0; t < t1; ++t) {
    if (t >= tend) {
      while (t >= c.tile1_start[wi + 1]) ++wi;
      tbeg = c.tile1_start[wi]; tend = c.tile1_start[wi + 1];
      seg = c.work[wi];
      n = c.plan[seg].n_old;
      const int spi = (seg / (c.batch * c.Hkv)) * c.Hkv + seg % c.Hkv;  // (layer, head)
      const uint8_t *sp = c.sp + (size_t)spi * c.sp_stride;
      const uint4 *w = reinterpret_cast<const uint4 *>(sp);
#pragma unroll
      for (int k = 0; k < 2 * KSH; ++k) {
        uint4 x = __ldg(w + k * 32 + lane);
        bw[k][0] = x.x; bw[k][1] = x.y; bw[k][2] = x.z; bw[k][3] = x.w;
      }
      __syncwarp();
      const float4 *wf = reinterpret_cast<const float4 *>(sp + c.sp_off_wf);
      for (int i = lane; i < c.F * 4; i += 32) wsm[i] = __ldg(wf + i);
      b1 = __ldg(reinterpret_cast<const float4 *>(sp + c.sp_off_b1) + tig);
      w2 = __ldg(reinterpret_cast<const float4 *>(sp + c.sp_off_w2) + tig);
      b2 = __ldg(reinterpret_cast<const float *>(sp + c.sp_off_b2));
      __syncwarp();
    }
    const int tin = t - tbeg;
    if ((tin * NCW + warp) * kPage >= n) continue;   // the segment's last tile may have fewer pages
    const int slot_i = warp + NCW * ks;
    if (!mbar_wait(smem_u32(&bars[slot_i]), ph)) { set_status(c, kDevWaitTimeout); break; }
    const uint8_t *page = smem + (size_t)slot_i * pitch;
    const uint32_t kbase = smem_u32(page), vbase = kbase + c.off_v;
    // Four accumulation chains per half of the hidden units (K / V channels, even / odd k-steps),
    // summed below in a fixed order: a quarter of the dependent-mma depth.
    float ac[4][2][4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
      for (int h = 0; h < 2; ++h) ac[q][h][0] = ac[q][h][1] = ac[q][h][2] = ac[q][h][3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < KSH; ++kk) {           // 16-channel step inside K and inside V
      const int ch = kk * 2 + lhi;               // 16-byte chunk this lane addresses
      uint32_t a[4], b[4];
      ldsm_x4(a, kbase + kv_chunk_off(lrow, ch, D));
      ldsm_x4(b, vbase + kv_chunk_off(lrow, ch, D));
      mma_bf16(ac[kk & 1][0], a[0], a[1], a[2], a[3], bw[kk][0], bw[kk][1]);
      mma_bf16(ac[kk & 1][1], a[0], a[1], a[2], a[3], bw[kk][2], bw[kk][3]);
      mma_bf16(ac[2 + (kk & 1)][0], b[0], b[1], b[2], b[3], bw[KSH + kk][0], bw[KSH + kk][1]);
      mma_bf16(ac[2 + (kk & 1)][1], b[0], b[1], b[2], b[3], bw[KSH + kk][2], bw[KSH + kk][3]);
    }
    float acc[2][4];
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[h][i] = (ac[0][h][i] + ac[1][h][i]) + (ac[2][h][i] + ac[3][h][i]);
    // Feature columns in fp32: this lane owns hidden units {2t, 2t+1, 8+2t, 9+2t} of rows gid and gid+8.
    float fz[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    const float *f0 = meta_row(c, page, gid), *f1 = meta_row(c, page, gid + 8);   // odd word stride: no bank conflicts
    for (int f = 0; f < c.F; f += 6) {   // one query head's six features at a time: all loads, then the FMAs
      float x0[6], x1[6];
      float4 w[6];
#pragma unroll
      for (int j = 0; j < 6; ++j) {
        x0[j] = f0[f + j]; x1[j] = f1[f + j];
        w[j] = wsm[(f + j) * 4 + tig];
      }
#pragma unroll
      for (int j = 0; j < 6; ++j) {
        fz[0][0] = fmaf(x0[j], w[j].x, fz[0][0]); fz[0][1] = fmaf(x0[j], w[j].y, fz[0][1]);
        fz[0][2] = fmaf(x0[j], w[j].z, fz[0][2]); fz[0][3] = fmaf(x0[j], w[j].w, fz[0][3]);
        fz[1][0] = fmaf(x1[j], w[j].x, fz[1][0]); fz[1][1] = fmaf(x1[j], w[j].y, fz[1][1]);
        fz[1][2] = fmaf(x1[j], w[j].z, fz[1][2]); fz[1][3] = fmaf(x1[j], w[j].w, fz[1][3]);
      }
    }
    float p[2];
    if (c.act == 0) score_rows<0>(acc, fz, b1, w2, 0, p);
    else score_rows<1>(acc, fz, b1, w2, c.act, p);
    // Every lane of a quad holds both sums; lane l < 16 takes the score of row l (from quad l % 8), so
    // the page's sixteen scores leave as one 64-byte store.
    const float lo = __shfl_sync(0xffffffffu, p[0], (lane & 7) * 4), hi = __shfl_sync(0xffffffffu, p[1], (lane & 7) * 4);
    const float mine = lane < 8 ? lo : hi;
    const int slot = tin * TILE + warp * kPage + lane;
    if (lane < kPage && slot < n) st_f32_hint(out + (size_t)(seg - seg_base) * c.cap + slot, mine + b2, keep);
    // The slot may be refilled as soon as this arrival is seen: tie it to the score, which depends on every value
    // read from the page, through a zero the compiler cannot see through (the grid is one-dimensional).
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&bars[nslots + slot_i]) + (__float_as_uint(mine) & (gridDim.y - 1)));
    if (++ks == spw) { ks = 0; ph ^= 1; }
  }
}

// Baseline scores that need no learned scorer (Appendix E.2): one attention-feature column averaged
// over the g query heads of the KV head - H2O's cumulative attention (column 4), SnapKV's window of
// the final 8 tokens (column 0).  The heads are summed in order and divided by g in fp32.
// grid (tiles of 128 pairs, work list); thread = pair; reads only the meta rows (4F + 4 bytes per pair).
__global__ void __launch_bounds__(128) k_score_feature(Ctx c, float *out, int seg_base, int column) {
  if ((int)blockIdx.y >= c.planhdr[PH_NWORK]) return;
  const int seg = c.work[blockIdx.y];
  const int n = c.plan[seg].n_old;
  const int slot = blockIdx.x * 128 + threadIdx.x;
  if (slot >= n) return;
  const uint8_t *page = c.pool + (size_t)c.pt[(size_t)seg * c.max_pages + slot / kPage] * c.page_bytes;
  const float *f = meta_row(c, page, slot % kPage) + column;
  float acc = 0.f;
  for (int j = 0; j < c.G; ++j) acc = acc + f[j * 6];
  out[(size_t)(seg - seg_base) * c.cap + slot] = acc / (float)c.G;
}

}  // namespace fkv
