// Kernel 1: the scorer of Appendix B.1,
//     phi_n = sigma(x_n W1 + b1) W2 + b2,   x_n = Concat(k_n, v_n, a_n),
// streamed over every pair of the segments on the work list.
//
// Roofline: HBM.  A pair is 4D + 4F bytes in and 4 bytes out, but 2(2D+F)H
// flops, which is more than the fp32 pipes can do at HBM speed, so the
// [16 pairs x 2D] . [2D x 16] part runs as bf16 mma with fp32 accumulation;
// the F feature columns stay in fp32 FMAs (they are not bf16 data).
//
// Structure: persistent CTAs, one per SM.  A producer warp brings whole page
// records (16 pairs: K, V, features, positions, one contiguous block) from
// HBM into a ring of shared-memory stages with one bulk async copy per page,
// completion counted on an mbarrier.  PPS consumer warps each take one page
// of a stage: ldmatrix reads the pre-swizzled K and V rows as A fragments,
// W1 sits in registers as B fragments for the whole segment.
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
  static __host__ __device__ size_t bytes(int page_bytes, int pps, int nst) {
    return (size_t)nst * pps * pitch(page_bytes) + 128;
  }
};

// out[(seg - seg_base) * cap + slot] receives the score of each pair.
template <int D, int PPS>
__global__ void __launch_bounds__((PPS + 1) * 32, 1) k_score(Ctx c, float *out, int seg_base, int nst) {
  constexpr int KS = 2 * D / 16;     // k-steps over the K and V channels
  constexpr int KSH = D / 16;        // k-steps per tensor
  extern __shared__ __align__(128) uint8_t smem[];
  const int pitch = ScoreSmem::pitch(c.page_bytes);
  const int stage_bytes = PPS * pitch;
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (size_t)nst * stage_bytes);  // full[nst], empty[nst]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  if (threadIdx.x == 0) {
    for (int s = 0; s < nst; ++s) {
      mbar_init(smem_u32(&bars[s]), 1);
      mbar_init(smem_u32(&bars[nst + s]), PPS);
    }
    fence_barrier_init();
  }
  __syncthreads();

  const int nwork = c.planhdr[PH_NWORK], total = c.planhdr[PH_TILES1];
  const int per = (total + gridDim.x - 1) / gridDim.x;
  const int t0 = blockIdx.x * per, t1 = min(t0 + per, total);
  if (t0 >= t1) return;
  constexpr int TILE = PPS * kPage;
  int wi = find_work(c.tile1_start, nwork, t0);

  if (warp == PPS) {
    // ---------------- producer ----------------
    int pid = -1, np = 0;
    auto meta = [&](int t) {
      while (t >= c.tile1_start[wi + 1]) ++wi;
      const int seg = c.work[wi], tin = t - c.tile1_start[wi];
      const int npages = (c.plan[seg].n_old + kPage - 1) / kPage;
      np = min(PPS, npages - tin * PPS);
      pid = lane < np ? c.pt[(size_t)seg * c.max_pages + tin * PPS + lane] : -1;
    };
    meta(t0);
    for (int t = t0, it = 0; t < t1; ++t, ++it) {
      const int s = it % nst, ph = (it / nst) & 1;
      if (!mbar_wait(smem_u32(&bars[nst + s]), ph ^ 1)) { set_status(c, kDevWaitTimeout); break; }
      if (lane == 0) mbar_arrive_expect_tx(smem_u32(&bars[s]), (uint32_t)(np * c.page_bytes));
      __syncwarp();
      if (lane < np)
        bulk_g2s(smem_u32(smem + (size_t)s * stage_bytes + lane * pitch), c.pool + (size_t)pid * c.page_bytes,
                 (uint32_t)c.page_bytes, smem_u32(&bars[s]));
      if (t + 1 < t1) meta(t + 1);
    }
    return;
  }

  // ---------------- consumers: warp w owns page w of every stage ----------------
  const int gid = lane >> 2, tig = lane & 3;
  uint32_t bw[KS][4];  // W1 (K and V rows) as mma B fragments: both 8-wide halves of the 16 hidden units
  const uint8_t *sp = nullptr;
  float4 b1 = make_float4(0.f, 0.f, 0.f, 0.f), w2 = b1;
  float b2 = 0.f;
  // The work item this warp is in: its tiles [tbeg, tend), its segment and length.  Reloaded only on a change.
  int tbeg = 0, tend = -1, seg = 0, n = 0;
  // ldmatrix row address pieces for this lane: matrix mi = lane / 8 covers rows (mi & 1) * 8 .. +8
  // and the low (mi < 2) or high 8 channels of a 16-channel step.
  const int lrow = ((lane >> 3) & 1) * 8 + (lane & 7), lhi = lane >> 4;

  for (int t = t0, it = 0; t < t1; ++t, ++it) {
    const int s = it % nst, ph = (it / nst) & 1;
    if (t >= tend) {
      while (t >= c.tile1_start[wi + 1]) ++wi;
      tbeg = c.tile1_start[wi]; tend = c.tile1_start[wi + 1];
      seg = c.work[wi];
      n = c.plan[seg].n_old;
      const int spi = (seg / (c.batch * c.Hkv)) * c.Hkv + seg % c.Hkv;  // (layer, head)
      sp = c.sp + (size_t)spi * c.sp_stride;
      const uint4 *w = reinterpret_cast<const uint4 *>(sp);
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        uint4 x = __ldg(w + ks * 32 + lane);
        bw[ks][0] = x.x; bw[ks][1] = x.y; bw[ks][2] = x.z; bw[ks][3] = x.w;
      }
      b1 = __ldg(reinterpret_cast<const float4 *>(sp + c.sp_off_b1) + tig);
      w2 = __ldg(reinterpret_cast<const float4 *>(sp + c.sp_off_w2) + tig);
      b2 = __ldg(reinterpret_cast<const float *>(sp + c.sp_off_b2));
    }
    const int tin = t - tbeg;
    const int np = min(PPS, (n + kPage - 1) / kPage - tin * PPS);
    if (!mbar_wait(smem_u32(&bars[s]), ph)) { set_status(c, kDevWaitTimeout); break; }
    if (warp < np) {
      const uint8_t *page = smem + (size_t)s * stage_bytes + warp * pitch;
      const uint32_t kbase = smem_u32(page), vbase = kbase + c.off_v;
      // Two accumulation chains per half of the hidden units (K channels and V channels), summed below
      // in a fixed order: half the dependent-mma depth.
      float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      float acv[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
      for (int kk = 0; kk < KSH; ++kk) {           // 16-channel step inside K and inside V
        const int ch = kk * 2 + lhi;               // 16-byte chunk this lane addresses
        uint32_t a[4], b[4];
        ldsm_x4(a, kbase + kv_chunk_off(lrow, ch));
        ldsm_x4(b, vbase + kv_chunk_off(lrow, ch));
        mma_bf16(acc[0], a[0], a[1], a[2], a[3], bw[kk][0], bw[kk][1]);
        mma_bf16(acc[1], a[0], a[1], a[2], a[3], bw[kk][2], bw[kk][3]);
        mma_bf16(acv[0], b[0], b[1], b[2], b[3], bw[KSH + kk][0], bw[KSH + kk][1]);
        mma_bf16(acv[1], b[0], b[1], b[2], b[3], bw[KSH + kk][2], bw[KSH + kk][3]);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) { acc[0][i] += acv[0][i]; acc[1][i] += acv[1][i]; }
      // Feature columns in fp32: this lane owns hidden units {2t, 2t+1, 8+2t, 9+2t} of rows gid and gid+8.
      float fz[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      const float *f0 = meta_row(c, page, gid), *f1 = meta_row(c, page, gid + 8);   // odd word stride: no bank conflicts
      const float4 *wf = reinterpret_cast<const float4 *>(sp + c.sp_off_wf) + tig;
      for (int f = 0; f < c.F; f += 6) {   // one query head's six features at a time: all loads, then the FMAs
        float x0[6], x1[6];
        float4 w[6];
#pragma unroll
        for (int j = 0; j < 6; ++j) {
          x0[j] = f0[f + j]; x1[j] = f1[f + j];
          w[j] = __ldg(wf + (f + j) * 4);
        }
#pragma unroll
        for (int j = 0; j < 6; ++j) {
          fz[0][0] = fmaf(x0[j], w[j].x, fz[0][0]); fz[0][1] = fmaf(x0[j], w[j].y, fz[0][1]);
          fz[0][2] = fmaf(x0[j], w[j].z, fz[0][2]); fz[0][3] = fmaf(x0[j], w[j].w, fz[0][3]);
          fz[1][0] = fmaf(x1[j], w[j].x, fz[1][0]); fz[1][1] = fmaf(x1[j], w[j].y, fz[1][1]);
          fz[1][2] = fmaf(x1[j], w[j].z, fz[1][2]); fz[1][3] = fmaf(x1[j], w[j].w, fz[1][3]);
        }
      }
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const float z0 = acc[0][2 * r] + fz[r][0] + b1.x, z1 = acc[0][2 * r + 1] + fz[r][1] + b1.y;
        const float z2 = acc[1][2 * r] + fz[r][2] + b1.z, z3 = acc[1][2 * r + 1] + fz[r][3] + b1.w;
        float p = activate(z0, c.act) * w2.x + activate(z1, c.act) * w2.y + activate(z2, c.act) * w2.z +
                  activate(z3, c.act) * w2.w;
        p += __shfl_xor_sync(0xffffffffu, p, 1);
        p += __shfl_xor_sync(0xffffffffu, p, 2);
        const int slot = tin * TILE + warp * kPage + gid + 8 * r;
        if (tig == 0 && slot < n) out[(size_t)(seg - seg_base) * c.cap + slot] = p + b2;
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&bars[nst + s]));
  }
}

}  // namespace fkv
