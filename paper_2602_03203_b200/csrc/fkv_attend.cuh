// Kernel 4: split-K GQA decode attention over the retained cache (Appendix A):
//     o = sum_{i in S} softmax_i(scale <q, k_i>) v_i,
// the softmax taken over the retained set S only.  The g query heads of a
// group share the KV head, so its K and V are read once for all of them.
//
// Roofline: HBM, 4D bytes per retained pair per token.  grid (splits,
// sequences x KV heads).  A CTA walks a contiguous range of pages: a producer
// warp copies the K|V part of each page record (one contiguous 4D*16-byte
// block) into a shared-memory ring with bulk async copies; PPS consumer warps
// each take one page per stage.  Queries sit on the M axis of the mma (rows
// >= g are zero), keys on N for S = Q K^T, and P V uses ldmatrix.trans on V.
// Softmax is online in fp32 with exp2.  Each CTA leaves an (m, l, O) partial;
// the last CTA of a segment to finish (atomic ticket - nobody waits) merges
// them and writes bf16.
#pragma once
#include "fkv_dev.cuh"

namespace fkv {

struct AttendSmem {
  static __host__ __device__ size_t bytes(int D, int pps, int nst) {
    size_t ring = (size_t)nst * pps * (4 * D * kPage);
    size_t merge = (size_t)pps * 8 * (D + 2) * 4;
    return (ring > merge ? ring : merge) + 128;
  }
};

template <int D, int PPS>
__global__ void __launch_bounds__((PPS + 1) * 32) k_attend(Ctx c, int layer, const __nv_bfloat16 *q,
                                                            __nv_bfloat16 *out, float scale_log2, int min_pages,
                                                            int nst) {
  constexpr int KSQ = D / 16;  // k-steps of Q K^T
  constexpr int NT = D / 8;    // n-tiles of P V
  constexpr int PAGE_KV = 4 * D * kPage;
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ int s_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
  const int y = blockIdx.y, seq = y / c.Hkv, head = y % c.Hkv, G = c.G;
  const int seg = seg_of(c, layer, seq, head);
  const int n = c.len[layer * c.batch + seq];
  const int npages = (n + kPage - 1) / kPage;
  const size_t qrow0 = ((size_t)seq * c.Hkv + head) * G;  // first query head of the group
  if (npages == 0) {
    if (blockIdx.x == 0)
      for (int i = tid; i < G * D; i += blockDim.x) out[qrow0 * D + i] = __float2bfloat16(0.f);
    return;
  }
  int ns = min((int)gridDim.x, (npages + min_pages - 1) / min_pages);
  const int pps_split = (npages + ns - 1) / ns;
  ns = (npages + pps_split - 1) / pps_split;
  if ((int)blockIdx.x >= ns) return;
  const int pg0 = blockIdx.x * pps_split, pg1 = min(npages, pg0 + pps_split);
  const int ntiles = (pg1 - pg0 + PPS - 1) / PPS;

  const size_t ring_bytes = (size_t)nst * PPS * PAGE_KV;
  const size_t merge_bytes = (size_t)PPS * 8 * (D + 2) * 4;
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (ring_bytes > merge_bytes ? ring_bytes : merge_bytes));
  if (tid == 0) {
    for (int s = 0; s < nst; ++s) {
      mbar_init(smem_u32(&bars[s]), 1);
      mbar_init(smem_u32(&bars[nst + s]), PPS);
    }
    fence_barrier_init();
  }
  __syncthreads();

  const int gid = lane >> 2, tig = lane & 3;
  float m_run = -INFINITY, l_run = 0.f;
  float o[NT][4];
  bool failed = false;

  if (warp == PPS) {
    // ---------------- producer ----------------
    const int *ptrow = c.pt + (size_t)seg * c.max_pages;
    for (int it = 0; it < ntiles; ++it) {
      const int s = it % nst, ph = (it / nst) & 1;
      const int p0 = pg0 + it * PPS, np = min(PPS, pg1 - p0);
      const int pid = lane < np ? ptrow[p0 + lane] : 0;
      if (!mbar_wait(smem_u32(&bars[nst + s]), ph ^ 1)) { set_status(c, kDevWaitTimeout); break; }
      if (lane == 0) mbar_arrive_expect_tx(smem_u32(&bars[s]), (uint32_t)(np * PAGE_KV));
      __syncwarp();
      if (lane < np)
        bulk_g2s(smem_u32(smem + ((size_t)s * PPS + lane) * PAGE_KV), c.pool + (size_t)pid * c.page_bytes, PAGE_KV,
                 smem_u32(&bars[s]));
    }
  } else {
    // ---------------- consumers ----------------
#pragma unroll
    for (int i = 0; i < NT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    // Q as A fragments: row gid = query head gid of the group (zero rows beyond g).
    uint32_t qa[KSQ][2];
    {
      const uint32_t *qr = reinterpret_cast<const uint32_t *>(q + (qrow0 + gid) * D);
#pragma unroll
      for (int ks = 0; ks < KSQ; ++ks) {
        qa[ks][0] = gid < G ? qr[ks * 8 + tig] : 0u;
        qa[ks][1] = gid < G ? qr[ks * 8 + 4 + tig] : 0u;
      }
    }
    const int lr = lane & 7, mi = lane >> 3;
    for (int it = 0; it < ntiles; ++it) {
      const int s = it % nst, ph = (it / nst) & 1;
      const int p0 = pg0 + it * PPS, np = min(PPS, pg1 - p0);
      if (!mbar_wait(smem_u32(&bars[s]), ph)) { set_status(c, kDevWaitTimeout); failed = true; break; }
      if (warp < np) {
        const uint32_t kbase = smem_u32(smem + ((size_t)s * PPS + warp) * PAGE_KV), vbase = kbase + 2 * D * kPage;
        float sacc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
        {
          // B fragments of K: matrix mi -> keys (mi >> 1) * 8 .. +8, channels low/high 8 of the step (mi & 1).
          const int krow = (mi >> 1) * 8 + lr;
#pragma unroll
          for (int ks = 0; ks < KSQ; ++ks) {
            uint32_t b[4];
            ldsm_x4(b, kbase + kv_chunk_off(krow, ks * 2 + (mi & 1)));
            mma_bf16(sacc[0], qa[ks][0], 0u, qa[ks][1], 0u, b[0], b[1]);
            mma_bf16(sacc[1], qa[ks][0], 0u, qa[ks][1], 0u, b[2], b[3]);
          }
        }
        // Row gid of S: keys nt*8 + 2*tig + e of this page.
        const int slot0 = (p0 + warp) * kPage;
        float sv[4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int slot = slot0 + nt * 8 + 2 * tig + e;
            sv[nt * 2 + e] = slot < n ? sacc[nt][e] * scale_log2 : -INFINITY;
          }
        float mx = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);  // finite: every page in range has a valid slot
        const float corr = exp2f(m_run - m_new);
        float pv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) pv[i] = exp2f(sv[i] - m_new);
        l_run = l_run * corr + (pv[0] + pv[1]) + (pv[2] + pv[3]);
        m_run = m_new;
        const uint32_t pa0 = pack_bf16(pv[0], pv[1]), pa2 = pack_bf16(pv[2], pv[3]);
#pragma unroll
        for (int i = 0; i < NT; ++i) { o[i][0] *= corr; o[i][1] *= corr; }
        // B fragments of V (transposed load): matrix mi -> keys (mi & 1) * 8 .. +8, channels chunk (mi >> 1).
        const int vrow = (mi & 1) * 8 + lr;
#pragma unroll
        for (int nt2 = 0; nt2 < NT / 2; ++nt2) {
          uint32_t b[4];
          ldsm_x4_trans(b, vbase + kv_chunk_off(vrow, nt2 * 2 + (mi >> 1)));
          mma_bf16(o[2 * nt2], pa0, 0u, pa2, 0u, b[0], b[1]);
          mma_bf16(o[2 * nt2 + 1], pa0, 0u, pa2, 0u, b[2], b[3]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars[nst + s]));
    }
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  }
  (void)failed;
  __syncthreads();  // every issued copy has landed and been consumed: the ring can be reused

  // ---- merge the PPS warps of this CTA: smem [PPS][8][D + 2] ----
  float *mg = reinterpret_cast<float *>(smem);
  if (warp < PPS) {
    float *row = mg + ((size_t)warp * 8 + gid) * (D + 2);
#pragma unroll
    for (int i = 0; i < NT; ++i) {
      row[i * 8 + 2 * tig] = o[i][0];
      row[i * 8 + 2 * tig + 1] = o[i][1];
    }
    if (tig == 0) { row[D] = m_run; row[D + 1] = l_run; }
  }
  __syncthreads();
  float *po = c.part_o + ((size_t)y * kMaxSplits + blockIdx.x) * 8 * D;
  float *pml = c.part_ml + ((size_t)y * kMaxSplits + blockIdx.x) * 8 * 2;
  for (int e = tid; e < G * D; e += blockDim.x) {
    const int r = e / D, ch = e - r * D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < PPS; ++w) M = fmaxf(M, mg[((size_t)w * 8 + r) * (D + 2) + D]);
    float acc = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < PPS; ++w) {
      const float *rw = mg + ((size_t)w * 8 + r) * (D + 2);
      const float f = rw[D] == -INFINITY ? 0.f : exp2f(rw[D] - M);
      acc += f * rw[ch];
      l += f * rw[D + 1];
    }
    if (ns == 1) {
      out[(qrow0 + r) * D + ch] = __float2bfloat16(acc / l);
    } else {
      po[r * D + ch] = acc;
      if (ch == 0) { pml[r * 2] = M; pml[r * 2 + 1] = l; }
    }
  }
  if (ns == 1) return;

  // ---- last CTA of the segment merges the splits ----
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int tk = atomicAdd(&c.tickets[y], 1);
    s_last = tk == ns - 1;
    if (s_last) c.tickets[y] = 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // Weights of the splits per query row: w[r][s] = 2^(m_s - M_r) / sum_s 2^(m_s - M_r) l_s, in shared memory.
  float *s_w = reinterpret_cast<float *>(smem);  // [8][kMaxSplits] m then weights; [8][kMaxSplits] l; ring is idle
  float *s_l = s_w + 8 * kMaxSplits;
  const float *ao = c.part_o + (size_t)y * kMaxSplits * 8 * D;
  const float2 *aml = reinterpret_cast<const float2 *>(c.part_ml + (size_t)y * kMaxSplits * 8 * 2);
  __syncthreads();
  for (int e = tid; e < G * ns; e += blockDim.x) {
    const int r = e / ns, sidx = e - r * ns;
    const float2 ml = __ldcg(aml + sidx * 8 + r);
    s_w[r * kMaxSplits + sidx] = ml.x;
    s_l[r * kMaxSplits + sidx] = ml.y;
  }
  __syncthreads();
  for (int r = warp; r < G; r += PPS + 1) {  // one warp per query row
    float *w = s_w + r * kMaxSplits, *l = s_l + r * kMaxSplits;
    float M = -INFINITY;
    for (int sidx = lane; sidx < ns; sidx += 32) M = fmaxf(M, w[sidx]);
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o2));
    float L = 0.f;
    for (int sidx = lane; sidx < ns; sidx += 32) {
      const float f = exp2f(w[sidx] - M);
      w[sidx] = f;
      L += f * l[sidx];
    }
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o2);
    const float inv = 1.f / L;
    for (int sidx = lane; sidx < ns; sidx += 32) w[sidx] *= inv;
  }
  __syncthreads();
  // Each thread owns 4 consecutive channels of one query row; the loads of 8 splits are in flight together.
  for (int e = tid; e < G * (D / 4); e += blockDim.x) {
    const int r = e / (D / 4), c4 = e - r * (D / 4);
    const float4 *src = reinterpret_cast<const float4 *>(ao + (size_t)r * D) + c4;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s0 = 0; s0 < ns; s0 += 8) {
      float4 x[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        x[u] = s0 + u < ns ? __ldcg(src + (size_t)(s0 + u) * 8 * (D / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float wgt = s0 + u < ns ? s_w[r * kMaxSplits + s0 + u] : 0.f;
        acc.x = fmaf(wgt, x[u].x, acc.x); acc.y = fmaf(wgt, x[u].y, acc.y);
        acc.z = fmaf(wgt, x[u].z, acc.z); acc.w = fmaf(wgt, x[u].w, acc.w);
      }
    }
    __nv_bfloat162 *dst = reinterpret_cast<__nv_bfloat162 *>(out + (qrow0 + r) * D + c4 * 4);
    dst[0] = __floats2bfloat162_rn(acc.x, acc.y);
    dst[1] = __floats2bfloat162_rn(acc.z, acc.w);
  }
}

}  // namespace fkv
