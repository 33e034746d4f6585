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
//
// The launch can also APPEND the token's new (k, v) pair first (Section 3.1:
// the cache grows by one pair per generated token): the CTA whose page range
// holds slot n writes the row into the page record and patches its own
// shared-memory copy of that page, so the pair is attended in the same launch
// and a decode step is one launch per layer.  The length is bumped by the last
// CTA of the sequence to finish (a second ticket), after every CTA has read it.
//
// Launch latency: the split geometry comes from the host (it mirrors the
// lengths), so length, page table and the first copies are in flight together.
// When the launch carries the programmatic-dependent-launch attribute, all of
// that - it touches only this layer's own cache state - runs before
// griddepcontrol.wait, i.e. while the previous layer's launch is still
// merging; queries, the new pair, scratch and outputs are touched after it.
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

struct AttendArgs {
  int layer;
  const __nv_bfloat16 *q;   // [batch][Hkv * g][D]
  __nv_bfloat16 *out;       // same
  float scale_log2;         // softmax scale times log2(e)
  int pps;                  // pages per split (>= 1); ceil(pages / pps) <= min(gridDim.x, kMaxSplits) for every segment
  int nst;                  // ring stages
  int append;               // 1: append k_new / v_new at slot n first
  const uint8_t *k_new, *v_new;  // [batch][Hkv][D] bf16
  const int32_t *pos_new;   // [batch] or null (last position + 1)
  unsigned long long seq_mask;   // sequences that append (0 = all)
};

__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <int D, int PPS>
__global__ void __launch_bounds__((PPS + 1) * 32) k_attend(Ctx c, AttendArgs a) {
  constexpr int KSQ = D / 16;  // k-steps of Q K^T
  constexpr int NT = D / 8;    // n-tiles of P V
  constexpr int NCH = D / 8;   // 16-byte chunks per K (or V) row
  constexpr int PAGE_KV = 4 * D * kPage;
  static_assert(2 * NCH <= 32, "one chunk of the new row per lane");
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ int s_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
  const int y = blockIdx.y, seq = y / c.Hkv, head = y % c.Hkv, G = c.G, nst = a.nst;
  const int seg = seg_of(c, a.layer, seq, head);
  // This layer's own state: nothing the previous launch of a decode step writes.
  const int n_old = c.len[a.layer * c.batch + seq];
  const bool app = a.append && (!a.seq_mask || ((a.seq_mask >> seq) & 1ull));
  const int n = n_old + (app ? 1 : 0);
  const int npages = (n + kPage - 1) / kPage;
  const int ns = (npages + a.pps - 1) / a.pps;
  const int pg0 = blockIdx.x * a.pps, pg1 = min(npages, pg0 + a.pps);
  const bool active = pg0 < pg1;
  const bool tail = app && active && pg1 == npages;   // this CTA's range holds the new pair
  const bool fresh = tail && (n_old % kPage) == 0;    // ... which opens a new page: nothing to copy for it
  const int ntiles = active ? (pg1 - pg0 + PPS - 1) / PPS : 0;
  const size_t qrow0 = ((size_t)seq * c.Hkv + head) * G;  // first query head of the group
  __nv_bfloat16 *out = a.out;

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
  __syncthreads();   // every thread has read the length by now (the length bump at the end relies on it)

  const int gid = lane >> 2, tig = lane & 3;
  float m_run = -INFINITY, l_run = 0.f;
  float o[NT][4];
  bool last = false;   // this CTA merges the splits of its segment

  if (!active) {
    griddep_wait();
    if (npages == 0 && blockIdx.x == 0)
      for (int i = tid; i < G * D; i += blockDim.x) out[qrow0 * D + i] = __float2bfloat16(0.f);
  } else {
    if (warp == PPS) {
      // ---------------- producer ----------------
      int *ptrow = c.pt + (size_t)seg * c.max_pages;
      bool ok = true;
      auto issue = [&](int it) {
        const int s = it % nst, ph = (it / nst) & 1;
        const int p0 = pg0 + it * PPS, np = min(PPS, pg1 - p0);
        const int ncopy = np - ((fresh && p0 + np == npages) ? 1 : 0);
        const int pid = lane < ncopy ? ptrow[p0 + lane] : 0;
        if (!mbar_wait(smem_u32(&bars[nst + s]), ph ^ 1)) { set_status(c, kDevWaitTimeout); ok = false; return; }
        if (lane == 0) mbar_arrive_expect_tx(smem_u32(&bars[s]), (uint32_t)(ncopy * PAGE_KV));
        __syncwarp();
        if (lane < ncopy)
          bulk_g2s(smem_u32(smem + ((size_t)s * PPS + lane) * PAGE_KV), c.pool + (size_t)pid * c.page_bytes, PAGE_KV,
                   smem_u32(&bars[s]));
      };
      int it = 0;
      for (; it < min(ntiles, nst) && ok; ++it) issue(it);   // the ring is empty: none of these waits
      griddep_wait();
      if (lane == 0) griddep_launch();
      if (tail) {
        // The new pair goes to slot n_old of the page record (and, below, into the consumers' copy of the page).
        int pid = -1;
        if (fresh) {
          if (lane == 0) {
            const int old = atomicSub(&c.ctrl[CTRL_FREE_TOP], 1);
            if (old < 1) {
              atomicAdd(&c.ctrl[CTRL_FREE_TOP], 1);
              set_status(c, kDevPoolExhausted);
            } else {
              pid = c.free_stack[old - 1];
              ptrow[npages - 1] = pid;
            }
          }
          pid = __shfl_sync(0xffffffffu, pid, 0);
        } else {
          pid = ptrow[npages - 1];
        }
        if (pid >= 0) {
          int32_t pdef = 0;
          if (!a.pos_new && n_old > 0) {
            const uint8_t *prev = c.pool + (size_t)ptrow[(n_old - 1) / kPage] * c.page_bytes;
            pdef = reinterpret_cast<const int32_t *>(prev + c.off_p)[(n_old - 1) % kPage] + 1;
          }
          const size_t row = (size_t)seq * c.Hkv + head;
          move_row<0>(c, c.pool + (size_t)pid * c.page_bytes, n_old % kPage, const_cast<uint8_t *>(a.k_new) + row * D * 2,
                      const_cast<uint8_t *>(a.v_new) + row * D * 2, nullptr,
                      a.pos_new ? const_cast<int32_t *>(a.pos_new) + seq : nullptr, lane, pdef);
        }
      }
      for (; it < ntiles && ok; ++it) issue(it);
    } else {
      // ---------------- consumers ----------------
      griddep_wait();
#pragma unroll
      for (int i = 0; i < NT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
      // Q as A fragments: row gid = query head gid of the group (zero rows beyond g).
      uint32_t qa[KSQ][2];
      {
        const uint32_t *qr = reinterpret_cast<const uint32_t *>(a.q + (qrow0 + gid) * D);
#pragma unroll
        for (int ks = 0; ks < KSQ; ++ks) {
          qa[ks][0] = gid < G ? qr[ks * 8 + tig] : 0u;
          qa[ks][1] = gid < G ? qr[ks * 8 + 4 + tig] : 0u;
        }
      }
      // The new pair, one 16-byte chunk per lane (K chunks, then V chunks), for the warp that gets its page.
      uint4 newrow = make_uint4(0u, 0u, 0u, 0u);
      if (tail && lane < 2 * NCH) {
        const size_t row = (size_t)seq * c.Hkv + head;
        const uint8_t *src = (lane < NCH ? a.k_new : a.v_new) + row * D * 2 + (lane % NCH) * 16;
        newrow = *reinterpret_cast<const uint4 *>(src);
      }
      const int lr = lane & 7, mi = lane >> 3;
      for (int it = 0; it < ntiles; ++it) {
        const int s = it % nst, ph = (it / nst) & 1;
        const int p0 = pg0 + it * PPS, np = min(PPS, pg1 - p0);
        if (!mbar_wait(smem_u32(&bars[s]), ph)) { set_status(c, kDevWaitTimeout); break; }
        if (warp < np) {
          uint8_t *page = smem + ((size_t)s * PPS + warp) * PAGE_KV;
          if (tail && p0 + warp == npages - 1) {
            if (fresh) {   // no copy was issued for a brand-new page: its other rows must still be finite
              for (int i = lane; i < PAGE_KV / 16; i += 32) reinterpret_cast<uint4 *>(page)[i] = make_uint4(0u, 0u, 0u, 0u);
              __syncwarp();
            }
            if (lane < 2 * NCH)
              *reinterpret_cast<uint4 *>(page + (lane < NCH ? 0 : 2 * D * kPage) + kv_chunk_off(n_old % kPage, lane % NCH)) =
                  newrow;
            __syncwarp();
          }
          const uint32_t kbase = smem_u32(page), vbase = kbase + 2 * D * kPage;
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
              sv[nt * 2 + e] = slot < n ? sacc[nt][e] * a.scale_log2 : -INFINITY;
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
    if (ns > 1) {
      // ---- the last CTA of the segment to get here merges the splits ----
      __threadfence();
      __syncthreads();
      if (tid == 0) {
        const int tk = atomicAdd(&c.tickets[y], 1);
        s_last = tk == ns - 1;
        if (s_last) c.tickets[y] = 0;
      }
      __syncthreads();
      last = s_last != 0;
    }
  }

  if (last) {
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

  // ---- the length grows once every CTA of the sequence (all heads, all splits) has read the old one ----
  if (app && tid == 0) {
    const int total = (int)gridDim.x * c.Hkv;
    const int tk = atomicAdd(&c.seq_tickets[seq], 1);
    if (tk == total - 1) {
      c.seq_tickets[seq] = 0;
      c.len[a.layer * c.batch + seq] = n_old + 1;
    }
  }
}

}  // namespace fkv
