// Kernel 4: split-K GQA decode attention over the retained cache (Appendix A):
//     o = sum_{i in S} softmax_i(scale <q, k_i>) v_i,
// the softmax taken over the retained set S only.  The g query heads of a
// group share the KV head, so its K and V are read once for all of them.
//
// Roofline: HBM, 4D bytes per retained pair per token.
//
// Shape: grid (splits, sequences x KV heads); the `splits` CTAs of a segment
// form ONE thread-block cluster, each walking a contiguous range of pages.
//   - A producer warp copies the K|V part of each page record (one contiguous
//     4D*16-byte block) into a ring of page slots with bulk async copies, one
//     full/empty mbarrier pair per slot.
//   - NCW consumer warps take pages round-robin, each on its own: keys sit on
//     the M axis of the mma (S^T = K Q^T, 16 keys x 8 query columns, columns
//     >= g zero), softmax is online in fp32 with exp2, the two 8 x 8 tiles of
//     P^T are transposed in registers (movmatrix) into the B operand of
//     O^T = V^T P^T, whose A operand comes from ldmatrix.trans on V.
//   - The warps' (m, l, O) are merged in shared memory; every CTA then PUSHES
//     its merged partial, slice by slice, into the shared memory of the CTA
//     that owns that slice of the output (distributed shared memory), one
//     cluster barrier follows, and every CTA reduces and writes its own slice.
//     No partial ever goes to global memory and nobody spins.
//
// The launch can also APPEND the token's new (k, v) pair first (Section 3.1:
// the cache grows by one pair per generated token): the CTA whose page range
// holds slot n writes the row into the page record and patches its own
// shared-memory copy of that page, so the pair is attended in the same launch
// and a decode step is one launch per layer.  The length is bumped by the last
// CTA of the sequence to finish (an atomic ticket), after every CTA has read it.
//
// Launch latency: the split geometry comes from the host (it mirrors the
// lengths), so length, page table and the first copies are in flight together.
// The kernel touches only ITS layer's cache state (length, page table, pages,
// length ticket) and its own q / k / v / out, and it never waits for another
// grid; it signals griddepcontrol.launch_dependents at once.  A decode step
// that has every layer's tensors at hand can therefore launch layer l with the
// programmatic-dependent-launch attribute: its CTAs start as soon as layer
// l-1's CTAs are all running and stream their pages while those still
// compute (a CTA needs under half an SM, so consecutive launches are
// co-resident).  Without the attribute the launch is ordered like any other.
#pragma once
#include "fkv_dev.cuh"

namespace fkv {

constexpr int kMaxSplits = 16;   // CTAs per cluster = splits per segment

struct AttendSmem {
  // ring | slot barriers (512 B) | received slices [kMaxSplits * per] (<= 8 * 128 + 16 floats) | received (m, l)
  static constexpr size_t kBars = 512, kRecvO = (8 * 128 + 4 * kMaxSplits) * 4, kRecvML = kMaxSplits * 8 * 2 * 4;
  static __host__ __device__ size_t ring(int D, int ncw, int slots) {
    const size_t r = (size_t)slots * (4 * D * kPage), merge = (size_t)ncw * 8 * (D + 2) * 4;
    return ((r > merge ? r : merge) + 127) & ~(size_t)127;
  }
  static __host__ __device__ size_t bytes(int D, int ncw, int slots) {
    return ring(D, ncw, slots) + kBars + kRecvO + kRecvML;
  }
};

struct AttendArgs {
  int layer;
  const __nv_bfloat16 *q;   // [batch][Hkv * g][D]
  __nv_bfloat16 *out;       // same
  float scale_log2;         // softmax scale times log2(e)
  int pps;                  // pages per split (>= 1); ceil(pages / pps) <= gridDim.x for every segment
  int append;               // 1: append k_new / v_new at slot n first (and record the query when the cache keeps a history)
  const uint8_t *k_new, *v_new;  // [batch][Hkv][D] bf16
  const int32_t *pos_new;   // [batch] or null (last position + 1)
  unsigned long long seq_mask;   // sequences that append (0 = all)
};

__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// All threads of all CTAs of the cluster: writes made before (also into other CTAs' shared memory) are visible after.
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of this CTA's shared-memory location `local` in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t dsmem_addr(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
__device__ __forceinline__ void dsmem_st(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void dsmem_st2(uint32_t addr, float x, float y) {
  asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(x), "f"(y) : "memory");
}

template <int D, int NCW, int SLOTS>
__global__ void __launch_bounds__((NCW + 1) * 32) k_attend(Ctx c, AttendArgs a) {
  constexpr int KSQ = D / 16;  // k-steps of K Q^T
  constexpr int MT = D / 16;   // m-tiles (16 channels) of O^T = V^T P^T
  constexpr int NCH = D / 8;   // 16-byte chunks per K (or V) row
  constexpr int PAGE_KV = 4 * D * kPage;
  static_assert(2 * NCH <= 32, "one chunk of the new row per lane");
  static_assert(SLOTS <= 32 && 2 * SLOTS * 8 <= (int)AttendSmem::kBars, "one lane of the producer per slot");
  // A slot must always be consumed by the same warp: its barriers carry one parity bit, so a warp
  // waiting for the slot's next page may not run ahead of another warp's wait for the previous one.
  static_assert(SLOTS % NCW == 0, "slot s belongs to consumer warp s % NCW");
  extern __shared__ __align__(128) uint8_t smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
  const int y = blockIdx.y, seq = y / c.Hkv, head = y % c.Hkv, G = c.G;
  const int S = gridDim.x, rank = blockIdx.x;   // the cluster is the grid's x extent
  const int seg = seg_of(c, a.layer, seq, head);
  const int n_old = c.len[a.layer * c.batch + seq];
  const bool app = a.append && (!a.seq_mask || ((a.seq_mask >> seq) & 1ull));
  const int n = n_old + (app ? 1 : 0);
  const int npages = (n + kPage - 1) / kPage;
  const int pg0 = rank * a.pps, pg1 = min(npages, pg0 + a.pps);
  const bool active = pg0 < pg1;
  const int npg = active ? pg1 - pg0 : 0;               // pages of this CTA
  const bool tail = app && active && pg1 == npages;     // this CTA's range holds the new pair
  const bool fresh = tail && (n_old % kPage) == 0;      // ... which opens a new page: nothing to copy for it
  const size_t qrow0 = ((size_t)seq * c.Hkv + head) * G;  // first query head of the group
  // Query record for the attention features: ring slot of this token in the (layer, sequence) history.
  const bool rec = app && c.hist_w > 0;
  const int hcnt = rec ? c.hist_cnt[a.layer * c.batch + seq] : 0;
  const size_t hrow = ((size_t)(a.layer * c.batch + seq) * (rec ? c.hist_w : 1) + (rec ? hcnt % c.hist_w : 0)) * (c.Hkv * G) +
                      (size_t)head * G;   // first query head of the group in the record

  const size_t ring_bytes = AttendSmem::ring(D, NCW, SLOTS);
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + ring_bytes);                      // full[SLOTS], empty[SLOTS]
  float *recv_o = reinterpret_cast<float *>(smem + ring_bytes + AttendSmem::kBars);      // [S][per]: my slice of every partial
  float *recv_ml = reinterpret_cast<float *>(smem + ring_bytes + AttendSmem::kBars + AttendSmem::kRecvO);  // [S][8][2]
  if (tid == 0) {
    griddep_launch();   // nothing here depends on, or is needed by, the next launch of a decode step
    for (int s = 0; s < 2 * SLOTS; ++s) mbar_init(smem_u32(&bars[s]), 1);
    fence_barrier_init();
  }
  __syncthreads();   // every thread has read the length by now (the length bump at the end relies on it)

  const int gid = lane >> 2, tig = lane & 3;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // queries 2 tig and 2 tig + 1
  float o[MT][4];
#pragma unroll
  for (int i = 0; i < MT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

  if (active && warp == NCW) {
    // ---------------- producer: lane l < SLOTS owns slot l and moves pages l, l + SLOTS, ... into it, in order
    // (a slot's barriers carry one parity bit, so its pages must be issued one phase at a time) ----------------
    int *ptrow = c.pt + (size_t)seg * c.max_pages;
    auto issue = [&](int i, int pid) {   // page i of the CTA into slot i % SLOTS
      const uint32_t full = smem_u32(&bars[i % SLOTS]);
      if (fresh && pg0 + i == npages - 1) {
        mbar_arrive(full);               // a brand-new page: the consumer builds it
      } else {
        mbar_arrive_expect_tx(full, PAGE_KV);
        bulk_g2s(smem_u32(smem + (size_t)(i % SLOTS) * PAGE_KV), c.pool + (size_t)pid * c.page_bytes, PAGE_KV, full);
      }
    };
    const bool owner = lane < SLOTS;
    int pid = owner && lane < npg ? ptrow[pg0 + lane] : 0;
    int nxt = owner && lane + SLOTS < npg ? ptrow[pg0 + lane + SLOTS] : 0;
    if (owner && lane < npg) issue(lane, pid);   // the ring is empty: no wait
    __syncwarp();
    if (tail) {
      // The new pair goes to slot n_old of the page record (and, below, into the consumer's copy of the page).
      int npid = -1;
      if (fresh) {
        if (lane == 0) {
          const int old = atomicSub(&c.ctrl[CTRL_FREE_TOP], 1);
          if (old < 1) {
            atomicAdd(&c.ctrl[CTRL_FREE_TOP], 1);
            set_status(c, kDevPoolExhausted);
          } else {
            npid = c.free_stack[old - 1];
            ptrow[npages - 1] = npid;
          }
        }
        npid = __shfl_sync(0xffffffffu, npid, 0);
      } else {
        npid = ptrow[npages - 1];
      }
      if (npid >= 0) {
        int32_t pdef = 0;
        if (!a.pos_new && n_old > 0) {
          const uint8_t *prev = c.pool + (size_t)ptrow[(n_old - 1) / kPage] * c.page_bytes;
          pdef = reinterpret_cast<const int32_t *>(meta_row(c, prev, (n_old - 1) % kPage))[c.F] + 1;
        }
        const size_t row = (size_t)seq * c.Hkv + head;
        move_row<0>(c, c.pool + (size_t)npid * c.page_bytes, n_old % kPage, const_cast<uint8_t *>(a.k_new) + row * D * 2,
                    const_cast<uint8_t *>(a.v_new) + row * D * 2, nullptr,
                    a.pos_new ? const_cast<int32_t *>(a.pos_new) + seq : nullptr, lane, pdef);
      }
      __syncwarp();
    }
    // The pages that did not fit the empty ring: each waits for the previous page of its slot to be consumed.
    if (owner)
      for (int i = lane + SLOTS; i < npg; i += SLOTS) {
        pid = nxt;
        if (i + SLOTS < npg) nxt = ptrow[pg0 + i + SLOTS];
        if (!mbar_wait(smem_u32(&bars[SLOTS + lane]), ((i / SLOTS) & 1) ^ 1)) { set_status(c, kDevWaitTimeout); break; }
        issue(i, pid);
      }
  } else if (active) {
    // ---------------- consumers: warp w takes pages w, w + NCW, ... of this CTA ----------------
    // Q^T as B fragments (channels x queries): column gid = query head gid of the group (zero beyond g).
    uint32_t qb[KSQ][2];
    {
      const uint32_t *qr = reinterpret_cast<const uint32_t *>(a.q + (qrow0 + gid) * D);
#pragma unroll
      for (int ks = 0; ks < KSQ; ++ks) {
        qb[ks][0] = gid < G ? qr[ks * 8 + tig] : 0u;
        qb[ks][1] = gid < G ? qr[ks * 8 + 4 + tig] : 0u;
      }
    }
    // The new pair, one 16-byte chunk per lane (K chunks, then V chunks), for the warp that gets its page.
    const bool mine_new = tail && (npg - 1) % NCW == warp;
    uint4 newrow = make_uint4(0u, 0u, 0u, 0u);
    if (mine_new && lane < 2 * NCH) {
      const size_t row = (size_t)seq * c.Hkv + head;
      const uint8_t *src = (lane < NCH ? a.k_new : a.v_new) + row * D * 2 + (lane % NCH) * 16;
      newrow = *reinterpret_cast<const uint4 *>(src);
    }
    // ldmatrix lane roles.  K (plain): matrix lane/8 -> keys ((lane/8)&1)*8.., channel chunk +lane/16.
    // V (transposed): matrix lane/8 -> keys (lane/16)*8.., channel chunk +(lane/8)&1.
    const int krow = ((lane >> 3) & 1) * 8 + (lane & 7), khi = lane >> 4;
    const int vrow = (lane >> 4) * 8 + (lane & 7), vhi = (lane >> 3) & 1;
    for (int i = warp; i < npg; i += NCW) {
      const int slot_i = i % SLOTS;
      if (!mbar_wait(smem_u32(&bars[slot_i]), (i / SLOTS) & 1)) { set_status(c, kDevWaitTimeout); break; }
      uint8_t *page = smem + (size_t)slot_i * PAGE_KV;
      if (mine_new && i == npg - 1) {
        if (fresh) {   // no copy was issued for a brand-new page: its other rows must still be finite
          for (int j = lane; j < PAGE_KV / 16; j += 32) reinterpret_cast<uint4 *>(page)[j] = make_uint4(0u, 0u, 0u, 0u);
          __syncwarp();
        }
        if (lane < 2 * NCH)
          *reinterpret_cast<uint4 *>(page + (lane < NCH ? 0 : 2 * D) + kv_chunk_off(n_old % kPage, lane % NCH, D)) =
              newrow;
        __syncwarp();
      }
      const uint32_t kbase = smem_u32(page), vbase = kbase + 2 * D;
      // S^T (16 keys x 8 queries) = K (16 x D) Q^T (D x 8): keys on the M axis, two accumulation chains.
      float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int ks = 0; ks < KSQ; ks += 2) {
        uint32_t x[4], z[4];
        ldsm_x4(x, kbase + kv_chunk_off(krow, ks * 2 + khi, D));
        ldsm_x4(z, kbase + kv_chunk_off(krow, ks * 2 + 2 + khi, D));
        mma_bf16(sa, x[0], x[1], x[2], x[3], qb[ks][0], qb[ks][1]);
        mma_bf16(sb, z[0], z[1], z[2], z[3], qb[ks + 1][0], qb[ks + 1][1]);
      }
      // This lane: keys gid and gid + 8 of the page, queries 2 tig and 2 tig + 1.
      const int slot = (pg0 + i) * kPage + gid;
      const bool ok0 = slot < n, ok1 = slot + 8 < n;
      const float v0 = ok0 ? (sa[0] + sb[0]) * a.scale_log2 : -INFINITY, v1 = ok0 ? (sa[1] + sb[1]) * a.scale_log2 : -INFINITY;
      const float v2 = ok1 ? (sa[2] + sb[2]) * a.scale_log2 : -INFINITY, v3 = ok1 ? (sa[3] + sb[3]) * a.scale_log2 : -INFINITY;
      float mx0 = fmaxf(v0, v2), mx1 = fmaxf(v1, v3);
#pragma unroll
      for (int sh = 4; sh < 32; sh <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
      }
      const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);  // finite: slot 0 of a page in range is valid
      const float c0 = exp2f(m_run[0] - mn0), c1 = exp2f(m_run[1] - mn1);
      const float e0 = exp2f(v0 - mn0), e1 = exp2f(v1 - mn1), e2 = exp2f(v2 - mn0), e3 = exp2f(v3 - mn1);
      l_run[0] = l_run[0] * c0 + e0 + e2;
      l_run[1] = l_run[1] * c1 + e1 + e3;
      m_run[0] = mn0; m_run[1] = mn1;
      // P^T as the B operand (keys x queries): transpose the two 8 x 8 bf16 tiles across the warp.
      const uint32_t pb0 = movmatrix_trans(pack_bf16(e0, e1)), pb1 = movmatrix_trans(pack_bf16(e2, e3));
      // O^T (D channels x 8 queries) += V^T (D x 16 keys) P^T (16 x 8)
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        uint32_t x[4];
        ldsm_x4_trans(x, vbase + kv_chunk_off(vrow, mt * 2 + vhi, D));
        o[mt][0] *= c0; o[mt][1] *= c1; o[mt][2] *= c0; o[mt][3] *= c1;
        mma_bf16(o[mt], x[0], x[1], x[2], x[3], pb0, pb1);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars[SLOTS + slot_i]));
    }
#pragma unroll
    for (int sh = 4; sh < 32; sh <<= 1) {
      l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], sh);
      l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], sh);
    }
  }
  __syncthreads();  // every issued copy has landed and been consumed: the ring can be reused

  // ---- merge the consumer warps of this CTA: smem [NCW][8 queries][D + 2] ----
  float *mg = reinterpret_cast<float *>(smem);
  if (active && warp < NCW) {
    float *r0 = mg + ((size_t)warp * 8 + 2 * tig) * (D + 2), *r1 = r0 + (D + 2);
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      r0[mt * 16 + gid] = o[mt][0]; r1[mt * 16 + gid] = o[mt][1];
      r0[mt * 16 + 8 + gid] = o[mt][2]; r1[mt * 16 + 8 + gid] = o[mt][3];
    }
    if (gid == 0) { r0[D] = m_run[0]; r0[D + 1] = l_run[0]; r1[D] = m_run[1]; r1[D + 1] = l_run[1]; }
  }
  __syncthreads();

  // ---- push: element e of the merged partial goes to the CTA that owns e / per (its slot `rank`) ----
  const int per = (G * D + S - 1) / S;   // output elements per owner
  const uint32_t recv_o_s = smem_u32(recv_o), recv_ml_s = smem_u32(recv_ml);
  for (int e = tid; e < G * D; e += blockDim.x) {
    const int r = e / D, ch = e - r * D;
    float acc = 0.f;
    if (active) {
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < NCW; ++w) M = fmaxf(M, mg[((size_t)w * 8 + r) * (D + 2) + D]);
#pragma unroll
      for (int w = 0; w < NCW; ++w) {
        const float *rw = mg + ((size_t)w * 8 + r) * (D + 2);
        acc += (rw[D] == -INFINITY ? 0.f : exp2f(rw[D] - M)) * rw[ch];
      }
    }
    const int owner = e / per;
    dsmem_st(dsmem_addr(recv_o_s + (uint32_t)(rank * per + (e - owner * per)) * 4u, owner), acc);
  }
  for (int e = tid; e < S * G; e += blockDim.x) {   // (m, l) of every query row, to every CTA
    const int owner = e / G, r = e - owner * G;
    float M = -INFINITY, l = 0.f;
    if (active) {
#pragma unroll
      for (int w = 0; w < NCW; ++w) M = fmaxf(M, mg[((size_t)w * 8 + r) * (D + 2) + D]);
#pragma unroll
      for (int w = 0; w < NCW; ++w) {
        const float *rw = mg + ((size_t)w * 8 + r) * (D + 2);
        l += (rw[D] == -INFINITY ? 0.f : exp2f(rw[D] - M)) * rw[D + 1];
      }
    }
    dsmem_st2(dsmem_addr(recv_ml_s + (uint32_t)(rank * 8 + r) * 8u, owner), M, l);
  }
  cluster_sync_all();

  // ---- reduce the slice this CTA owns over the S partials and write it ----
  for (int e = tid; e < per; e += blockDim.x) {
    const int ge = rank * per + e;
    if (ge >= G * D) break;
    const int r = ge / D;
    float M = -INFINITY;
    for (int s = 0; s < S; ++s) M = fmaxf(M, recv_ml[(s * 8 + r) * 2]);
    float acc = 0.f, L = 0.f;
    for (int s = 0; s < S; ++s) {
      const float ms = recv_ml[(s * 8 + r) * 2];
      const float f = ms == -INFINITY ? 0.f : exp2f(ms - M);
      L = fmaf(f, recv_ml[(s * 8 + r) * 2 + 1], L);
      acc = fmaf(f, recv_o[s * per + e], acc);
    }
    a.out[qrow0 * D + ge] = __float2bfloat16(L > 0.f ? acc / L : 0.f);   // an empty sequence gives zeros
    if (rec && ge - r * D == 0) reinterpret_cast<float2 *>(c.hist_ml)[hrow + r] = make_float2(M, L);
  }
  if (rec && rank == 0)   // the queries themselves: G rows of D bf16
    for (int i = tid; i < G * D / 8; i += blockDim.x)
      reinterpret_cast<uint4 *>(c.hist_q + hrow * D * 2)[i] = reinterpret_cast<const uint4 *>(a.q + qrow0 * D)[i];

  // ---- the length grows once every CTA of the sequence (all heads, all splits) has read the old one ----
  if (app && tid == 0) {
    const int total = (int)gridDim.x * c.Hkv;
    int *ticket = &c.seq_tickets[a.layer * c.batch + seq];
    const int tk = atomicAdd(ticket, 1);
    if (tk == total - 1) {
      *ticket = 0;
      c.len[a.layer * c.batch + seq] = n_old + 1;
      if (rec) {
        c.hist_n[(size_t)(a.layer * c.batch + seq) * c.hist_w + hcnt % c.hist_w] = n_old + 1;
        c.hist_cnt[a.layer * c.batch + seq] = hcnt + 1;
      }
    }
  }
}

}  // namespace fkv
