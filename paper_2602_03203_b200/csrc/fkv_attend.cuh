// Kernel 4: split-K GQA decode attention over the retained cache (Appendix A):
//     o = sum_{i in S} softmax_i(scale <q, k_i>) v_i,
// the softmax taken over the retained set S only.  The g query heads of a
// group share the KV head, so its K and V are read once for all of them.
//
// Roofline: HBM, 4D bytes per retained pair per token.
//
// Shape: grid (splits, sequences x KV heads); each of the `splits` CTAs of a
// segment walks a contiguous range of its pages.
//   - A producer warp copies the K|V part of each page record (one contiguous
//     4D*16-byte block) into a ring of page slots with bulk async copies, one
//     full/empty mbarrier pair per slot.  Pages are issued in page order, NCW
//     at a time, by a converged warp.
//   - NCW consumer warps take pages round-robin, each on its own: keys sit on
//     the M axis of the mma (S^T = K Q^T, 16 keys x 8 query columns, columns
//     >= g zero), softmax is online in fp32 with exp2, the two 8 x 8 tiles of
//     P^T are transposed in registers (movmatrix) into the B operand of
//     O^T = V^T P^T, whose A operand comes from ldmatrix.trans on V.
//   - The warps' (m, l, O) are merged in shared memory and the CTA's partial
//     goes to a small global buffer (it never leaves L2); an arrival counter
//     per segment tells the last CTA to finish, which merges the partials (one
//     round trip to L2, every load in flight at once) and writes the output.
//     A CTA that is not last exits as soon as its partial is out, so its
//     shared memory is free for the next launch.
//   - A launch that runs on its own over few segments (the per-layer entry
//     points at small batch) merges differently: the splits of a segment are
//     one thread-block cluster, every CTA owns a slice of the output and
//     receives that slice of every split's partial in its shared memory
//     (distributed shared memory stores), and after one cluster barrier each
//     CTA reduces and writes its slice.  No partial touches L2.
//
// The launch can also APPEND the token's new (k, v) pair first (Section 3.1:
// the cache grows by one pair per generated token): the CTA whose page range
// holds slot n writes the row into the page record and patches its own
// shared-memory copy of that page, so the pair is attended in the same launch
// and a decode step is one launch per layer.  The length is bumped by the CTA
// of the sequence that takes the last of the atomic tickets every CTA takes
// once it has read the old length (early in the kernel).
//
// Launch latency: the split geometry comes from the host (it mirrors the
// lengths), so length, page table and the first copies are in flight together.
// The kernel touches only ITS layer's cache state (length, page table, pages,
// length ticket) and its own q / k / v / out, and it never waits for another
// grid; it signals griddepcontrol.launch_dependents at once.  A decode step
// that has every layer's tensors at hand can therefore launch layer l with the
// programmatic-dependent-launch attribute: its CTAs start as soon as layer
// l-1's CTAs are all running and stream their pages while those still
// compute (three CTAs fit on an SM, so consecutive launches are co-resident).
// Without the attribute the launch is ordered like any other.  Since such a
// grid starts while the one before it is still running, everything an earlier
// launch may have written (lengths, page tables, free stack, the caller's
// q / k / v) is read with L2-only loads (ld.global.cg), so that no L1 line
// filled earlier can be involved; pages come through the bulk-copy engine,
// which reads L2 as well.
#pragma once
#include "fkv_dev.cuh"

namespace fkv {

constexpr int kMaxSplits = 32;   // splits per segment (one lane of the merging warp per split)
constexpr int kClusterSplits = 16;   // splits per segment when they form one thread-block cluster

struct AttendSmem {
  // ring | slot barriers (512 B)
  static constexpr size_t kBars = 512;
  static __host__ __device__ size_t ring(int D, int ncw, int slots) {
    const size_t r = (size_t)slots * (4 * D * kPage), merge = (size_t)ncw * 8 * (D + 4) * 4;
    return ((r > merge ? r : merge) + 127) & ~(size_t)127;
  }
  // With the cluster merge: this CTA's slice of the output from every split (8 query rows x D floats in all) and
  // every split's statistics (16 splits x 8 rows x (m, l)).
  static __host__ __device__ size_t recv(int D) { return (size_t)8 * D * 4 + (size_t)kClusterSplits * 8 * 8; }
  static __host__ __device__ size_t bytes(int D, int ncw, int slots, bool cluster = false) {
    return ring(D, ncw, slots) + kBars + (cluster ? recv(D) : 0);
  }
};

struct AttendArgs {
  int layer;
  const __nv_bfloat16 *q;   // [batch][Hkv * g][D]
  __nv_bfloat16 *out;       // same
  float scale_log2;         // softmax scale times log2(e)
  int pps;                  // pages per split (>= 1) as the host sees the lengths; the kernel raises it where a segment is longer
  int append;               // 1: append k_new / v_new at slot n first (and record the query when the cache keeps a history)
  const uint8_t *k_new, *v_new;  // [batch][Hkv][D] bf16
  const int32_t *pos_new;   // [batch] or null (last position + 1)
  SeqMask seq_mask;         // sequences that append
  int wait_first;           // 1: the grid was launched with the programmatic attribute but depends on everything
                            // before it: wait for the launch before it ahead of the first global read
};

// The CTA-wide barrier, for the place where the producer warp and the consumer warps meet from different branches.
__device__ __forceinline__ void cta_sync() { asm volatile("bar.sync 0;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// The merge of a segment's split partials, run by the whole CTA that finished last.  part: [nact][G][D + 4] fp32
// (O relative to the partial's own maximum, then m and l); out: G rows of D bf16; scratch: shared memory,
// NW * 8 * D + 16 floats.  One round trip to L2 per pass: warp w asks for partials w, w + NW, ... (PASS of them
// per pass, all query rows, four channels per lane) and, lane s, for the statistics of partial s, before it uses
// any of them.  R = query rows handled (>= G), a compile-time bound that sizes the register arrays.
template <int D, int NW, int R, int PASS>
__device__ __forceinline__ void merge_partials(const float *part, int nact, int G, float *scratch, __nv_bfloat16 *out,
                                               float *hist_mp, int hist_stride) {
  constexpr int PRS = D + 4;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
  float *red = scratch;               // [NW][8][D]: one partial sum per warp
  float *tot = red + NW * 8 * D;      // [8]: 1 / L of every query row
  const bool mine = lane < D / 4;
  float2 st[R];
#pragma unroll
  for (int r = 0; r < R; ++r)
    st[r] = (r < G && lane < nact) ? __ldcg(reinterpret_cast<const float2 *>(part + ((size_t)lane * G + r) * PRS + D))
                                   : make_float2(-INFINITY, 0.f);
  float4 acc[R];
#pragma unroll
  for (int r = 0; r < R; ++r) acc[r] = make_float4(0.f, 0.f, 0.f, 0.f);
  float Mr[R];
  bool have_max = false;
  for (int sp0 = warp; sp0 < nact; sp0 += NW * PASS) {
    float4 x[PASS][R];
#pragma unroll
    for (int k = 0; k < PASS; ++k)
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const int sp = sp0 + k * NW;
        x[k][r] = (mine && r < G && sp < nact)
                      ? __ldcg(reinterpret_cast<const float4 *>(part + ((size_t)sp * G + r) * PRS + lane * 4))
                      : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    if (!have_max) {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float M = st[r].x;
#pragma unroll
        for (int sh = 16; sh >= 1; sh >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, sh));
        Mr[r] = M;
      }
      have_max = true;
    }
#pragma unroll
    for (int k = 0; k < PASS; ++k)
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const int sp = sp0 + k * NW;
        const float ms = __shfl_sync(0xffffffffu, st[r].x, sp & 31);
        const float fs = (sp < nact && ms != -INFINITY) ? exp2f(ms - Mr[r]) : 0.f;
        acc[r].x = fmaf(fs, x[k][r].x, acc[r].x); acc[r].y = fmaf(fs, x[k][r].y, acc[r].y);
        acc[r].z = fmaf(fs, x[k][r].z, acc[r].z); acc[r].w = fmaf(fs, x[k][r].w, acc[r].w);
      }
  }
#pragma unroll
  for (int r = 0; r < R; ++r)
    if (r < G && mine) *reinterpret_cast<float4 *>(red + ((size_t)warp * 8 + r) * D + lane * 4) = acc[r];
  if (warp == NW - 1) {   // the totals of every row: M, then L = sum_s exp2(m_s - M) l_s
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float M = st[r].x;
#pragma unroll
      for (int sh = 16; sh >= 1; sh >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, sh));
      float L = st[r].x == -INFINITY ? 0.f : exp2f(st[r].x - M) * st[r].y;
#pragma unroll
      for (int sh = 16; sh >= 1; sh >>= 1) L += __shfl_xor_sync(0xffffffffu, L, sh);
      if (lane == 0 && r < G) {
        tot[r] = L > 0.f ? 1.f / L : 0.f;   // an empty sequence gives zeros
        if (hist_mp) hist_mp[(size_t)r * hist_stride] = M + log2f(L);
      }
    }
  }
  __syncthreads();
  // Sum over the warps, normalise, write: one thread per four channels of a query row.
  for (int e = tid * 4; e < G * D; e += blockDim.x * 4) {
    const int r = e / D, ch = e - r * D;
    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float4 v = *reinterpret_cast<const float4 *>(red + ((size_t)w * 8 + r) * D + ch);
      sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
    }
    const float inv = tot[r];
    const __nv_bfloat162 p0 = __floats2bfloat162_rn(sum.x * inv, sum.y * inv);
    const __nv_bfloat162 p1 = __floats2bfloat162_rn(sum.z * inv, sum.w * inv);
    uint2 pk;
    pk.x = *reinterpret_cast<const uint32_t *>(&p0);
    pk.y = *reinterpret_cast<const uint32_t *>(&p1);
    *reinterpret_cast<uint2 *>(out + r * D + ch) = pk;
  }
}

// CLUSTER: the splits of a segment (the grid's x extent, a power of two <= kClusterSplits) are one thread-block
// cluster and merge through distributed shared memory instead of global memory: every CTA owns a slice of the
// segment's output, receives that slice of every split's partial, and after one cluster barrier reduces and writes
// it - no partial leaves the SMs and no ticket is taken.  For launches that run on their own (the per-layer entry
// points at small batch), where the merge's round trips to L2 are a sixth of the launch.
template <int D, int NCW, int SLOTS, bool CLUSTER>
__global__ void __launch_bounds__((NCW + 1) * 32, NCW <= 4 ? 3 : 1) k_attend(Ctx c, AttendArgs a) {
  constexpr int KSQ = D / 16;  // k-steps of K Q^T
  constexpr int MT = D / 16;   // m-tiles (16 channels) of O^T = V^T P^T
  constexpr int NCH = D / 8;   // 16-byte chunks per K (or V) row
  constexpr int PAGE_KV = 4 * D * kPage;
  static_assert(2 * NCH <= 32, "one chunk of the new row per lane");
  static_assert(SLOTS <= 32 && 2 * SLOTS * 8 <= (int)AttendSmem::kBars, "the first SLOTS pages are issued one per lane");
  // A slot must always be consumed by the same warp: its barriers carry one parity bit, so a warp
  // waiting for the slot's next page may not run ahead of another warp's wait for the previous one.
  static_assert(SLOTS % NCW == 0, "slot s belongs to consumer warp s % NCW");
  static_assert(32 % NCW == 0, "a group of NCW pages never straddles two 32-entry blocks of page ids");
  extern __shared__ __align__(128) uint8_t smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
  const int y = blockIdx.y, seq = y / c.Hkv, head = y % c.Hkv, G = c.G;
  const int S = gridDim.x, rank = blockIdx.x;   // splits of the segment, and this CTA's
  const int seg = seg_of(c, a.layer, seq, head);
  // A launch that depends on all earlier work (the per-layer entry points: the caller's q, k, v come from the
  // kernel before) still carries the programmatic attribute, so that the grid is scheduled and set up while
  // that kernel drains; it then waits here, before it reads anything, and is ordered like an ordinary launch.
  // (Asking the pages into L2 ahead of the wait was measured and set aside: the early traffic slows the kernel
  // that is still running by more than it saves this one.)
  if (a.wait_first) griddep_wait();
  // Cluster merge: every CTA says "I am running" now and checks, just before it writes into the others' shared
  // memory, that all of them have said so.
  if (CLUSTER && S > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  int *ptrow = c.pt + (size_t)seg * c.max_pages;
  // The producer warp asks for its first page-table entries before the length is known, at the place the host's
  // pages-per-split figure puts them (entries past the segment's pages are never used), so that the two reads
  // overlap instead of following one another.
  int ptv = 0, ptn = 0;
  if (warp == NCW) {
    const int e = rank * a.pps + lane;
    if (e < c.max_pages) ptv = __ldcg(ptrow + e);
    if (e + 32 < c.max_pages) ptn = __ldcg(ptrow + e + 32);
  }
  const int n_old = __ldcg(c.len + a.layer * c.batch + seq);
  // The host refuses an append past the capacity; a replayed launch (CUDA graph) is checked here instead.
  const bool want = a.append && a.seq_mask.has(seq);
  const bool app = want && n_old < c.cap;
  if (want && !app && tid == 0 && rank == 0) set_status(c, kDevCapacity);
  const int n = n_old + (app ? 1 : 0);
  const int npages = (n + kPage - 1) / kPage;
  // Pages per split: the host's figure, or more when the segment has outgrown it since the launch was recorded.
  const int pps = max(a.pps, (npages + S - 1) / S);
  const int pg0 = rank * pps, pg1 = min(npages, pg0 + pps);
  const bool active = pg0 < pg1;
  const int npg = active ? pg1 - pg0 : 0;               // pages of this CTA
  const bool tail = app && active && pg1 == npages;     // this CTA's range holds the new pair
  const bool fresh = tail && (n_old % kPage) == 0;      // ... which opens a new page: nothing to copy for it
  const size_t qrow0 = ((size_t)seq * c.Hkv + head) * G;  // first query head of the group
  // Query record for the attention features: ring slot of this token in the (layer, sequence) history.
  const bool rec = app && c.hist_w > 0;
  const int hcnt = rec ? __ldcg(c.hist_cnt + a.layer * c.batch + seq) : 0;
  const int hslot = rec ? hcnt % c.hist_w : 0;
  const size_t hhead = (size_t)(a.layer * c.batch + seq) * (c.Hkv * G) + (size_t)head * G;   // first query head of the group in the record
  float *hist_mp = rec ? c.hist_mp + hhead * c.hist_wp + hslot : nullptr;                    // its statistic of this token; next head: + hist_wp

  const size_t ring_bytes = AttendSmem::ring(D, NCW, SLOTS);
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + ring_bytes);                      // full[SLOTS], empty[SLOTS]
  const int gid = lane >> 2, tig = lane & 3;
  const uint32_t rt_zero = gridDim.z - 1;   // 0 at run time (the grid is two-dimensional), unknown at compile time
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // queries 2 tig and 2 tig + 1
  float o[MT][4];
#pragma unroll
  for (int i = 0; i < MT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

  // The cache is far larger than L2 and every page is read once per token: mark the pages evict-first so that
  // the small state every launch starts from (lengths, page tables) tends to stay in L2.
  const uint64_t stream_policy = l2_policy_evict_first();
  auto issue = [&](int i, int pid) {   // page i of the CTA into slot i % SLOTS
    const uint32_t full = smem_u32(&bars[i % SLOTS]);
    if (fresh && pg0 + i == npages - 1) {
      mbar_arrive(full);               // a brand-new page: the consumer builds it
    } else {
      mbar_arrive_expect_tx(full, PAGE_KV);
      bulk_g2s_hint(smem_u32(smem + (size_t)(i % SLOTS) * PAGE_KV), c.pool + (size_t)pid * c.page_bytes, PAGE_KV, full,
                    stream_policy);
    }
  };

  if (warp == NCW) {
    // ---------------- producer: page i of the CTA goes to slot i % SLOTS; pages are issued in page order, so a
    // slot's barriers (one parity bit each) see exactly one phase at a time.  The warp sets the barriers up itself
    // and fills the empty ring before it meets the consumers at the CTA barrier. ----------------
    if (lane == 0) {
      for (int s = 0; s < 2 * SLOTS; ++s) mbar_init(smem_u32(&bars[s]), 1);
      fence_barrier_init();
    }
    __syncwarp();
    // ptv / ptn: page ids of the CTA's pages [0, 32) and [32, 64), one per lane.
    if (active && pps != a.pps) {   // the early read looked in the wrong place
      ptv = lane < npg ? __ldcg(ptrow + pg0 + lane) : 0;
      ptn = 32 + lane < npg ? __ldcg(ptrow + pg0 + 32 + lane) : 0;
    }
    if (lane < SLOTS && lane < npg) issue(lane, ptv);         // the ring is empty: no wait
    cta_sync();
  } else {
    if (tid == 0) griddep_launch();   // nothing here depends on, or is needed by, the next launch of a decode step
    cta_sync();                       // the barriers are set up
  }

  // ---- the length grows once every CTA of the sequence (all heads, all splits) has read the old one: a ticket per
  // CTA, taken by the producer warp's first lane as soon as the CTA's part of the append is done (early in the
  // kernel, so that the atomic's round trip is not on the way out); the last ticket moves the length ----
  auto take_length_ticket = [&]() {
    const int total = (int)gridDim.x * c.Hkv, ls = a.layer * c.batch + seq;
    int *ticket = &c.seq_tickets[ls];
    __threadfence();   // this CTA's page-table and failure writes come before its ticket
    const int tk = atomicAdd(ticket, 1);
    if (tk == total - 1) {
      *ticket = 0;
      __threadfence();
      if ((n_old % kPage) == 0 && atomicExch(&c.seq_fail[ls], 0) != 0) {
        // a head found no free page: no head's length moves, the token is not recorded
      } else {
        c.len[ls] = n_old + 1;
        if (rec) {
          c.hist_n[(size_t)ls * c.hist_w + hcnt % c.hist_w] = n_old + 1;
          c.hist_cnt[ls] = hcnt + 1;
        }
      }
    }
  };

  if (active && warp == NCW) {
    if (tail) {
      // The new pair goes to slot n_old of the page record (and, below, into the consumer's copy of the page).
      int npid = -1;
      if (fresh) {
        // A fresh page for this head.  If there is none, the append of the whole sequence is abandoned: the
        // launch's last CTA then leaves the length of every head alone.  Pages that sibling heads did take sit
        // in their page tables past the length, unused; with the pool empty no eviction can run either, so
        // the way on is fkv_reset, which rebuilds the free stack.
        if (lane == 0) {
          const int old = atomicSub(&c.ctrl[CTRL_FREE_TOP], 1);
          if (old < 1) {
            atomicAdd(&c.ctrl[CTRL_FREE_TOP], 1);
            set_status(c, kDevPoolExhausted);
            atomicOr(&c.seq_fail[a.layer * c.batch + seq], 1);
          } else {
            npid = __ldcg(c.free_stack + old - 1);
            ptrow[npages - 1] = npid;
          }
        }
        npid = __shfl_sync(0xffffffffu, npid, 0);
      } else {
        npid = __ldcg(ptrow + npages - 1);
      }
      if (npid >= 0) {
        int32_t pdef = 0;
        if (!a.pos_new && n_old > 0) {
          const uint8_t *prev = c.pool + (size_t)__ldcg(ptrow + (n_old - 1) / kPage) * c.page_bytes;
          pdef = __ldcg(reinterpret_cast<const int32_t *>(meta_row(c, prev, (n_old - 1) % kPage)) + c.F) + 1;
        }
        const size_t row = (size_t)seq * c.Hkv + head;
        move_row<0>(c, c.pool + (size_t)npid * c.page_bytes, n_old % kPage, const_cast<uint8_t *>(a.k_new) + row * D * 2,
                    const_cast<uint8_t *>(a.v_new) + row * D * 2, nullptr,
                    a.pos_new ? const_cast<int32_t *>(a.pos_new) + seq : nullptr, lane, pdef);
      }
      __syncwarp();
    }
    if (app && lane == 0) take_length_ticket();
    __syncwarp();
    // The pages that did not fit the empty ring, in page order and NCW at a time (one page of every consumer warp:
    // their slots come free together).  The whole warp waits, converged, for the previous pages of the group's
    // slots to be consumed; then lanes 0 .. NCW-1 issue one copy each.
    for (int i = SLOTS; i < npg; i += NCW) {
      if ((i & 31) == 0) {
        ptv = ptn;
        ptn = i + 32 + lane < npg ? __ldcg(ptrow + pg0 + i + 32 + lane) : 0;
      }
      const int pid = __shfl_sync(0xffffffffu, ptv, (i + lane) & 31);
      bool ok = true;
#pragma unroll
      for (int j = 0; j < NCW; ++j)
        if (i + j < npg) ok = ok && mbar_wait(smem_u32(&bars[SLOTS + (i + j) % SLOTS]), (((i + j) / SLOTS) & 1) ^ 1);
      if (!__all_sync(0xffffffffu, ok)) {
        if (lane == 0) set_status(c, kDevWaitTimeout);
        break;
      }
      if (lane < NCW && i + lane < npg) issue(i + lane, pid);
    }
  } else if (warp == NCW) {
    if (app && lane == 0) take_length_ticket();   // a CTA without pages still counts
  } else if (active) {
    // ---------------- consumers: warp w takes pages w, w + NCW, ... of this CTA ----------------
    // Q^T as B fragments (channels x queries): column gid = query head gid of the group (zero beyond g).
    uint32_t qb[KSQ][2];
    {
      const uint32_t *qr = reinterpret_cast<const uint32_t *>(a.q + (qrow0 + gid) * D);
#pragma unroll
      for (int ks = 0; ks < KSQ; ++ks) {
        qb[ks][0] = gid < G ? __ldcg(qr + ks * 8 + tig) : 0u;
        qb[ks][1] = gid < G ? __ldcg(qr + ks * 8 + 4 + tig) : 0u;
      }
    }
    // The new pair, one 16-byte chunk per lane (K chunks, then V chunks), for the warp that gets its page.
    const bool mine_new = tail && (npg - 1) % NCW == warp;
    uint4 newrow = make_uint4(0u, 0u, 0u, 0u);
    if (mine_new && lane < 2 * NCH) {
      const size_t row = (size_t)seq * c.Hkv + head;
      const uint8_t *src = (lane < NCH ? a.k_new : a.v_new) + row * D * 2 + (lane % NCH) * 16;
      newrow = __ldcg(reinterpret_cast<const uint4 *>(src));
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
      // The slot may be refilled as soon as the arrival below is seen, so every read of the page has to be
      // complete before it: the barrier's address is made to depend on the results of all the V mma's (whose
      // operands are the last fragments read from the page) through a zero the compiler cannot see through.
      uint32_t done = 0;
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) done |= __float_as_uint(o[mt][0]);
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars[SLOTS + slot_i]) + (done & rt_zero));
    }
#pragma unroll
    for (int sh = 4; sh < 32; sh <<= 1) {
      l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], sh);
      l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], sh);
    }
  }
  __syncthreads();  // every issued copy has landed and been consumed: the ring can be reused

  // ---- merge the consumer warps of this CTA: smem [NCW][8 queries][D + 4] (rows 16-byte aligned) ----
  constexpr int MGS = D + 4;
  float *mg = reinterpret_cast<float *>(smem);
  if (active && warp < NCW) {
    float *r0 = mg + ((size_t)warp * 8 + 2 * tig) * MGS, *r1 = r0 + MGS;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      r0[mt * 16 + gid] = o[mt][0]; r1[mt * 16 + gid] = o[mt][1];
      r0[mt * 16 + 8 + gid] = o[mt][2]; r1[mt * 16 + 8 + gid] = o[mt][3];
    }
    if (gid == 0) { r0[D] = m_run[0]; r0[D + 1] = l_run[0]; r1[D] = m_run[1]; r1[D + 1] = l_run[1]; }
  }
  __syncthreads();

  if (CLUSTER && S > 1) {
    float *recv_o = reinterpret_cast<float *>(smem + ring_bytes + AttendSmem::kBars);   // [S][per]: my slice of every split's O
    float *recv_ml = recv_o + 8 * D;                                                     // [S][8][2]: every split's (m, l)
    // ---- push: elements [o * per, (o + 1) * per) of this CTA's merged partial go to CTA o of the cluster (its
    // slot `rank`), four channels per store; the producer warp sends the (m, l) of every query row to every CTA ----
    const int per = G * D / S;   // output elements per owner: S is a power of two <= 16 and 64 divides G * D
    const uint32_t recv_o_s = smem_u32(recv_o), recv_ml_s = smem_u32(recv_ml);
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");   // every CTA of the cluster has started
    if (warp < NCW) {
      for (int e = tid * 4; e < G * D; e += NCW * 32 * 4) {
        const int r = e / D, ch = e - r * D;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (active) {
          float mw[NCW], M = -INFINITY;
#pragma unroll
          for (int w = 0; w < NCW; ++w) {
            mw[w] = mg[((size_t)w * 8 + r) * MGS + D];
            M = fmaxf(M, mw[w]);
          }
#pragma unroll
          for (int w = 0; w < NCW; ++w) {
            const float f = mw[w] == -INFINITY ? 0.f : exp2f(mw[w] - M);
            const float4 x = *reinterpret_cast<const float4 *>(mg + ((size_t)w * 8 + r) * MGS + ch);
            acc.x = fmaf(f, x.x, acc.x); acc.y = fmaf(f, x.y, acc.y);
            acc.z = fmaf(f, x.z, acc.z); acc.w = fmaf(f, x.w, acc.w);
          }
        }
        const int owner = e / per;
        dsmem_st4(dsmem_addr(recv_o_s + (uint32_t)(rank * per + (e - owner * per)) * 4u, owner), acc);
      }
    } else {
      for (int e = lane; e < S * G; e += 32) {
        const int owner = e / G, r = e - owner * G;
        float M = -INFINITY, l = 0.f;
        if (active) {
#pragma unroll
          for (int w = 0; w < NCW; ++w) M = fmaxf(M, mg[((size_t)w * 8 + r) * MGS + D]);
#pragma unroll
          for (int w = 0; w < NCW; ++w) {
            const float *rw = mg + ((size_t)w * 8 + r) * MGS;
            l += (rw[D] == -INFINITY ? 0.f : exp2f(rw[D] - M)) * rw[D + 1];
          }
        }
        dsmem_st2(dsmem_addr(recv_ml_s + (uint32_t)(rank * 8 + r) * 8u, owner), M, l);
      }
    }
    cluster_sync_all();
    // ---- reduce the slice this CTA owns, [rank * per, (rank + 1) * per), over the S partials and write it: one
    // warp per query row of the slice; lane s holds the statistics of partial s; the lanes form 4 groups that each
    // sum every fourth partial for 8 x 4 channels, and the groups are added with shuffles ----
    const int lo = rank * per, hi = lo + per;
    for (int r = lo / D + warp; r * D < hi; r += NCW + 1) {
      const int e0 = max(lo, r * D), e1 = min(hi, (r + 1) * D);
      const float ms = lane < S ? recv_ml[(lane * 8 + r) * 2] : -INFINITY;
      const float ls = lane < S ? recv_ml[(lane * 8 + r) * 2 + 1] : 0.f;
      float M = ms;
#pragma unroll
      for (int sh = 16; sh >= 1; sh >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, sh));
      const float f = ms == -INFINITY ? 0.f : exp2f(ms - M);
      float L = f * ls;
#pragma unroll
      for (int sh = 16; sh >= 1; sh >>= 1) L += __shfl_xor_sync(0xffffffffu, L, sh);
      const float inv = L > 0.f ? 1.f / L : 0.f;   // an empty sequence gives zeros
      const int grp = lane >> 3, l8 = lane & 7;
      for (int base = e0; base < e1; base += 32) {
        const int e = base + l8 * 4;
        const bool valid = e < e1;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int k = 0; k < kClusterSplits / 4; ++k) {
          const int sp = grp + 4 * k;
          const float fs = __shfl_sync(0xffffffffu, f, sp);
          if (sp < S && valid) {
            const float4 x = *reinterpret_cast<const float4 *>(recv_o + sp * per + (e - lo));
            acc.x = fmaf(fs, x.x, acc.x); acc.y = fmaf(fs, x.y, acc.y);
            acc.z = fmaf(fs, x.z, acc.z); acc.w = fmaf(fs, x.w, acc.w);
          }
        }
#pragma unroll
        for (int sh = 8; sh <= 16; sh <<= 1) {
          acc.x += __shfl_xor_sync(0xffffffffu, acc.x, sh); acc.y += __shfl_xor_sync(0xffffffffu, acc.y, sh);
          acc.z += __shfl_xor_sync(0xffffffffu, acc.z, sh); acc.w += __shfl_xor_sync(0xffffffffu, acc.w, sh);
        }
        if (grp == 0 && valid) {
          const __nv_bfloat162 p0 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
          const __nv_bfloat162 p1 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
          uint2 pk;
          pk.x = *reinterpret_cast<const uint32_t *>(&p0);
          pk.y = *reinterpret_cast<const uint32_t *>(&p1);
          *reinterpret_cast<uint2 *>(a.out + qrow0 * D + e) = pk;
        }
      }
      if (rec && e0 == r * D && lane == 0) hist_mp[(size_t)r * c.hist_wp] = M + log2f(L);
    }
  } else if (S == 1) {
    // ---- one CTA holds the whole segment (many segments per launch, or a short one): normalise and write the
    // output straight from the warps' partials; nothing goes through global memory and no ticket is taken ----
    if (warp < NCW) {
      for (int e = tid * 4; e < G * D; e += NCW * 32 * 4) {
        const int r = e / D, ch = e - r * D;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float M = -INFINITY, Lr = 0.f;
        if (active) {
          float mw[NCW];
#pragma unroll
          for (int w = 0; w < NCW; ++w) {
            mw[w] = mg[((size_t)w * 8 + r) * MGS + D];
            M = fmaxf(M, mw[w]);
          }
#pragma unroll
          for (int w = 0; w < NCW; ++w) {
            const float f = mw[w] == -INFINITY ? 0.f : exp2f(mw[w] - M);
            const float *rw = mg + ((size_t)w * 8 + r) * MGS;
            const float4 x = *reinterpret_cast<const float4 *>(rw + ch);
            acc.x = fmaf(f, x.x, acc.x); acc.y = fmaf(f, x.y, acc.y);
            acc.z = fmaf(f, x.z, acc.z); acc.w = fmaf(f, x.w, acc.w);
            Lr = fmaf(f, rw[D + 1], Lr);
          }
        }
        const float inv = Lr > 0.f ? 1.f / Lr : 0.f;   // an empty sequence gives zeros
        const __nv_bfloat162 p0 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
        const __nv_bfloat162 p1 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
        uint2 pk;
        pk.x = *reinterpret_cast<const uint32_t *>(&p0);
        pk.y = *reinterpret_cast<const uint32_t *>(&p1);
        *reinterpret_cast<uint2 *>(a.out + (qrow0 + r) * D + ch) = pk;
        if (rec && ch == 0) hist_mp[(size_t)r * c.hist_wp] = M + log2f(Lr);
      }
    }
  } else {
    // ---- this CTA's partial, relative to its own maximum, goes to global memory (it stays in L2): per query row
    // D floats of O, then m and l ----
    constexpr int PRS = D + 4;   // floats per row of a partial record
    float *seg_part = c.att_part + (size_t)seg * c.att_smax * G * PRS;
    if (active) {
      float *part = seg_part + (size_t)rank * G * PRS;
      if (warp < NCW) {
        for (int e = tid * 4; e < G * D; e += NCW * 32 * 4) {
          const int r = e / D, ch = e - r * D;
          float mw[NCW], M = -INFINITY;
  #pragma unroll
          for (int w = 0; w < NCW; ++w) {
            mw[w] = mg[((size_t)w * 8 + r) * MGS + D];
            M = fmaxf(M, mw[w]);
          }
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  #pragma unroll
          for (int w = 0; w < NCW; ++w) {
            const float f = mw[w] == -INFINITY ? 0.f : exp2f(mw[w] - M);
            const float4 x = *reinterpret_cast<const float4 *>(mg + ((size_t)w * 8 + r) * MGS + ch);
            acc.x = fmaf(f, x.x, acc.x); acc.y = fmaf(f, x.y, acc.y);
            acc.z = fmaf(f, x.z, acc.z); acc.w = fmaf(f, x.w, acc.w);
          }
          __stcg(reinterpret_cast<float4 *>(part + r * PRS + ch), acc);
        }
      } else if (lane < G) {
        const int r = lane;
        float M = -INFINITY, l = 0.f;
  #pragma unroll
        for (int w = 0; w < NCW; ++w) M = fmaxf(M, mg[((size_t)w * 8 + r) * MGS + D]);
  #pragma unroll
        for (int w = 0; w < NCW; ++w) {
          const float *rw = mg + ((size_t)w * 8 + r) * MGS;
          l += (rw[D] == -INFINITY ? 0.f : exp2f(rw[D] - M)) * rw[D + 1];
        }
        __stcg(reinterpret_cast<float2 *>(part + r * PRS + D), make_float2(M, l));
      }
    }
    // ---- the last CTA of the segment to get here merges the partials and writes the output ----
    __shared__ int s_last;
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      const int tk = atomicAdd(&c.att_tickets[seg], 1);
      s_last = tk == S - 1;
      if (tk == S - 1) c.att_tickets[seg] = 0;
    }
    __syncthreads();
    if (s_last) {
      __threadfence();
      const int nact = min(S, (npages + pps - 1) / pps);   // CTAs that had pages (the first nact)
      if (G <= 4)
        merge_partials<D, NCW + 1, 4, 4>(seg_part, nact, G, reinterpret_cast<float *>(smem), a.out + qrow0 * D, hist_mp, c.hist_wp);
      else
        merge_partials<D, NCW + 1, 8, 1>(seg_part, nact, G, reinterpret_cast<float *>(smem), a.out + qrow0 * D, hist_mp, c.hist_wp);
    }
  }
  if (rec && rank == 0)   // the queries themselves: G rows of D bf16, laid out as the feature kernel's operand tile
    for (int i = tid; i < G * D / 8; i += blockDim.x) {
      const int r = i / (D / 8), ch = i % (D / 8);
      *reinterpret_cast<uint4 *>(c.hist_q + hist_q_off(hhead + r, ch, hslot, c.hist_wp, D)) =
          __ldcg(reinterpret_cast<const uint4 *>(a.q + qrow0 * D) + i);
    }

  // A launch with the programmatic attribute starts without waiting for the launch before it; it must not be
  // COMPLETE before that one is, or whatever is ordered after this grid (the next decode step, an eviction, the end
  // of a recorded graph) would not be ordered after the whole chain.  One thread of the grid waits for the
  // launch before (all its own work is done by now; without the attribute this returns at once); every other CTA
  // leaves and frees its SM.
  if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0) griddep_wait();
}

}  // namespace fkv
