// Shared device-side definitions: the cache context handed to every kernel,
// the page-record layout, and thin wrappers over the PTX this library uses
// (mbarrier, bulk async copy, ldmatrix, bf16 mma).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace fkv {

constexpr int kPage = 16;        // pairs per page
constexpr int kHidden = 16;      // scorer hidden width (Section 4.1)

// Device status bits (mirrors include/fkv.h).
constexpr unsigned kDevPoolExhausted = 1u, kDevCapacity = 2u, kDevWaitTimeout = 4u, kDevBadIndex = 8u;

// ctrl[] slots
enum { CTRL_FREE_TOP = 0, CTRL_STATUS = 1, CTRL_WORDS = 8 };
// planhdr[] slots
enum { PH_NWORK = 0, PH_TILES1 = 1, PH_NEW_PAGES = 2, PH_OLD_PAGES = 3, PH_PUSH_START = 4, PH_WORDS = 8 };

// What the plan kernel decides for one segment of the current call.
struct SegPlan {
  int n_old;   // pairs before
  int n_new;   // pairs after (== n_old when the segment is left alone)
  int r;       // protected recent pairs
  int k_sel;   // pairs to select among slots [0, n_old - r)
  int active;  // 1 if the segment is compacted in this call
  int push_base;  // offset of its old pages in the push region of the free stack
  int pad0, pad1;
};

// One page record holds 16 pairs of one segment:
//   kv   [16][K row (D bf16) | V row (D bf16)]: a pair's key and value are one contiguous 4D-byte run
//        (a gather of the pair reads one place); the 16-byte chunks of every 128-byte span are
//        XOR-swizzled by the row index
//   meta [16][F + 1] 32-bit words: the pair's F fp32 attention features, then its
//        original token position (int32) - one contiguous run per pair, so a
//        gather of the pair touches one place for both
// The swizzle (chunk c of row r sits at chunk c ^ (r & 7)) is the 128-byte
// shared-memory swizzle, applied in HBM so that ONE bulk copy of the record
// lands in shared memory ready for conflict-free ldmatrix (rows are a
// multiple of 128 bytes apart).
struct Ctx {
  int L, Hkv, G, D, batch, act, R, F;
  int cap;        // segment capacity in pairs (multiple of 16)
  int max_pages;  // cap / 16
  int num_pages;
  int page_bytes, off_v, off_f;  // off_f: start of the meta rows (F + 1 words each)
  int sp_stride, sp_off_wf, sp_off_b1, sp_off_w2, sp_off_b2;
  uint8_t *pool;
  int *free_stack;
  int *ctrl;
  int *pt, *pt_new;  // [L][batch][Hkv][max_pages]
  int *len;          // [L][batch]
  int *budget;       // [batch]
  uint8_t *sp;       // scorer blocks [L][Hkv]
  float *scores;     // [L][batch][Hkv][cap]
  int *idx;          // [L][batch][Hkv][cap]
  SegPlan *plan;     // [L*batch*Hkv]
  int *work;         // work list of segment ids
  int *tile1_start;  // prefix of score tiles over the work list
  int *planhdr;
  int *seq_tickets;  // [L][batch]
  int *seq_fail;     // [L][batch]: set by a head whose append found no free page; read and cleared by the launch's last CTA
  // Split-K attention: partial results [L*batch*Hkv][att_smax][G][D + 4] fp32 and one arrival counter per segment.
  float *att_part;
  int *att_tickets;
  int att_smax;
  // Record of the decode queries of the current chunk (attention-feature maintenance; hist_w = 0: off).
  int hist_w;          // ring capacity W in queries
  int hist_wp;         // W rounded up to a multiple of 16: the row count of one operand tile
  uint8_t *hist_q;     // [L][batch][Hkv * G][D / 64][hist_wp][64] bf16: per query head the K-major operand tile of
                       // the feature kernel (row = ring slot, 128-byte rows, chunks XOR-swizzled by the row)
  float *hist_mp;      // [L][batch][Hkv * G][hist_wp]: log2 of the softmax denominator of that query, max included
  int *hist_n;         // [L][batch][W]: pairs the query saw
  int *hist_cnt;       // [L][batch]: queries recorded since the last eviction
};

// The sequences that take part in an append: bit s of word s / 64; use == 0 means every sequence.
constexpr int kMaxBatch = 256;
struct SeqMask {
  unsigned long long w[kMaxBatch / 64];
  int use;
  __host__ __device__ bool has(int s) const {   // (no indexed access: the struct is a kernel parameter)
    const unsigned long long x = s < 64 ? w[0] : s < 128 ? w[1] : s < 192 ? w[2] : w[3];
    return !use || ((x >> (s & 63)) & 1ull);
  }
  static_assert(kMaxBatch == 256, "four words");
};

__device__ __forceinline__ int seg_of(const Ctx &c, int layer, int seq, int head) {
  return (layer * c.batch + seq) * c.Hkv + head;
}

// Byte offset, inside a page record, of 16-byte chunk `ch` (8 channels) of the K row of pair r; the V row
// follows the K row (+ 2D bytes).  Chunks are XOR-swizzled by the row index inside each 128-byte span.
__device__ __forceinline__ int kv_chunk_off(int r, int ch, int D) {
  return r * (4 * D) + ((ch >> 3) << 7) + (((ch & 7) ^ (r & 7)) << 4);
}

// Byte offset, inside the query record, of 16-byte chunk `ch` of the query that head `qhead` (index over layer,
// sequence and query head) issued at ring slot `slot`: one tile of wp rows x 128 bytes per 64 channels, the
// chunks of a row XOR-swizzled by the row index like the K rows of a page record.
__device__ __forceinline__ size_t hist_q_off(size_t qhead, int ch, int slot, int wp, int D) {
  return ((qhead * (D / 64) + (ch >> 3)) * wp + slot) * 128 + (size_t)(((ch & 7) ^ (slot & 7)) << 4);
}

// Meta row of pair r of a page record: F feature floats, then the position id.
__device__ __forceinline__ float *meta_row(const Ctx &c, uint8_t *page, int r) {
  return reinterpret_cast<float *>(page + c.off_f) + r * (c.F + 1);
}
__device__ __forceinline__ const float *meta_row(const Ctx &c, const uint8_t *page, int r) {
  return reinterpret_cast<const float *>(page + c.off_f) + r * (c.F + 1);
}

__device__ __forceinline__ void set_status(const Ctx &c, unsigned bits) { atomicOr((unsigned *)&c.ctrl[CTRL_STATUS], bits); }

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("{ .reg .b64 st; mbarrier.arrive.shared::cta.b64 st, [%0]; }" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }" ::"r"(bar), "r"(bytes)
               : "memory");
}
// Bounded wait on a phase parity.  try_wait suspends for a hardware time slice
// per call, so the cap is seconds, far beyond any copy latency; false = gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < (1u << 22); ++i) {
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// One-dimensional bulk copy global -> shared, completion counted in bytes on an mbarrier.
// Both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

// L2 eviction policies: "first" for data streamed through once, "last" for small results the next
// kernel reads back (they then never leave L2 while the stream runs).
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void st_f32_hint(float *p, float v, uint64_t pol) {
  asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(p), "f"(v), "l"(pol) : "memory");
}

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// D(16x8, fp32) += A(16x8, tf32, row) * B(8x8, tf32, col); operands are fp32 bit patterns whose low 13 bits are zero.
__device__ __forceinline__ void mma_tf32(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Transpose of an 8 x 8 tile of 16-bit values held one row-pair per lane (the mma fragment layout).
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// 16-byte asynchronous copy global -> shared (bypasses L1).
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// Waits for this thread's async copies; other threads see the data after the next barrier.
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}
// Groups of this thread's async copies: close the current group; wait until at most N groups are still in flight.
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_pending() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

// ---------------------------------------------------------------- thread-block clusters
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
__device__ __forceinline__ void dsmem_st4(uint32_t addr, float4 v) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
               : "memory");
}
__device__ __forceinline__ void dsmem_st2(uint32_t addr, float x, float y) {
  asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(x), "f"(y) : "memory");
}
__device__ __forceinline__ uint32_t dsmem_ld_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ unsigned long long dsmem_ld_u64(uint32_t addr) {
  unsigned long long v;
  asm volatile("ld.shared::cluster.u64 %0, [%1];" : "=l"(v) : "r"(addr) : "memory");
  return v;
}

// ---------------------------------------------------------------- row movers
// One warp moves one pair (K row, V row, feature row, position) between a
// dense row and a slot of a page record.  DIR 0: dense -> page, 1: page -> dense.
// The dense side is read through L2 (callers may run alongside the launch before them, see k_attend).
template <int DIR>
__device__ __forceinline__ void move_row(const Ctx &c, uint8_t *page, int r, uint8_t *k, uint8_t *v, float *feat,
                                         int32_t *pos, int lane, int32_t pos_default) {
  const int nch = c.D >> 3;  // 16-byte chunks per K (or V) row
  for (int q = lane; q < 2 * nch; q += 32) {
    const int isv = q >= nch, ch = isv ? q - nch : q;
    uint4 *pp = reinterpret_cast<uint4 *>(page + (isv ? c.off_v : 0) + kv_chunk_off(r, ch, c.D));
    uint8_t *dense = isv ? v : k;
    if (DIR == 0) {
      *pp = dense ? __ldcg(reinterpret_cast<const uint4 *>(dense + ch * 16)) : make_uint4(0, 0, 0, 0);
    } else if (dense) {
      *reinterpret_cast<uint4 *>(dense + ch * 16) = *pp;
    }
  }
  float *pf = meta_row(c, page, r);
  for (int f = lane; f < c.F; f += 32) {
    if (DIR == 0) pf[f] = feat ? __ldcg(feat + f) : 0.f;
    else if (feat) feat[f] = pf[f];
  }
  if (lane == 0) {
    int32_t *pp = reinterpret_cast<int32_t *>(pf + c.F);
    if (DIR == 0) *pp = pos ? __ldcg(pos) : pos_default;
    else if (pos) *pos = *pp;
  }
}

// Block-wide exclusive prefix sum of one int per thread (blockDim.x <= 1024,
// a multiple of 32).  `total` gets the block total.  smem: 33 ints.
__device__ __forceinline__ int block_excl_scan(int v, int *smem, int &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();  // smem may still be read from a previous call
  if (lane == 31) smem[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = lane < nw ? smem[lane] : 0, winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    smem[lane] = winc - w;
    if (lane == 31) smem[32] = winc;
  }
  __syncthreads();
  total = smem[32];
  return smem[warp] + inc - v;
}

}  // namespace fkv
