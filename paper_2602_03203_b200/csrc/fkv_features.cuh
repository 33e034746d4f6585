// Kernel 6: the attention features a_n of Appendix B.1, refreshed when an eviction closes a chunk.
//
// Per query head: recent-window attention for windows 8, 16, 32 and the update length, the sum of
// the chunk scores over chunks, and the same sum decayed by 0.9 per chunk.  Reading taken: a
// window feature is the MEAN over the last w decode queries of the softmax probability the head
// gave to the pair (0 for queries older than the pair); the chunk score is the window = update
// length feature; both cumulative features are updated before the scorer reads them.
//
// Nothing is accumulated during decoding.  Each decode launch that appends a token records its
// queries and, per query head, the softmax statistics (max M and sum L, log2 domain) and the
// number of pairs it saw.  Here the probabilities are RECOMPUTED for the whole chunk at once,
//     p[t][i] = 2^(scale <q_t, k_i> - M_t) / L_t,
// which is a dense contraction [128 pairs x D] . [D x queries] per tile - the one step of this
// library that is compute-shaped, so it runs on the 5th-generation tensor cores:
//   - A = the K rows of 8 pages (128 pairs), B = one query head's recorded queries, newest first;
//     both are staged in shared memory as K-major tiles of 128-byte rows with the 128-byte swizzle
//     (the page record's own swizzle: 16-byte async copies move the chunks verbatim);
//   - one elected thread issues tcgen05.mma (kind::f16, bf16 x bf16 -> fp32, M = 128, N = the
//     padded query count, K = 16 per instruction) with shared-memory descriptors; the accumulator
//     lives in tensor memory (one fp32 column per query), completion arrives on an mbarrier
//     through tcgen05.commit;
//   - the warps read the accumulator back with tcgen05.ld (lane = pair, 32 query columns at a
//     time); a thread owns ONE pair, and because the queries are ordered newest first the windows
//     8 / 16 / 32 / all are running prefix sums along its row: exp2, (mask,) add.  Warps 0-3 take
//     the newer half of the query axis, warps 4-7 the older half, whose sum they hand over
//     through shared memory;
//   - while a head is being multiplied and reduced, the next head's queries stream in.
// The decode path pays 2 g D + 12 g bytes per token for the record instead of a read-modify-write
// of every pair's feature row per token.
//
// grid (groups of 8 pages, work list), 256 threads.  Tensor memory: the CTA allocates a power of
// two >= the padded query count (<= 256 columns) and frees it before it exits; the launch asks for
// enough shared memory that at most two CTAs share an SM, so allocation never has to wait.
#pragma once
#include "fkv_dev.cuh"

namespace fkv {

constexpr float kFeatDecay = 0.9f;   // Appendix B.1: per-chunk decay of the decayed sum
constexpr int kFeatPages = 8;        // pages (of 16 pairs) per CTA: the M = 128 rows of the mma
constexpr int kFeatMaxQueries = 256; // N of one mma and the widest tensor-memory allocation used

struct FeatSmem {
  static __host__ __device__ int lq(int W) { return (W + 15) & ~15; }                      // padded query count
  static __host__ __device__ size_t meta(int F) { return (size_t)kPage * (F + 1) * 4; }    // a multiple of 64 bytes
  // 1 KB alignment slack | A: K rows [D/64 halves][128 rows][128 B] | Q: 2 buffers x [D/64][lq][128 B] |
  // statistics: 2 x lq x (float M + log2 L, int pairs seen) | meta blocks of the 8 pages | barrier + tmem address
  static __host__ __device__ size_t bytes(int D, int F, int W) {
    const size_t need = 1024 + (size_t)(D / 64) * 128 * 128 + 2 * (size_t)(D / 64) * lq(W) * 128 + 2 * (size_t)lq(W) * 8 +
                        kFeatPages * meta(F) + 64 + 128 * 4;   // + one float per pair: the older half's sum
    return need > 77 * 1024 ? need : 77 * 1024;   // never more than two CTAs per SM (tensor-memory budget)
  }
};

// 2^x for x <= 0 (tiny results may flush to zero).
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- tcgen05 wrappers (5th-generation tensor cores, tensor memory) ----
// Shared-memory matrix descriptor of a K-major tile with 128-byte rows and the 128-byte swizzle:
// start address, stride between 8-row groups = 1024 bytes, descriptor version 1, layout 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3ffffu) >> 4) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, N and M of the instruction.
__device__ __forceinline__ uint32_t umma_idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {   // one full warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {    // the same warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {   // the barrier gets one arrival when the issued mmas are done
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// 32 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

template <int D>
__global__ void __launch_bounds__(256) k_features(Ctx c, float scale_log2) {
  constexpr int HALVES = D / 64, NCH = D / 8, ROWS = kFeatPages * kPage;   // 128 pairs
  extern __shared__ uint8_t smem_raw[];
  if ((int)blockIdx.y >= c.planhdr[PH_NWORK]) return;
  const int seg = c.work[blockIdx.y];
  const int n = c.plan[seg].n_old;
  const int npages = (n + kPage - 1) / kPage, pg0 = blockIdx.x * kFeatPages;
  if (pg0 >= npages) return;
  const int ls = seg / c.Hkv, head = seg % c.Hkv, G = c.G, W = c.hist_w, Hq = c.Hkv * G;
  const int cnt = c.hist_cnt[ls];
  const int Lc = min(cnt, W);            // queries of the chunk that are on record
  if (Lc == 0) return;                   // nothing recorded: the stored features stand as they are
  const int Lq = (Lc + 15) & ~15;        // N of the mma
  const int Lw = FeatSmem::lq(W);        // buffer rows
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
  const int np = min(kFeatPages, npages - pg0);

  uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t *At = smem;                                              // [HALVES][128][128 B]
  uint8_t *Qt = At + (size_t)HALVES * ROWS * 128;                  // [2][HALVES][Lw][128 B]
  const size_t qbuf = (size_t)HALVES * Lw * 128;
  uint8_t *stats = Qt + 2 * qbuf;                                  // [2][Lw] float, then [2][Lw] int
  const size_t meta_bytes = FeatSmem::meta(c.F);
  uint8_t *metas = stats + 2 * (size_t)Lw * 8;
  uint64_t *bar = reinterpret_cast<uint64_t *>(metas + kFeatPages * meta_bytes);
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bar + 1);
  float *older = reinterpret_cast<float *>(smem + FeatSmem::bytes(D, c.F, W) - 1024 - 128 * 4);   // [128]: sums of the older half

  // Tensor memory: a power of two >= 32 columns that holds one fp32 column per query.
  uint32_t ncols = 32;
  while ((int)ncols < Lq) ncols <<= 1;
  if (warp == 0) tmem_alloc(smem_u32(tmem_slot), ncols);
  if (tid == 0) {
    mbar_init(smem_u32(bar), 1);
    fence_barrier_init();
  }

  // ---- A: the K rows of this group's pages, chunk for chunk (row pitch 128 B per 64-channel half) ----
  {
    // Thread = one 16-byte chunk column (ch) of rows R0, R0 + 256 / NCH, ...: fixed offsets, a pointer per page.
    constexpr int RSTEP = 256 / NCH;
    const int ch = tid % NCH, R0 = tid / NCH;
    const uint32_t dst0 = smem_u32(At) + (uint32_t)((ch >> 3) * ROWS * 128 + (ch & 7) * 16);
    const int *ptrow = c.pt + (size_t)seg * c.max_pages + pg0;
#pragma unroll
    for (int k = 0; k < ROWS / RSTEP; ++k) {
      const int Rr = R0 + k * RSTEP, pg = Rr / kPage, r = Rr % kPage;
      if (pg < np)
        cp_async16(dst0 + Rr * 128, c.pool + (size_t)ptrow[pg] * c.page_bytes + r * 4 * D + ch * 16);
      else
        *reinterpret_cast<uint4 *>(At + (size_t)(ch >> 3) * ROWS * 128 + (size_t)Rr * 128 + (ch & 7) * 16) =
            make_uint4(0u, 0u, 0u, 0u);
    }
  }
  const int meta_chunks = (int)(meta_bytes / 16);
  for (int e = tid; e < np * meta_chunks; e += blockDim.x) {
    const int pg = e / meta_chunks, ch = e - pg * meta_chunks;
    const int pid = c.pt[(size_t)seg * c.max_pages + pg0 + pg];
    cp_async16(smem_u32(metas + (size_t)pg * meta_bytes + ch * 16), c.pool + (size_t)pid * c.page_bytes + c.off_f + ch * 16);
  }

  const uint8_t *hq = c.hist_q + (size_t)ls * W * Hq * D * 2;
  const float2 *hml = reinterpret_cast<const float2 *>(c.hist_ml) + (size_t)ls * W * Hq;
  const int *hn = c.hist_n + (size_t)ls * W;
  const int newest = (cnt - 1) % W;                  // ring slot of the most recent query (cnt >= 1 here)
  // Stages head j's queries newest first (row a = age) into buffer b, swizzled like the K rows, and their
  // statistics.  Rows beyond the record are zero / "saw nothing".
  auto stage = [&](int j, int b) {
    const int qh = head * G + j;
    uint8_t *qs = Qt + (size_t)b * qbuf;
    float *sM = reinterpret_cast<float *>(stats) + (size_t)b * Lw;
    int *sN = reinterpret_cast<int *>(stats + 2 * (size_t)Lw * 4) + (size_t)b * Lw;
    {
      constexpr int RSTEP = 256 / NCH;
      const int ch = tid % NCH;
      uint8_t *col = qs + (size_t)(ch >> 3) * Lw * 128;
      const uint8_t *src0 = hq + (size_t)qh * D * 2 + ch * 16;
      const size_t hstride = (size_t)Hq * D * 2;
      for (int a = tid / NCH; a < Lq; a += RSTEP) {
        uint8_t *dst = col + (size_t)a * 128 + (((ch & 7) ^ (a & 7)) << 4);
        if (a < Lc) {
          const int hs = newest - a + (newest < a ? W : 0);
          cp_async16(smem_u32(dst), src0 + hs * hstride);
        } else {
          *reinterpret_cast<uint4 *>(dst) = make_uint4(0u, 0u, 0u, 0u);
        }
      }
    }
    for (int a = tid; a < Lq; a += blockDim.x) {
      float Mp = 0.f;
      int nv = 0;
      if (a < Lc) {
        const int hs = newest - a + (newest < a ? W : 0);
        const float2 ml = hml[(size_t)hs * Hq + qh];
        Mp = ml.x + log2f(ml.y); nv = hn[hs];
      }
      sM[a] = Mp; sN[a] = nv;
    }
  };
  stage(0, 0);

  const uint32_t idesc = umma_idesc_bf16(ROWS, Lq);
  const int R = (warp & 3) * 32 + lane;              // epilogue: this thread's pair row of the tile
  const int slot = pg0 * kPage + R;
  // Did every recorded query see the whole tile?  (The oldest one saw the fewest pairs.)
  const bool whole = pg0 * kPage + ROWS <= hn[(cnt - Lc) % W];
  bool ok = true;
  uint32_t tmem_base = 0;

  for (int j = 0; j < G; ++j) {
    const int b = j & 1;
    cp_async_wait_all();       // this thread's copies (A, meta, head j's queries) have landed
    fence_proxy_async();       // ... and are visible to the tensor core's reads of shared memory
    tc_fence_before();
    __syncthreads();           // everybody's; and the previous head's accumulator has been read
    tc_fence_after();
    if (j == 0) tmem_base = *tmem_slot;
    if (tid == 0) {
      const uint32_t a0 = smem_u32(At), q0 = smem_u32(Qt + (size_t)b * qbuf);
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {          // K = 16 channels per instruction: 32 bytes inside the swizzled row
        const uint64_t ad = umma_desc_sw128(a0 + (ks >> 2) * ROWS * 128 + (ks & 3) * 32);
        const uint64_t bd = umma_desc_sw128(q0 + (ks >> 2) * Lw * 128 + (ks & 3) * 32);
        umma_bf16(tmem_base, ad, bd, idesc, ks > 0);
      }
      umma_commit(smem_u32(bar));
    }
    if (j + 1 < G) stage(j + 1, b ^ 1);              // streams in while head j is multiplied and reduced
    {
      // ---- epilogue: one pair per thread, its row of the accumulator, newest query first.  The query axis is
      // split in two at a multiple of 32: warps 0-3 reduce [0, split), warps 4-7 [split, Lq). ----
      if (ok && !mbar_wait(smem_u32(bar), j & 1)) { set_status(c, kDevWaitTimeout); ok = false; }
      ok = __all_sync(0xffffffffu, ok);   // the tensor-memory loads below need the whole warp
      tc_fence_after();
      const int split = Lq > 32 ? ((Lq / 2 + 31) & ~31) : Lq;
      const int abeg = warp < 4 ? 0 : split, aend = warp < 4 ? split : Lq;
      const float *sM = reinterpret_cast<const float *>(stats) + (size_t)b * Lw;
      const int *sN = reinterpret_cast<const int *>(stats + 2 * (size_t)Lw * 4) + (size_t)b * Lw;
      float run = 0.f, w8 = 0.f, w16 = 0.f, w32 = 0.f;
      if (ok) {
        for (int a0 = abeg; a0 < aend; a0 += 32) {
          if (a0 == 32) w32 = run;
          float v[32];
          tmem_ld32(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)a0, v);
          if (whole && a0 + 32 <= Lc) {              // every query of the chunk saw the whole tile: no masks
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              const float4 M4 = *reinterpret_cast<const float4 *>(sM + a0 + i);
              if (i == 8 && a0 == 0) w8 = run;
              if (i == 16 && a0 == 0) w16 = run;
              run += (ex2(v[i] * scale_log2 - M4.x) + ex2(v[i + 1] * scale_log2 - M4.y)) +
                     (ex2(v[i + 2] * scale_log2 - M4.z) + ex2(v[i + 3] * scale_log2 - M4.w));
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              if (i < 16 || a0 + i < Lq) {           // Lq is a multiple of 16: the second half of a chunk may be padding
                const float4 M4 = *reinterpret_cast<const float4 *>(sM + a0 + i);
                const int4 N4 = *reinterpret_cast<const int4 *>(sN + a0 + i);
                if (i == 8 && a0 == 0) w8 = run;
                if (i == 16 && a0 == 0) w16 = run;
                run += slot < N4.x ? ex2(v[i] * scale_log2 - M4.x) : 0.f;
                run += slot < N4.y ? ex2(v[i + 1] * scale_log2 - M4.y) : 0.f;
                run += slot < N4.z ? ex2(v[i + 2] * scale_log2 - M4.z) : 0.f;
                run += slot < N4.w ? ex2(v[i + 3] * scale_log2 - M4.w) : 0.f;
              }
            }
          }
        }
      }
      tc_fence_before();
      if (warp >= 4) older[R] = run;
      asm volatile("bar.sync 1, 256;" ::: "memory");   // the older half's sums are in shared memory
      if (warp < 4 && ok) {
        if (split <= 16) w16 = run;   // windows wider than this thread's half (split is 16, or a multiple of 32)
        if (split <= 32) w32 = run;
        run += older[R];
        if (slot < n) {
          float *f = reinterpret_cast<float *>(metas + (size_t)(R / kPage) * meta_bytes) + (R % kPage) * (c.F + 1) + j * 6;
          const float chunk = run / (float)Lc;
          f[0] = w8 * (1.f / 8.f); f[1] = w16 * (1.f / 16.f); f[2] = w32 * (1.f / 32.f);
          f[3] = chunk;
          f[4] = f[4] + chunk;
          f[5] = fmaf(kFeatDecay, f[5], chunk);
        }
      }
    }
  }
  // ---- the refreshed meta blocks go back to their page records (every row was written by one thread) ----
  cp_async_wait_all();
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, ncols);
  for (int e = tid; e < np * meta_chunks; e += blockDim.x) {
    const int pg = e / meta_chunks, ch = e - pg * meta_chunks;
    const int pid = c.pt[(size_t)seg * c.max_pages + pg0 + pg];
    *reinterpret_cast<uint4 *>(c.pool + (size_t)pid * c.page_bytes + c.off_f + ch * 16) =
        *reinterpret_cast<const uint4 *>(metas + (size_t)pg * meta_bytes + ch * 16);
  }
}

}  // namespace fkv
