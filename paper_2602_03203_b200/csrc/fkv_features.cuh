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
// a dense contraction [pairs x D] . [D x queries] on the tensor cores: keys on the M axis of the
// mma (the K rows of a page record, already swizzled for ldmatrix), queries on N from a staged,
// newest-first copy of the history, so the windows are prefixes of the query axis.  The decode path
// pays 2 g D + 12 g bytes per token for the record instead of a read-modify-write of every pair's
// feature row per token.
//
// grid (groups of NW * PPW pages, work list); NW warps, each owning PPW pages of the group.  Only the K
// rows of the pages are staged (16-byte async copies keep the record's swizzle); the CTA walks the
// query heads with two query buffers: the next head's queries stream in (async copies again) while
// the current head is computed.
#pragma once
#include "fkv_dev.cuh"

namespace fkv {

constexpr float kFeatDecay = 0.9f;   // Appendix B.1: per-chunk decay of the decayed sum

constexpr int kFeatPPW = 1;   // pages per warp

struct FeatSmem {
  // K rows of the pages [nw * PPW][16][2D] | their meta rows [nw * PPW][16 * 49 words, padded] |
  // 2 x { queries of one head [W][2D] | M + log2 L [W] | pairs seen [W] }
  static __host__ __device__ size_t meta(int F) { return (size_t)kPage * (F + 1) * 4; }   // a multiple of 64 bytes
  static __host__ __device__ size_t qbuf(int D, int W) { return (size_t)W * 2 * D + (size_t)W * 8; }
  static __host__ __device__ size_t bytes(int D, int F, int nw, int W) {
    return (size_t)nw * kFeatPPW * (2 * D * kPage + meta(F)) + 2 * qbuf(D, W) + 16;
  }
};

// 2^x for x <= 0 (tiny results may flush to zero).
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Offset of 16-byte chunk ch of row r in a [rows][2D bytes] tile whose chunks are XOR-swizzled by the row index.
__device__ __forceinline__ int row_chunk_off(int r, int ch, int D) {
  return r * 2 * D + ((ch >> 3) << 7) + (((ch & 7) ^ (r & 7)) << 4);
}

template <int D, int NW>
__global__ void __launch_bounds__(NW * 32) k_features(Ctx c, float scale_log2) {
  constexpr int KSH = D / 16, NCH = D / 8, PPW = kFeatPPW, PG = NW * PPW;
  constexpr int PAGE_K = 2 * D * kPage;
  extern __shared__ __align__(128) uint8_t smem[];
  if ((int)blockIdx.y >= c.planhdr[PH_NWORK]) return;
  const int seg = c.work[blockIdx.y];
  const int n = c.plan[seg].n_old;
  const int npages = (n + kPage - 1) / kPage, pg0 = blockIdx.x * PG;
  if (pg0 >= npages) return;
  const int ls = seg / c.Hkv, head = seg % c.Hkv, G = c.G, W = c.hist_w, Hq = c.Hkv * G;
  const int cnt = c.hist_cnt[ls];
  const int Lc = min(cnt, W);            // queries of the chunk that are on record
  if (Lc == 0) return;                   // nothing recorded: the stored features stand as they are
  const int Lp = (Lc + 7) & ~7;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
  const int gid = lane >> 2, tig = lane & 3;
  uint8_t *kpages = smem;
  const size_t meta_bytes = FeatSmem::meta(c.F);
  uint8_t *metas = smem + (size_t)PG * PAGE_K;                     // the pages' meta blocks (features + positions)
  uint8_t *qbuf0 = metas + (size_t)PG * meta_bytes;           // two buffers of FeatSmem::qbuf bytes
  const size_t qbytes = FeatSmem::qbuf(D, W);
  const int np = min(PG, npages - pg0);

  // ---- K rows of this group's pages: 16-byte async copies, chunk for chunk (the swizzle is kept) ----
  for (int e = tid; e < np * kPage * NCH; e += blockDim.x) {
    const int pg = e / (kPage * NCH), rc = e - pg * (kPage * NCH), r = rc / NCH, ch = rc - r * NCH;
    const int pid = c.pt[(size_t)seg * c.max_pages + pg0 + pg];
    cp_async16(smem_u32(kpages + (size_t)pg * PAGE_K + r * 2 * D + ch * 16),
               c.pool + (size_t)pid * c.page_bytes + (size_t)r * 4 * D + ch * 16);
  }
  const int meta_chunks = (kPage * (c.F + 1) * 4) / 16;   // the meta block is a multiple of 16 bytes (64 (F + 1))
  for (int e = tid; e < np * meta_chunks; e += blockDim.x) {
    const int pg = e / meta_chunks, ch = e - pg * meta_chunks;
    const int pid = c.pt[(size_t)seg * c.max_pages + pg0 + pg];
    cp_async16(smem_u32(metas + (size_t)pg * meta_bytes + ch * 16), c.pool + (size_t)pid * c.page_bytes + c.off_f + ch * 16);
  }
  const uint8_t *hq = c.hist_q + (size_t)ls * W * Hq * D * 2;
  const float2 *hml = reinterpret_cast<const float2 *>(c.hist_ml) + (size_t)ls * W * Hq;
  const int *hn = c.hist_n + (size_t)ls * W;
  const int newest = (cnt - 1) % W;                  // ring slot of the most recent query (cnt >= 1 here)
  const int nv_min = hn[(cnt - Lc) % W];             // the oldest recorded query saw the fewest pairs
  // ldmatrix roles.  K as A (keys x channels): matrix lane/8 -> keys ((lane/8)&1)*8.., chunk +lane/16.
  // Queries as B (queries x channels, row-major): matrix lane/8 -> chunk +lane/8; one x4 = two k-steps.
  const int krow = ((lane >> 3) & 1) * 8 + (lane & 7), khi = lane >> 4;
  const int qrow = lane & 7, qmi = lane >> 3;

  // Stages head j's queries newest first (index a = age) into buffer b: the vectors by async copies, the
  // statistics through registers.  Rows beyond the record are zero / "saw nothing".
  auto stage = [&](int j, int b) {
    const int qh = head * G + j;
    uint8_t *qs = qbuf0 + (size_t)b * qbytes;
    float *sM = reinterpret_cast<float *>(qs + (size_t)W * 2 * D);
    int *sN = reinterpret_cast<int *>(sM + W);
    for (int e = tid; e < Lp * NCH; e += blockDim.x) {
      const int a = e / NCH, ch = e - a * NCH;
      uint8_t *dst = qs + row_chunk_off(a, ch, D);
      if (a < Lc) {
        const int hs = newest - a + (newest < a ? W : 0);
        cp_async16(smem_u32(dst), hq + ((size_t)hs * Hq + qh) * D * 2 + ch * 16);
      } else {
        *reinterpret_cast<uint4 *>(dst) = make_uint4(0u, 0u, 0u, 0u);
      }
    }
    for (int a = tid; a < Lp; a += blockDim.x) {
      float Mp = 0.f;
      int nv = 0;
      if (a < Lc) {
        const int hs = newest - a + (newest < a ? W : 0);
        const float2 ml = hml[(size_t)hs * Hq + qh];
        Mp = ml.x + log2f(ml.y); nv = hn[hs];
      }
      sM[a] = Mp; sN[a] = nv;
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  stage(0, 0);   // (its group also carries the page copies issued above)

  for (int j = 0; j < G; ++j) {
    const uint8_t *qs = qbuf0 + (size_t)(j & 1) * qbytes;
    const float *sM = reinterpret_cast<const float *>(qs + (size_t)W * 2 * D);
    const int *sN = reinterpret_cast<const int *>(sM + W);
    __syncthreads();   // the other buffer (head j - 1) is no longer read
    if (j + 1 < G) {
      stage(j + 1, (j + 1) & 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");   // head j (and the pages) have landed; j + 1 is in flight
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    const uint32_t qbase = smem_u32(qs);
#pragma unroll 1
    for (int u = 0; u < PPW; ++u) {
      const int pg = warp * PPW + u;
      if (pg >= np) break;
      // K rows of the page as A fragments.
      uint32_t ka[KSH][4];
      const uint32_t kbase = smem_u32(kpages + (size_t)pg * PAGE_K);
#pragma unroll
      for (int ks = 0; ks < KSH; ++ks) ldsm_x4(ka[ks], kbase + row_chunk_off(krow, ks * 2 + khi, D));
      const int slot0 = (pg0 + pg) * kPage + gid;   // this lane's pairs: slot0 and slot0 + 8
      const bool whole = (pg0 + pg) * kPage + kPage <= nv_min;   // every recorded query saw the whole page
      float run0 = 0.f, run1 = 0.f;                 // running sums over the queries, newest first
      float w8[2] = {0.f, 0.f}, w16[2] = {0.f, 0.f}, w32[2] = {0.f, 0.f};
      for (int a0 = 0; a0 < Lp; a0 += 8) {
        if (a0 == 8) { w8[0] = run0; w8[1] = run1; }
        if (a0 == 16) { w16[0] = run0; w16[1] = run1; }
        if (a0 == 32) { w32[0] = run0; w32[1] = run1; }
        float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int kp = 0; kp < KSH / 2; ++kp) {
          uint32_t b[4];
          ldsm_x4(b, qbase + row_chunk_off(a0 + qrow, kp * 4 + qmi, D));
          mma_bf16(sa, ka[2 * kp][0], ka[2 * kp][1], ka[2 * kp][2], ka[2 * kp][3], b[0], b[1]);
          mma_bf16(sb, ka[2 * kp + 1][0], ka[2 * kp + 1][1], ka[2 * kp + 1][2], ka[2 * kp + 1][3], b[2], b[3]);
        }
        // [0], [1]: pair slot0, queries a0 + 2 tig (+1); [2], [3]: pair slot0 + 8.
        const float2 M2 = *reinterpret_cast<const float2 *>(sM + a0 + 2 * tig);
        float p00 = ex2((sa[0] + sb[0]) * scale_log2 - M2.x), p01 = ex2((sa[1] + sb[1]) * scale_log2 - M2.y);
        float p10 = ex2((sa[2] + sb[2]) * scale_log2 - M2.x), p11 = ex2((sa[3] + sb[3]) * scale_log2 - M2.y);
        if (!whole) {
          const int2 N2 = *reinterpret_cast<const int2 *>(sN + a0 + 2 * tig);
          if (slot0 >= N2.x) p00 = 0.f;
          if (slot0 >= N2.y) p01 = 0.f;
          if (slot0 + 8 >= N2.x) p10 = 0.f;
          if (slot0 + 8 >= N2.y) p11 = 0.f;
        } else if (a0 + 8 > Lc) {   // the padded tail of the query axis
          if (a0 + 2 * tig >= Lc) { p00 = 0.f; p10 = 0.f; }
          if (a0 + 2 * tig + 1 >= Lc) { p01 = 0.f; p11 = 0.f; }
        }
        run0 += p00 + p01;
        run1 += p10 + p11;
      }
      if (Lp <= 8) { w8[0] = run0; w8[1] = run1; }
      if (Lp <= 16) { w16[0] = run0; w16[1] = run1; }
      if (Lp <= 32) { w32[0] = run0; w32[1] = run1; }
      float vals[2][4] = {{w8[0], w16[0], w32[0], run0}, {w8[1], w16[1], w32[1], run1}};
#pragma unroll
      for (int r = 0; r < 2; ++r)
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          vals[r][k] += __shfl_xor_sync(0xffffffffu, vals[r][k], 1);
          vals[r][k] += __shfl_xor_sync(0xffffffffu, vals[r][k], 2);
        }
      // Lane tig == r of a quad writes row r's six features of this head (rows gid and gid + 8).
      if (tig < 2) {
        const int slot = slot0 + 8 * tig;
        if (slot < n) {
          const float a8 = tig ? vals[1][0] : vals[0][0], a16 = tig ? vals[1][1] : vals[0][1];
          const float a32 = tig ? vals[1][2] : vals[0][2], all = tig ? vals[1][3] : vals[0][3];
          float *f = reinterpret_cast<float *>(metas + (size_t)pg * meta_bytes) + (slot % kPage) * (c.F + 1) + j * 6;
          const float chunk = all / (float)Lc;
          f[0] = a8 * (1.f / 8.f); f[1] = a16 * (1.f / 16.f); f[2] = a32 * (1.f / 32.f);
          f[3] = chunk;
          f[4] = f[4] + chunk;
          f[5] = fmaf(kFeatDecay, f[5], chunk);
        }
      }
    }
  }
  // ---- the refreshed meta blocks go back to their page records (every row was written by one lane) ----
  __syncthreads();
  for (int e = tid; e < np * meta_chunks; e += blockDim.x) {
    const int pg = e / meta_chunks, ch = e - pg * meta_chunks;
    const int pid = c.pt[(size_t)seg * c.max_pages + pg0 + pg];
    *reinterpret_cast<uint4 *>(c.pool + (size_t)pid * c.page_bytes + c.off_f + ch * 16) =
        *reinterpret_cast<const uint4 *>(metas + (size_t)pg * meta_bytes + ch * 16);
  }
}

}  // namespace fkv
