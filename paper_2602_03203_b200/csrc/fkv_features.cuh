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
// grid (groups of NW pages, work list); NW warps, warp w owns page w of the group: its K fragments
// stay in registers while the CTA walks the query heads, staging one head's queries at a time.
#pragma once
#include "fkv_dev.cuh"

namespace fkv {

constexpr float kFeatDecay = 0.9f;   // Appendix B.1: per-chunk decay of the decayed sum

struct FeatSmem {
  // pages [nw][4D * 16] | queries of one head [W][2D] | M [W] | 1/L [W] | pairs seen [W]
  static __host__ __device__ size_t bytes(int D, int nw, int W) {
    return (size_t)nw * 4 * D * kPage + (size_t)W * 2 * D + (size_t)W * 12 + 16;
  }
};

template <int D, int NW>
__global__ void __launch_bounds__(NW * 32) k_features(Ctx c, float scale_log2) {
  constexpr int KSH = D / 16;
  constexpr int PAGE_KV = 4 * D * kPage;
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ uint64_t s_bar;
  if ((int)blockIdx.y >= c.planhdr[PH_NWORK]) return;
  const int seg = c.work[blockIdx.y];
  const int n = c.plan[seg].n_old;
  const int npages = (n + kPage - 1) / kPage, pg0 = blockIdx.x * NW;
  if (pg0 >= npages) return;
  const int ls = seg / c.Hkv, head = seg % c.Hkv, G = c.G, W = c.hist_w, Hq = c.Hkv * G;
  const int cnt = c.hist_cnt[ls];
  const int Lc = min(cnt, W);            // queries of the chunk that are on record
  if (Lc == 0) return;                   // nothing recorded: the stored features stand as they are
  const int Lp = (Lc + 7) & ~7;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
  const int gid = lane >> 2, tig = lane & 3;
  uint8_t *pages = smem;
  uint8_t *qs = smem + (size_t)NW * PAGE_KV;                       // [Lp][2D], 16-byte chunks swizzled by row
  float *sM = reinterpret_cast<float *>(qs + (size_t)W * 2 * D), *sIL = sM + W;
  int *sN = reinterpret_cast<int *>(sIL + W);
  const int np = min(NW, npages - pg0);

  // ---- the K|V blocks of this group's pages: one bulk copy each, one barrier ----
  if (tid == 0) {
    mbar_init(smem_u32(&s_bar), 1);
    fence_barrier_init();
  }
  __syncthreads();
  if (warp == 0) {
    if (lane == 0) mbar_arrive_expect_tx(smem_u32(&s_bar), (uint32_t)(np * PAGE_KV));
    __syncwarp();
    if (lane < np) {
      const int pid = c.pt[(size_t)seg * c.max_pages + pg0 + lane];
      bulk_g2s(smem_u32(pages + (size_t)lane * PAGE_KV), c.pool + (size_t)pid * c.page_bytes, PAGE_KV, smem_u32(&s_bar));
    }
  }
  const bool ok = mbar_wait(smem_u32(&s_bar), 0);
  if (!ok) set_status(c, kDevWaitTimeout);   // falls through: every thread still reaches the barriers below

  // K rows of this warp's page as A fragments (keys x channels), for all heads.
  uint32_t ka[KSH][4];
  const int krow = ((lane >> 3) & 1) * 8 + (lane & 7), khi = lane >> 4;
  if (warp < np) {
    const uint32_t kbase = smem_u32(pages + (size_t)warp * PAGE_KV);
#pragma unroll
    for (int ks = 0; ks < KSH; ++ks) ldsm_x4(ka[ks], kbase + kv_chunk_off(krow, ks * 2 + khi, D));
  }
  const int slot0 = (pg0 + warp) * kPage + gid;   // this lane's pairs: slot0 and slot0 + 8
  const uint8_t *hq = c.hist_q + (size_t)ls * W * Hq * D * 2;
  const float2 *hml = reinterpret_cast<const float2 *>(c.hist_ml) + (size_t)ls * W * Hq;
  const int *hn = c.hist_n + (size_t)ls * W;
  // ldmatrix roles for the queries as B (queries x channels, row-major): matrix mi -> 8 queries,
  // channel chunk 2 * kp * 2 + mi: one x4 load gives the B fragments of two k-steps.
  const int qrow = lane & 7, qmi = lane >> 3;

  for (int j = 0; j < G; ++j) {
    const int qh = head * G + j;
    __syncthreads();   // the previous head's queries are no longer read
    // ---- stage this head's queries newest first (index a = age), with their statistics ----
    for (int e = tid; e < Lp * (D / 8); e += blockDim.x) {
      const int a = e / (D / 8), ch = e - a * (D / 8);
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (a < Lc) {
        const int hs = ((cnt - 1 - a) % W + W) % W;
        v = *reinterpret_cast<const uint4 *>(hq + ((size_t)hs * Hq + qh) * D * 2 + ch * 16);
      }
      *reinterpret_cast<uint4 *>(qs + (size_t)a * 2 * D + ((ch & ~7) | ((ch ^ a) & 7)) * 16) = v;
    }
    for (int a = tid; a < Lp; a += blockDim.x) {
      float M = 0.f, il = 0.f;
      int nv = 0;
      if (a < Lc) {
        const int hs = ((cnt - 1 - a) % W + W) % W;
        const float2 ml = hml[(size_t)hs * Hq + qh];
        M = ml.x; il = 1.f / ml.y; nv = hn[hs];
      }
      sM[a] = M; sIL[a] = il; sN[a] = nv;
    }
    __syncthreads();
    if (warp >= np) continue;
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};   // rows gid, gid + 8: windows 8, 16, 32, all
    const uint32_t qbase = smem_u32(qs);
    for (int a0 = 0; a0 < Lp; a0 += 8) {
      float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int kp = 0; kp < KSH / 2; ++kp) {
        uint32_t b[4];
        const int r = a0 + qrow, ch = kp * 4 + qmi;
        ldsm_x4(b, qbase + r * 2 * D + (((ch & ~7) | ((ch ^ r) & 7)) << 4));
        mma_bf16(s, ka[2 * kp][0], ka[2 * kp][1], ka[2 * kp][2], ka[2 * kp][3], b[0], b[1]);
        mma_bf16(s, ka[2 * kp + 1][0], ka[2 * kp + 1][1], ka[2 * kp + 1][2], ka[2 * kp + 1][3], b[2], b[3]);
      }
      // s[0], s[1]: pair slot0, queries a0 + 2 tig (+1); s[2], s[3]: pair slot0 + 8.
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int a = a0 + 2 * tig + e;
        const float M = sM[a], il = sIL[a];
        const int nv = sN[a];
        const float p0 = slot0 < nv ? exp2f(s[e] * scale_log2 - M) * il : 0.f;
        const float p1 = slot0 + 8 < nv ? exp2f(s[2 + e] * scale_log2 - M) * il : 0.f;
        if (a0 < 8) { acc[0][0] += p0; acc[1][0] += p1; }
        if (a0 < 16) { acc[0][1] += p0; acc[1][1] += p1; }
        if (a0 < 32) { acc[0][2] += p0; acc[1][2] += p1; }
        acc[0][3] += p0; acc[1][3] += p1;
      }
    }
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        acc[r][k] += __shfl_xor_sync(0xffffffffu, acc[r][k], 1);
        acc[r][k] += __shfl_xor_sync(0xffffffffu, acc[r][k], 2);
      }
    // Lane tig == r of a quad writes row r's six features of this head (rows gid and gid + 8).
    if (tig < 2) {
      const int slot = slot0 + 8 * tig;
      if (slot < n) {
        const float w8 = tig ? acc[1][0] : acc[0][0], w16 = tig ? acc[1][1] : acc[0][1];
        const float w32 = tig ? acc[1][2] : acc[0][2], wall = tig ? acc[1][3] : acc[0][3];
        const int pid = c.pt[(size_t)seg * c.max_pages + slot / kPage];
        float *f = meta_row(c, c.pool + (size_t)pid * c.page_bytes, slot % kPage) + j * 6;
        const float chunk = wall / (float)Lc;
        f[0] = w8 * (1.f / 8.f); f[1] = w16 * (1.f / 16.f); f[2] = w32 * (1.f / 32.f);
        f[3] = chunk;
        f[4] = f[4] + chunk;
        f[5] = fmaf(kFeatDecay, f[5], chunk);
      }
    }
  }
}

}  // namespace fkv
