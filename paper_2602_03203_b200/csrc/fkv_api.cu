// Host side of the C ABI declared in include/fkv.h: argument checks, the
// carve-up of the caller's workspace, a host mirror of the segment lengths
// (lengths evolve deterministically, so no call reads them back), and the
// kernel launches.  No device memory is allocated here.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <algorithm>
#include <cmath>
#include <new>
#include <string>
#include <vector>

#include "../../include/fkv.h"
#include "fkv_attend.cuh"
#include "fkv_aux.cuh"
#include "fkv_compact.cuh"
#include "fkv_dev.cuh"
#include "fkv_features.cuh"
#include "fkv_golden.cuh"
#include "fkv_rkv.cuh"
#include "fkv_score.cuh"
#include "fkv_select.cuh"

using namespace fkv;

namespace {

thread_local std::string g_cuda_error;

constexpr int kScorePPS = 8;  // consumer warps of the scorer = pages per tile
constexpr int kAttendMinPages = 4;
constexpr size_t kMaxSmem = 227 * 1024;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// The dynamic shared-memory opt-in is a per-device attribute of a kernel: remember, per kernel and per
// device, the largest size already granted, and ask again only for more.
struct SmemOptIn {
  size_t granted[64] = {};
  template <class Kernel>
  cudaError_t ensure(Kernel kernel, size_t bytes) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    size_t &g = granted[dev & 63];
    if (bytes <= g) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) g = bytes;
    return e;
  }
};

struct Layout {
  size_t pool, free_stack, ctrl, planhdr, pt, pt_new, len, budget, sp, scores, idx, plan, work, tile1, seq_tickets, seq_fail, att_part, att_tickets, hist_q, hist_mp, hist_n, hist_cnt, total;
  int cap, max_pages, num_pages, page_bytes, F, att_smax, sp_stride, sp_off_wf, sp_off_b1, sp_off_w2, sp_off_b2;
};

bool valid_config(const fkv_config *c) {
  if (!c) return false;
  if (c->num_layers < 1 || c->num_kv_heads < 1 || c->num_kv_heads > 32 || c->max_batch < 1 || c->max_batch > kMaxBatch)
    return false;
  if (c->group_size < 1 || c->group_size > 8) return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->page_size != kPage || c->scorer_hidden != kHidden) return false;
  if (c->activation < 0 || c->activation > 3) return false;
  if (c->budget < 1 || c->recent_keep < 0 || c->max_tokens_per_head < 1 || c->num_pages < 0) return false;
  if ((int64_t)c->num_layers * c->max_batch * c->num_kv_heads > (1 << 20)) return false;
  if (c->feature_window < 0 || c->feature_window % 8) return false;
  if (c->feature_window > kFeatMaxQueries) return false;
  return true;
}

Layout make_layout(const fkv_config &c) {
  Layout L{};
  const int D = c.head_dim;
  L.F = 6 * c.group_size;
  L.cap = (int)align_up((size_t)c.max_tokens_per_head, kPage);
  L.max_pages = L.cap / kPage;
  L.page_bytes = 64 * D + 64 * L.F + 64;
  const size_t nseg = (size_t)c.num_layers * c.max_batch * c.num_kv_heads;
  const int bpages = (std::min(c.budget, L.cap) + kPage - 1) / kPage;
  L.num_pages = c.num_pages ? c.num_pages : (int)std::min<size_t>(nseg * ((size_t)L.max_pages + bpages + 1), 0x7fffffff);
  const int KS = 2 * D / 16;
  L.sp_off_wf = 2 * KS * 512;   // fragments of the roundings, then of the remainders
  L.sp_off_b1 = L.sp_off_wf + ScoreSmem::fk(L.F) * 1024;   // feature rows: tf32 fragments, truncations and remainders
  L.sp_off_w2 = L.sp_off_b1 + 64;
  L.sp_off_b2 = L.sp_off_w2 + 64;
  L.sp_stride = (int)align_up((size_t)L.sp_off_b2 + 16, 256);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  L.pool = take((size_t)L.num_pages * L.page_bytes);
  L.free_stack = take((size_t)L.num_pages * 4);
  L.ctrl = take(CTRL_WORDS * 4);
  L.planhdr = take(PH_WORDS * 4);
  L.pt = take(nseg * L.max_pages * 4);
  L.pt_new = take(nseg * L.max_pages * 4);
  L.len = take((size_t)c.num_layers * c.max_batch * 4);
  L.budget = take((size_t)c.max_batch * 4);
  L.sp = take((size_t)c.num_layers * c.num_kv_heads * L.sp_stride);
  L.scores = take(nseg * L.cap * 4);
  L.idx = take(nseg * L.cap * 4);
  L.plan = take(nseg * sizeof(SegPlan));
  L.work = take(nseg * 4);
  L.tile1 = take((nseg + 1) * 4);
  L.seq_tickets = take((size_t)c.num_layers * c.max_batch * 4);
  L.seq_fail = take((size_t)c.num_layers * c.max_batch * 4);
  // Split-K attention: up to att_smax splits per segment (enough for a few CTAs per SM at this batch size).
  L.att_smax = std::max(1, std::min(kMaxSplits, 512 / (c.max_batch * c.num_kv_heads)));
  L.att_part = take(nseg * L.att_smax * c.group_size * (D + 4) * 4);
  L.att_tickets = take(nseg * 4);
  const size_t ls = (size_t)c.num_layers * c.max_batch, W = (size_t)c.feature_window, Hq = (size_t)c.num_kv_heads * c.group_size;
  const size_t Wp = (W + 15) & ~(size_t)15;   // rows of one query tile
  L.hist_q = take(ls * Wp * Hq * D * 2);
  L.hist_mp = take(ls * Wp * Hq * 4);
  L.hist_n = take(ls * W * 4);
  L.hist_cnt = take(W ? ls * 4 : 0);
  L.total = off;
  return L;
}

uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40u);
  u += 0x7fffu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

float bf16_to_f32(uint16_t b) {
  const uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

}  // namespace

struct fkv_cache {
  fkv_config cfg;
  Layout lay;
  Ctx ctx;
  std::vector<int> h_len;     // [L][batch] mirror of the device lengths
  std::vector<int> h_budget;  // [batch]
  std::vector<uint8_t> loaded;  // [L][Hkv] scorer present
  std::vector<uint8_t> staging;
  uint64_t launches = 0;
  int sm_count = 148;
  int max_cluster = 0;        // largest attention cluster the device places (found at the first stand-alone launch)
  float feature_scale = 0.f;  // softmax scale of the recorded queries (the last decode call's)
  bool timing = false, timed = false;
  CUtensorMap k_rows;         // the page pool's K rows as [page][row][64-channel half][64 channels] (R-KV's tensor copies)
  bool k_rows_ready = false;
  cudaEvent_t ev[7] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};  // [6]: after the plan
};

namespace fkv {
// For the library's other translation units: record the text of a failed CUDA call for fkv_last_cuda_error.
void note_cuda_error(cudaError_t e) { g_cuda_error = cudaGetErrorString(e); }
}  // namespace fkv

namespace {

int cuda_fail(cudaError_t e) {
  g_cuda_error = cudaGetErrorString(e);
  return FKV_ERR_CUDA;
}
#define FKV_CUDA(x)                           \
  do {                                        \
    cudaError_t e_ = (x);                     \
    if (e_ != cudaSuccess) return cuda_fail(e_); \
  } while (0)
#define FKV_LAUNCHED(c)                       \
  do {                                        \
    ++(c)->launches;                          \
    cudaError_t e_ = cudaGetLastError();      \
    if (e_ != cudaSuccess) return cuda_fail(e_); \
  } while (0)

// The caller's bit array (host, one word per 64 sequences; NULL = every sequence) as the kernels take it.
SeqMask make_mask(const fkv_cache *c, const uint64_t *bits) {
  SeqMask m = {};
  if (bits) {
    m.use = 1;
    for (int i = 0; i < (c->cfg.max_batch + 63) / 64; ++i) m.w[i] = bits[i];
  }
  return m;
}

bool layer_ok(const fkv_cache *c, int layer) { return layer >= 0 && layer < c->cfg.num_layers; }

// Page slots of the scorer's ring: as many as fit the shared memory, a multiple of the number of warps (a slot
// must always come back to the warp that refilled it: its barrier carries one phase bit, and only the warp that
// waited for the slot's previous page knows that phase is over), at most four per warp.
int score_ring_slots(const fkv_cache *c) {
  for (int n = 4 * kScorePPS; n >= kScorePPS; n -= kScorePPS)
    if (ScoreSmem::bytes(c->lay.page_bytes, c->lay.F, kScorePPS, n) <= kMaxSmem) return n;
  return 0;
}

template <int D>
int launch_score(fkv_cache *c, float *out, int seg_base, int tiles_bound, cudaStream_t st) {
  const int nslots = score_ring_slots(c);
  if (nslots == 0) return FKV_ERR_INVALID_ARG;
  const size_t smem = ScoreSmem::bytes(c->lay.page_bytes, c->lay.F, kScorePPS, nslots);
  static SmemOptIn opt_in;
  FKV_CUDA(opt_in.ensure(k_score<D, kScorePPS>, kMaxSmem));
  const int grid = std::max(1, std::min(c->sm_count, tiles_bound));
  k_score<D, kScorePPS><<<grid, kScorePPS * 32, smem, st>>>(c->ctx, out, seg_base, nslots);
  FKV_LAUNCHED(c);
  return FKV_OK;
}

int launch_score_any(fkv_cache *c, float *out, int seg_base, int tiles_bound, cudaStream_t st) {
  return c->cfg.head_dim == 128 ? launch_score<128>(c, out, seg_base, tiles_bound, st)
                                : launch_score<64>(c, out, seg_base, tiles_bound, st);
}

// One selection launch: mode 0 writes kept slot lists, mode 1 keep-priorities of the sampled action.
void launch_select(fkv_cache *c, int mode, int max_old, int nblocks, const float *scores, int32_t *idx,
                   int32_t *kept_count, int seg_base, int fill_pages, float *prio, const float *noise, int noise_stride,
                   int noise_base, cudaStream_t st) {
  // Variant by the longest segment: registers hold a whole segment up to 2048 (256-thread CTAs, many per SM), 8192
  // (two CTAs per SM) or 32768 keys, a pair of CTAs 65536; longer segments stream their rounds from L2.
#define FKV_SEL(S, M, T, P) \
  k_select<S, M, T, P><<<nblocks, T, 0, st>>>(c->ctx, scores, idx, kept_count, seg_base, fill_pages, prio, noise, \
                                             noise_stride, noise_base)
  if (max_old <= kSelTinyThreads * kSelTinyPerThread) {
    if (mode == 0) FKV_SEL(true, 0, kSelTinyThreads, kSelTinyPerThread); else FKV_SEL(true, 1, kSelTinyThreads, kSelTinyPerThread);
  } else if (max_old <= kSelSmallThreads * kSelSmallPerThread) {
    if (mode == 0) FKV_SEL(true, 0, kSelSmallThreads, kSelSmallPerThread); else FKV_SEL(true, 1, kSelSmallThreads, kSelSmallPerThread);
  } else if (max_old <= kSelRound) {
    if (mode == 0) FKV_SEL(true, 0, kSelThreads, 32); else FKV_SEL(true, 1, kSelThreads, 32);
  } else if (max_old <= 2 * kSelRound) {
    // Up to 65536 keys: a pair of CTAs (one cluster) per segment, each with half of the keys in registers.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * nblocks);
    cfg.blockDim = dim3(kSelThreads);
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (mode == 0)
      (void)cudaLaunchKernelEx(&cfg, k_select<true, 0, kSelThreads, 32, true>, c->ctx, scores, idx, kept_count, seg_base,
                               fill_pages, prio, noise, noise_stride, noise_base);
    else
      (void)cudaLaunchKernelEx(&cfg, k_select<true, 1, kSelThreads, 32, true>, c->ctx, scores, idx, kept_count, seg_base,
                               fill_pages, prio, noise, noise_stride, noise_base);
  } else {
    if (mode == 0) FKV_SEL(false, 0, kSelThreads, 32); else FKV_SEL(false, 1, kSelThreads, 32);
  }
#undef FKV_SEL
}

// Attention features of the segments on the work list (after a k_plan): one persistent CTA per SM, each a
// contiguous range of the plan's 128-pair tiles.
template <int D>
int launch_features_t(fkv_cache *c, int max_old, int nwork_bound, float scale_log2, cudaStream_t st) {
  static_assert(kFeatPages == kScorePPS, "the feature kernel walks the plan's score tiles");
  int na = 0, nq = 0;
  FeatSmem::rings(D, c->cfg.group_size, c->cfg.feature_window, na, nq);
  if (na < 1) return FKV_ERR_INVALID_ARG;
  const size_t smem = FeatSmem::bytes(D, c->cfg.group_size, c->cfg.feature_window, na, nq);
  if (max_old <= 0 || nwork_bound <= 0) return FKV_OK;
  if (FeatSmem::lq(c->cfg.feature_window) <= 128) {   // four accumulators: three reducing warpgroups
    static SmemOptIn opt_in;
    FKV_CUDA(opt_in.ensure(k_features<D, 3>, smem));
    k_features<D, 3><<<c->sm_count, feat_threads(3), smem, st>>>(c->ctx, scale_log2, na, nq);
  } else {                                            // two accumulators, two warpgroups on each
    static SmemOptIn opt_in;
    FKV_CUDA(opt_in.ensure(k_features<D, 4>, smem));
    k_features<D, 4><<<c->sm_count, feat_threads(4), smem, st>>>(c->ctx, scale_log2, na, nq);
  }
  FKV_LAUNCHED(c);
  return FKV_OK;
}
int launch_features(fkv_cache *c, int max_old, int nwork_bound, cudaStream_t st) {
  const float scale_log2 = c->feature_scale * 1.4426950408889634f;
  return c->cfg.head_dim == 128 ? launch_features_t<128>(c, max_old, nwork_bound, scale_log2, st)
                                : launch_features_t<64>(c, max_old, nwork_bound, scale_log2, st);
}

// The tensor map of R-KV's copies: bf16 [num_pages][16 rows][D / 64 halves][64 channels] over the page pool, one box =
// the 16 rows x 64 channels of one page (2 KB, 16 rows of 128 bytes in shared memory; the record's own chunk swizzle
// stays as it is).  The driver's encoder is reached through the runtime, so the library links no driver stub.
int ensure_k_rows_map(fkv_cache *c) {
  if (c->k_rows_ready) return FKV_OK;
  typedef CUresult (*encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  void *fn = nullptr;
  cudaDriverEntryPointQueryResult found;
  FKV_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &found));
  if (fn == nullptr || found != cudaDriverEntryPointSuccess) {
    g_cuda_error = "cuTensorMapEncodeTiled is not available from this driver";
    return FKV_ERR_CUDA;
  }
  const int D = c->cfg.head_dim;
  const cuuint64_t dims[4] = {64, (cuuint64_t)(D / 64), (cuuint64_t)kPage, (cuuint64_t)c->ctx.num_pages};
  const cuuint64_t strides[3] = {128, (cuuint64_t)(4 * D), (cuuint64_t)c->ctx.page_bytes};   // bytes, dimensions 1 .. 3
  const cuuint32_t box[4] = {64, 1, (cuuint32_t)kPage, 1}, step[4] = {1, 1, 1, 1};
  const CUresult r = reinterpret_cast<encode_fn>(fn)(&c->k_rows, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, c->ctx.pool, dims, strides,
                                                     box, step, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_cuda_error = "cuTensorMapEncodeTiled failed with driver error " + std::to_string((int)r);
    return FKV_ERR_CUDA;
  }
  c->k_rows_ready = true;
  return FKV_OK;
}

// R-KV baseline scores of the segments on the work list (after a k_plan): the attention term and the reciprocal
// key norms first (the index scratch holds the norms until the selection overwrites it), then the n x n
// contraction.  Work items sit on grid.x (no 65535 limit).
template <int D>
int launch_rkv_t(fkv_cache *c, float *out, int seg_base, int max_old, int nwork_bound, long long tiles, float la, float ls,
                 cudaStream_t st) {
  if (max_old <= 0 || nwork_bound <= 0) return FKV_OK;
  if (int e = ensure_k_rows_map(c)) return e;
  float *rn = reinterpret_cast<float *>(c->ctx.idx);
  k_rkv_prepare<D><<<dim3(nwork_bound, (max_old + 127) / 128), 128, 0, st>>>(c->ctx, out, rn, seg_base,
                                                                             FKV_FEATURE_WINDOW8);
  FKV_LAUNCHED(c);
  if (tiles > 4) {
    // Pairs of CTAs that multiply as one (a unit is up to four tiles).
    const size_t smem = RkvPairSmem::bytes(D);
    static SmemOptIn opt_in;
    FKV_CUDA(opt_in.ensure(k_rkv_score_pair<D>, smem));
    const int npairs = (int)std::max<long long>(1, std::min<long long>(c->sm_count / 2, (tiles + 3) / 4));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * npairs);
    cfg.blockDim = dim3(kRkvThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    FKV_CUDA(cudaLaunchKernelEx(&cfg, k_rkv_score_pair<D>, c->ctx, c->k_rows, out, (const float *)rn, seg_base, la, ls));
  } else {
    const size_t smem = RkvSmem::bytes(D);
    static SmemOptIn opt_in;
    FKV_CUDA(opt_in.ensure(k_rkv_score<D>, smem));
    const int grid = (int)std::max<long long>(1, std::min<long long>(c->sm_count, tiles));
    k_rkv_score<D><<<grid, kRkvThreads, smem, st>>>(c->ctx, c->k_rows, out, rn, seg_base, la, ls);
  }
  FKV_LAUNCHED(c);
  return FKV_OK;
}
int launch_rkv(fkv_cache *c, float *out, int seg_base, int max_old, int nwork_bound, long long tiles, float la, float ls,
               cudaStream_t st) {
  return c->cfg.head_dim == 128 ? launch_rkv_t<128>(c, out, seg_base, max_old, nwork_bound, tiles, la, ls, st)
                                : launch_rkv_t<64>(c, out, seg_base, max_old, nwork_bound, tiles, la, ls, st);
}

int launch_compact(fkv_cache *c, const int32_t *idx, int seg_base, int max_new, int nwork_bound, cudaStream_t st) {
  const int tiles = (max_new + kCompactRows - 1) / kCompactRows;
  const long long ctas = (long long)nwork_bound * tiles;   // one flat grid: no 65535 limit on the work list
  if (ctas == 0) return FKV_OK;
  if (ctas > 0x7fffffffLL) return FKV_ERR_INVALID_ARG;
  if (c->cfg.head_dim == 128) k_compact<128><<<(unsigned)ctas, 256, 0, st>>>(c->ctx, idx, seg_base, tiles);
  else k_compact<64><<<(unsigned)ctas, 256, 0, st>>>(c->ctx, idx, seg_base, tiles);
  FKV_LAUNCHED(c);
  return FKV_OK;
}

// One launch of the attention kernel: `splits` CTAs per segment.  pdl: the launch may run alongside the one
// before it on the stream.  cluster: the splits of a segment are one thread-block cluster (the merge goes through
// distributed shared memory).
template <int D, int NCW, int SLOTS, bool CLUSTER>
int launch_attend_t(fkv_cache *c, const AttendArgs *a, int splits, bool pdl, cudaStream_t st) {
  const size_t smem = AttendSmem::bytes(D, NCW, SLOTS, CLUSTER);
  auto kern = k_attend<D, NCW, SLOTS, CLUSTER>;
  static SmemOptIn opt_in;
  FKV_CUDA(opt_in.ensure(kern, smem));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(splits, c->cfg.max_batch * c->cfg.num_kv_heads);
  cfg.blockDim = dim3((NCW + 1) * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (pdl || a->wait_first) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  if (CLUSTER) {
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = splits; at[na].val.clusterDim.y = 1; at[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = at;
  cfg.numAttrs = na;
  FKV_CUDA(cudaLaunchKernelEx(&cfg, kern, c->ctx, *a));
  ++c->launches;
  return FKV_OK;
}

// The largest cluster of attention CTAs this device places: 16 (needs the non-portable opt-in), else 8; found once
// per handle.
template <int D, int NCW, int SLOTS>
int attend_max_cluster(fkv_cache *c) {
  auto kern = k_attend<D, NCW, SLOTS, true>;
  const size_t smem = AttendSmem::bytes(D, NCW, SLOTS, true);
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
      cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
    (void)cudaGetLastError();
    return 1;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kClusterSplits, 1);
  cfg.blockDim = dim3((NCW + 1) * 32);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = kClusterSplits; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  int nclusters = 0;
  const bool ok16 = cudaOccupancyMaxActiveClusters(&nclusters, kern, &cfg) == cudaSuccess && nclusters > 0;
  (void)cudaGetLastError();
  return ok16 ? kClusterSplits : 8;
}

int attend_dispatch(fkv_cache *c, const AttendArgs *a, int splits, bool pdl, bool cluster, cudaStream_t st) {
  if (cluster)
    return c->cfg.head_dim == 128 ? launch_attend_t<128, 4, 8, true>(c, a, splits, pdl, st)
                                  : launch_attend_t<64, 4, 16, true>(c, a, splits, pdl, st);
  return c->cfg.head_dim == 128 ? launch_attend_t<128, 4, 8, false>(c, a, splits, pdl, st)
                                : launch_attend_t<64, 4, 16, false>(c, a, splits, pdl, st);
}

// Attention over `layer`, with the new pair of every participating sequence appended first when k_new is given.
int launch_attend(fkv_cache *c, int layer, const void *q, void *out, float scale, const void *k_new, const void *v_new,
                  const int32_t *pos, const SeqMask &seq_mask, bool pdl, cudaStream_t st) {
  const int batch = c->cfg.max_batch, Hkv = c->cfg.num_kv_heads, D = c->cfg.head_dim;
  const bool app = k_new != nullptr;
  int maxpages = 0;
  for (int s = 0; s < batch; ++s) {
    const int n = c->h_len[(size_t)layer * batch + s] + ((app && seq_mask.has(s)) ? 1 : 0);
    maxpages = std::max(maxpages, (n + kPage - 1) / kPage);
  }
  // Splits per segment, at least kAttendMinPages pages each.  Consecutive launches of a decode step share the SMs
  // (three CTAs fit on one): CTAs for about three quarters of the SMs per launch.  A launch on its own has the GPU to
  // itself and lasts as long as its longest CTA: CTAs for every slot of every SM - but never more than
  // kSoloMaxSplits per segment, because the merge in a segment's last CTA grows with the splits (8 segments of 8192
  // pairs: 16.9 us per layer launch at 14 splits, 17.6 at 20, 20.4 at 32; 64 segments of 2K - 16K pairs: 96 us at 2
  // splits, which this rule turns into 7).
  constexpr int kSoloMaxSplits = 14;
  const int nseg = batch * Hkv;
  const int want_ctas = pdl ? c->sm_count * 3 / 4 : c->sm_count * 3;
  // (a launch on its own must fit one wave: rounded down, so that no CTA starts after the others have finished)
  int splits = std::min(c->lay.att_smax, std::max(1, pdl ? (want_ctas + nseg / 2) / nseg : want_ctas / nseg));
  if (!pdl) splits = std::min(splits, kSoloMaxSplits);
  splits = std::max(1, std::min(splits, maxpages / kAttendMinPages));
  // A launch on its own over few segments: the splits of a segment as one cluster of 16 (or 8) CTAs, merged through
  // distributed shared memory.  The cluster size is a power of two; with many segments the global-memory merge
  // above, whose split count is free, fills the GPU better.
  bool cluster = false;
  if (!pdl && nseg * kClusterSplits <= c->sm_count * 3 / 2) {
    if (c->max_cluster == 0)
      c->max_cluster = c->cfg.head_dim == 128 ? attend_max_cluster<128, 4, 8>(c) : attend_max_cluster<64, 4, 16>(c);
    int cs = 1;
    while (cs * 2 <= c->max_cluster && cs * 2 <= kClusterSplits && maxpages / (cs * 2) >= kAttendMinPages) cs *= 2;
    if (cs >= 8) { cluster = true; splits = cs; }
  }
  const int pps = std::max(1, (maxpages + splits - 1) / splits);
  if (scale == 0.f) scale = 1.f / sqrtf((float)D);
  if (app) c->feature_scale = scale;
  AttendArgs a;
  a.layer = layer; a.q = (const __nv_bfloat16 *)q; a.out = (__nv_bfloat16 *)out;
  a.scale_log2 = scale * 1.4426950408889634f; a.pps = pps; a.append = app ? 1 : 0;
  a.k_new = (const uint8_t *)k_new; a.v_new = (const uint8_t *)v_new; a.pos_new = pos; a.seq_mask = seq_mask;
  a.wait_first = pdl ? 0 : 1;
  const int rc = attend_dispatch(c, &a, splits, pdl, cluster, st);
  if (rc) return rc;
  if (app)
    for (int s = 0; s < batch; ++s)
      if (seq_mask.has(s)) ++c->h_len[(size_t)layer * batch + s];
  return FKV_OK;
}

}  // namespace

extern "C" {

int fkv_workspace_bytes(const fkv_config *cfg, size_t *bytes) {
  if (!valid_config(cfg) || !bytes) return FKV_ERR_INVALID_ARG;
  *bytes = make_layout(*cfg).total;
  return FKV_OK;
}

int fkv_init_cache(const fkv_config *cfg, void *dev_workspace, size_t bytes, void *stream, fkv_cache **out) {
  if (!valid_config(cfg) || !dev_workspace || !out) return FKV_ERR_INVALID_ARG;
  if (((uintptr_t)dev_workspace & 255u) != 0) return FKV_ERR_INVALID_ARG;
  const Layout L = make_layout(*cfg);
  if (bytes < L.total) return FKV_ERR_WORKSPACE_TOO_SMALL;
  fkv_cache *c = new (std::nothrow) fkv_cache();
  if (!c) return FKV_ERR_INVALID_ARG;
  c->cfg = *cfg;
  c->lay = L;
  uint8_t *ws = (uint8_t *)dev_workspace;
  Ctx &x = c->ctx;
  x.L = cfg->num_layers; x.Hkv = cfg->num_kv_heads; x.G = cfg->group_size; x.D = cfg->head_dim;
  x.batch = cfg->max_batch; x.act = cfg->activation; x.R = cfg->recent_keep; x.F = L.F;
  x.cap = L.cap; x.max_pages = L.max_pages; x.num_pages = L.num_pages;
  x.page_bytes = L.page_bytes; x.off_v = 2 * cfg->head_dim; x.off_f = 64 * cfg->head_dim;
  x.sp_stride = L.sp_stride; x.sp_off_wf = L.sp_off_wf; x.sp_off_b1 = L.sp_off_b1; x.sp_off_w2 = L.sp_off_w2;
  x.sp_off_b2 = L.sp_off_b2;
  x.pool = ws + L.pool; x.free_stack = (int *)(ws + L.free_stack); x.ctrl = (int *)(ws + L.ctrl);
  x.planhdr = (int *)(ws + L.planhdr); x.pt = (int *)(ws + L.pt); x.pt_new = (int *)(ws + L.pt_new);
  x.len = (int *)(ws + L.len); x.budget = (int *)(ws + L.budget); x.sp = ws + L.sp;
  x.scores = (float *)(ws + L.scores); x.idx = (int *)(ws + L.idx); x.plan = (SegPlan *)(ws + L.plan);
  x.work = (int *)(ws + L.work); x.tile1_start = (int *)(ws + L.tile1);
  x.seq_tickets = (int *)(ws + L.seq_tickets);
  x.seq_fail = (int *)(ws + L.seq_fail);
  x.att_part = (float *)(ws + L.att_part); x.att_tickets = (int *)(ws + L.att_tickets); x.att_smax = L.att_smax;
  x.hist_w = cfg->feature_window; x.hist_q = ws + L.hist_q; x.hist_mp = (float *)(ws + L.hist_mp); x.hist_wp = (cfg->feature_window + 15) & ~15;
  x.hist_n = (int *)(ws + L.hist_n); x.hist_cnt = (int *)(ws + L.hist_cnt);
  c->h_len.assign((size_t)cfg->num_layers * cfg->max_batch, 0);
  c->h_budget.assign(cfg->max_batch, cfg->budget);
  c->loaded.assign((size_t)cfg->num_layers * cfg->num_kv_heads, 0);
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev);
  cudaStream_t st = (cudaStream_t)stream;
  // Zero everything: freshly taken pages then hold finite values in the slots not yet written.
  if (e == cudaSuccess) e = cudaMemsetAsync(ws, 0, L.total, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(x.budget, c->h_budget.data(), (size_t)cfg->max_batch * 4, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    delete c;
    return cuda_fail(e);
  }
  k_reset<<<256, 256, 0, st>>>(c->ctx);
  ++c->launches;
  e = cudaGetLastError();
  if (e != cudaSuccess) {
    delete c;
    return cuda_fail(e);
  }
  *out = c;
  return FKV_OK;
}

int fkv_destroy(fkv_cache *c) {
  if (c)
    for (cudaEvent_t e : c->ev)
      if (e) cudaEventDestroy(e);
  delete c;
  return FKV_OK;
}

int fkv_reset(fkv_cache *c, void *stream) {
  if (!c) return FKV_ERR_INVALID_ARG;
  k_reset<<<256, 256, 0, (cudaStream_t)stream>>>(c->ctx);
  FKV_LAUNCHED(c);
  std::fill(c->h_len.begin(), c->h_len.end(), 0);
  return FKV_OK;
}

int fkv_load_scorer(fkv_cache *c, int layer, int kv_head, const float *W1, const float *b1, const float *W2, float b2,
                    void *stream) {
  if (!c || !layer_ok(c, layer) || kv_head < 0 || kv_head >= c->cfg.num_kv_heads || !W1 || !b1 || !W2)
    return FKV_ERR_INVALID_ARG;
  const int D = c->cfg.head_dim, F = c->lay.F, H = kHidden, KS = 2 * D / 16;
  c->staging.assign(c->lay.sp_stride, 0);
  uint32_t *wkv = (uint32_t *)c->staging.data();
  auto w1 = [&](int row, int col) { return W1[(size_t)row * H + col]; };
  // Part 0 of a weight is its bf16 rounding, part 1 the bf16 rounding of what that left over.
  auto part = [&](int row, int col, int which) {
    const float w = w1(row, col);
    const uint16_t hi = f32_to_bf16_rne(w);
    if (which == 0) return hi;
    if (!std::isfinite(bf16_to_f32(hi))) return (uint16_t)0;   // inf and NaN carry no remainder
    return f32_to_bf16_rne(w - bf16_to_f32(hi));
  };
  auto pack = [&](int row, int col, int which) {
    return (uint32_t)part(row, col, which) | ((uint32_t)part(row + 1, col, which) << 16);
  };
  // mma B fragments (16 x 8, "col"): lane (gid, tig) holds rows k0 + 2 tig (+1) and k0 + 8 + 2 tig (+1) of
  // column gid; registers 0-1 for hidden units 0-7, 2-3 for hidden units 8-15.  All fragments of the
  // roundings first, then all fragments of the remainders.
  for (int which = 0; which < 2; ++which)
    for (int ks = 0; ks < KS; ++ks)
      for (int lane = 0; lane < 32; ++lane) {
        const int gid = lane >> 2, tig = lane & 3, k0 = ks * 16;
        uint32_t *r = wkv + ((size_t)(which * KS + ks) * 32 + lane) * 4;
        r[0] = pack(k0 + 2 * tig, gid, which);
        r[1] = pack(k0 + 8 + 2 * tig, gid, which);
        r[2] = pack(k0 + 2 * tig, 8 + gid, which);
        r[3] = pack(k0 + 8 + 2 * tig, 8 + gid, which);
      }
  // Per quad lane t the hidden units {2t, 2t+1, 8+2t, 9+2t}: the mma accumulator columns that lane owns.
  auto quad = [&](float *dst, auto get) {
    for (int t = 0; t < 4; ++t) {
      dst[t * 4 + 0] = get(2 * t); dst[t * 4 + 1] = get(2 * t + 1);
      dst[t * 4 + 2] = get(8 + 2 * t); dst[t * 4 + 3] = get(9 + 2 * t);
    }
  };
  // Feature rows of W1 as tf32 mma B fragments (8 x 8, "col"): lane (gid, tig) holds rows k0 + tig and k0 + 4 + tig
  // of column gid.  A weight is its truncation to tf32 (10 mantissa bits) plus the truncated remainder; per k-step
  // and lane eight words: truncations for hidden units 0-7 and 8-15, then the remainders.  Rows past F are zero.
  uint32_t *wf = (uint32_t *)(c->staging.data() + c->lay.sp_off_wf);
  auto tf32_part = [&](int row, int col, int which) -> uint32_t {
    if (row >= F) return 0u;
    const float w = w1(2 * D + row, col);
    uint32_t u;
    memcpy(&u, &w, 4);
    const uint32_t t = u & 0xffffe000u;
    if (which == 0) return t;
    float tf;
    memcpy(&tf, &t, 4);
    if (!std::isfinite(tf)) return 0u;
    const float r = w - tf;
    memcpy(&u, &r, 4);
    return u & 0xffffe000u;
  };
  for (int ks = 0; ks < ScoreSmem::fk(F); ++ks)
    for (int lane = 0; lane < 32; ++lane) {
      const int gid = lane >> 2, tig = lane & 3, k0 = ks * 8;
      uint32_t *r = wf + ((size_t)ks * 32 + lane) * 8;
      for (int which = 0; which < 2; ++which) {
        r[which * 4 + 0] = tf32_part(k0 + tig, gid, which);
        r[which * 4 + 1] = tf32_part(k0 + 4 + tig, gid, which);
        r[which * 4 + 2] = tf32_part(k0 + tig, 8 + gid, which);
        r[which * 4 + 3] = tf32_part(k0 + 4 + tig, 8 + gid, which);
      }
    }
  quad((float *)(c->staging.data() + c->lay.sp_off_b1), [&](int j) { return b1[j]; });
  quad((float *)(c->staging.data() + c->lay.sp_off_w2), [&](int j) { return W2[j]; });
  *(float *)(c->staging.data() + c->lay.sp_off_b2) = b2;
  cudaStream_t st = (cudaStream_t)stream;
  FKV_CUDA(cudaMemcpyAsync(c->ctx.sp + ((size_t)layer * c->cfg.num_kv_heads + kv_head) * c->lay.sp_stride,
                           c->staging.data(), c->lay.sp_stride, cudaMemcpyHostToDevice, st));
  FKV_CUDA(cudaStreamSynchronize(st));
  c->loaded[(size_t)layer * c->cfg.num_kv_heads + kv_head] = 1;
  return FKV_OK;
}

int fkv_set_budget(fkv_cache *c, int seq, int32_t budget, void *stream) {
  if (!c || seq < 0 || seq >= c->cfg.max_batch || budget < 1) return FKV_ERR_INVALID_ARG;
  c->h_budget[seq] = budget;
  cudaStream_t st = (cudaStream_t)stream;
  FKV_CUDA(cudaMemcpyAsync(c->ctx.budget + seq, &c->h_budget[seq], 4, cudaMemcpyHostToDevice, st));
  FKV_CUDA(cudaStreamSynchronize(st));
  return FKV_OK;
}

int fkv_prefill(fkv_cache *c, int layer, int seq, const void *k, const void *v, const float *feat, const int32_t *pos,
                int32_t n, void *stream) {
  if (!c || !layer_ok(c, layer) || seq < 0 || seq >= c->cfg.max_batch || !k || !v || n < 1) return FKV_ERR_INVALID_ARG;
  if (n > c->lay.cap) return FKV_ERR_CAPACITY;
  int &hl = c->h_len[(size_t)layer * c->cfg.max_batch + seq];
  if (hl != 0) return FKV_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  k_prefill_alloc<<<1, 1024, 0, st>>>(c->ctx, layer, seq, n);
  FKV_LAUNCHED(c);
  dim3 grid((n + 7) / 8, c->cfg.num_kv_heads);
  k_prefill_rows<0><<<grid, 256, 0, st>>>(c->ctx, layer, seq, n, (const uint8_t *)k, (const uint8_t *)v, feat, pos);
  FKV_LAUNCHED(c);
  hl = n;
  return FKV_OK;
}

int fkv_set_features(fkv_cache *c, int layer, int seq, const float *feat, void *stream) {
  if (!c || !layer_ok(c, layer) || seq < 0 || seq >= c->cfg.max_batch || !feat) return FKV_ERR_INVALID_ARG;
  const int n = c->h_len[(size_t)layer * c->cfg.max_batch + seq];
  if (n == 0) return FKV_OK;
  dim3 grid((n + 7) / 8, c->cfg.num_kv_heads);
  k_prefill_rows<1><<<grid, 256, 0, (cudaStream_t)stream>>>(c->ctx, layer, seq, n, nullptr, nullptr, feat, nullptr);
  FKV_LAUNCHED(c);
  return FKV_OK;
}

int fkv_append(fkv_cache *c, int layer, const void *k, const void *v, const int32_t *pos, const uint64_t *seq_mask,
               void *stream) {
  if (!c || !layer_ok(c, layer) || !k || !v) return FKV_ERR_INVALID_ARG;
  const int batch = c->cfg.max_batch;
  const SeqMask m = make_mask(c, seq_mask);
  for (int s = 0; s < batch; ++s)
    if (m.has(s) && c->h_len[(size_t)layer * batch + s] >= c->lay.cap) return FKV_ERR_CAPACITY;
  k_append<<<batch, 32 * c->cfg.num_kv_heads, 0, (cudaStream_t)stream>>>(c->ctx, layer, (const uint8_t *)k,
                                                                        (const uint8_t *)v, pos, m);
  FKV_LAUNCHED(c);
  for (int s = 0; s < batch; ++s)
    if (m.has(s)) ++c->h_len[(size_t)layer * batch + s];
  return FKV_OK;
}

// Candidates the sampled action needs noise for in one segment: min(2E, competing pairs).
static int sampled_candidates(int n, int B, int R) {
  if (n <= B) return 0;
  return std::min(2 * (n - B), n - std::min(R, B));
}

// score_kind: -1 the learned scorer, 0..5 a feature column (baseline), kScoreRkv the R-KV baseline with its two weights.
constexpr int kScoreRkv = 100;
static int evict_impl(fkv_cache *c, int layer, const float *noise, int noise_stride, int feature_column, float rkv_a,
                      float rkv_s, void *stream) {
  if (!c || (layer != FKV_ALL_LAYERS && !layer_ok(c, layer))) return FKV_ERR_INVALID_ARG;
  const int l0 = layer == FKV_ALL_LAYERS ? 0 : layer, l1 = layer == FKV_ALL_LAYERS ? c->cfg.num_layers : layer + 1;
  const int batch = c->cfg.max_batch, Hkv = c->cfg.num_kv_heads;
  int nactive = 0, max_new = 0, max_old = 0;
  long long tiles = 0;
  for (int l = l0; l < l1; ++l)
    for (int s = 0; s < batch; ++s) {
      const int n = c->h_len[(size_t)l * batch + s], B = c->h_budget[s];
      if (n > B) {
        for (int h = 0; h < Hkv && feature_column < 0; ++h)
          if (!c->loaded[(size_t)l * Hkv + h]) return FKV_ERR_NOT_READY;
        if (noise && sampled_candidates(n, B, c->cfg.recent_keep) > noise_stride) return FKV_ERR_INVALID_ARG;
        nactive += Hkv;
        max_new = std::max(max_new, B);
        max_old = std::max(max_old, n);
        tiles += (long long)Hkv * ((n + kScorePPS * kPage - 1) / (kScorePPS * kPage));
      }
    }
  if (nactive == 0) return FKV_OK;
  cudaStream_t st = (cudaStream_t)stream;
  const bool tm = c->timing;
  if (tm) FKV_CUDA(cudaEventRecord(c->ev[0], st));
  k_plan<<<1, 1024, 0, st>>>(c->ctx, l0, l1, PLAN_EVICT, kScorePPS * kPage, nullptr);
  FKV_LAUNCHED(c);
  if (tm) FKV_CUDA(cudaEventRecord(c->ev[6], st));
  if (c->cfg.feature_window > 0 && c->feature_scale > 0.f) {   // refresh a_n from the chunk's recorded queries first
    const int rcf = launch_features(c, max_old, nactive, st);
    if (rcf) return rcf;
  }
  if (tm) FKV_CUDA(cudaEventRecord(c->ev[1], st));
  int rc = FKV_OK;
  if (feature_column < 0) {
    rc = launch_score_any(c, c->ctx.scores, 0, (int)std::min<long long>(tiles, 1 << 30), st);
  } else if (feature_column == kScoreRkv) {
    rc = launch_rkv(c, c->ctx.scores, 0, max_old, nactive, tiles, rkv_a, rkv_s, st);
  } else {   // a baseline: the score is a feature column
    k_score_feature<<<dim3(nactive, (max_old + 127) / 128), 128, 0, st>>>(c->ctx, c->ctx.scores, 0, feature_column);
    FKV_LAUNCHED(c);
  }
  if (rc) return rc;
  if (tm) FKV_CUDA(cudaEventRecord(c->ev[2], st));
  if (noise) {   // sampled action: scores -> keep-priorities (in place), then the same selection over them
    launch_select(c, 1, max_old, nactive, c->ctx.scores, nullptr, nullptr, 0, 0, c->ctx.scores, noise, noise_stride,
                  l0 * batch * Hkv, st);
    FKV_LAUNCHED(c);
  }
  launch_select(c, 0, max_old, nactive, c->ctx.scores, c->ctx.idx, nullptr, 0, 1, nullptr, nullptr, 0, 0, st);
  FKV_LAUNCHED(c);
  if (tm) FKV_CUDA(cudaEventRecord(c->ev[3], st));
  rc = launch_compact(c, c->ctx.idx, 0, max_new, nactive, st);
  if (rc) return rc;
  if (tm) FKV_CUDA(cudaEventRecord(c->ev[4], st));
  k_commit<<<(l1 - l0) * batch * Hkv, 256, 0, st>>>(c->ctx, l0, l1);
  FKV_LAUNCHED(c);
  if (tm) {
    FKV_CUDA(cudaEventRecord(c->ev[5], st));
    c->timed = true;
  }
  for (int l = l0; l < l1; ++l)
    for (int s = 0; s < batch; ++s) {
      int &n = c->h_len[(size_t)l * batch + s];
      n = std::min(n, c->h_budget[s]);
    }
  return FKV_OK;
}

int fkv_evict(fkv_cache *c, int layer, void *stream) { return evict_impl(c, layer, nullptr, 0, -1, 0.f, 0.f, stream); }

int fkv_evict_by_feature(fkv_cache *c, int layer, int32_t column, void *stream) {
  if (column < 0 || column > 5) return FKV_ERR_INVALID_ARG;
  return evict_impl(c, layer, nullptr, 0, column, 0.f, 0.f, stream);
}

int fkv_evict_rkv(fkv_cache *c, int layer, float lambda_attn, float lambda_sim, void *stream) {
  if (!std::isfinite(lambda_attn) || !std::isfinite(lambda_sim)) return FKV_ERR_INVALID_ARG;
  return evict_impl(c, layer, nullptr, 0, kScoreRkv, lambda_attn, lambda_sim, stream);
}

int fkv_score_rkv(fkv_cache *c, int layer, float lambda_attn, float lambda_sim, float *scores_out, void *stream) {
  if (!c || !layer_ok(c, layer) || !scores_out || !std::isfinite(lambda_attn) || !std::isfinite(lambda_sim))
    return FKV_ERR_INVALID_ARG;
  const int batch = c->cfg.max_batch, Hkv = c->cfg.num_kv_heads;
  long long tiles = 0;
  int max_old = 0;
  for (int s = 0; s < batch; ++s) {
    const int n = c->h_len[(size_t)layer * batch + s];
    tiles += (long long)Hkv * ((n + kScorePPS * kPage - 1) / (kScorePPS * kPage));
    max_old = std::max(max_old, n);
  }
  if (tiles == 0) return FKV_OK;
  cudaStream_t st = (cudaStream_t)stream;
  k_plan<<<1, 1024, 0, st>>>(c->ctx, layer, layer + 1, PLAN_SCORE_ALL, kScorePPS * kPage, nullptr);
  FKV_LAUNCHED(c);
  return launch_rkv(c, scores_out, layer * batch * Hkv, max_old, batch * Hkv, tiles, lambda_attn, lambda_sim, st);
}

int fkv_evict_sampled(fkv_cache *c, int layer, const float *noise, int32_t noise_stride, void *stream) {
  if (!noise || noise_stride < 1) return FKV_ERR_INVALID_ARG;
  return evict_impl(c, layer, noise, noise_stride, -1, 0.f, 0.f, stream);
}

int fkv_decode_attn(fkv_cache *c, int layer, const void *q, void *out, float scale, void *stream) {
  if (!c || !layer_ok(c, layer) || !q || !out) return FKV_ERR_INVALID_ARG;
  return launch_attend(c, layer, q, out, scale, nullptr, nullptr, nullptr, make_mask(c, nullptr), false, (cudaStream_t)stream);
}

int fkv_append_decode_attn(fkv_cache *c, int layer, const void *k, const void *v, const int32_t *pos,
                           const uint64_t *seq_mask, const void *q, void *out, float scale, void *stream) {
  if (!c || !layer_ok(c, layer) || !k || !v || !q || !out) return FKV_ERR_INVALID_ARG;
  const int batch = c->cfg.max_batch;
  const SeqMask m = make_mask(c, seq_mask);
  for (int s = 0; s < batch; ++s)
    if (m.has(s) && c->h_len[(size_t)layer * batch + s] >= c->lay.cap) return FKV_ERR_CAPACITY;
  return launch_attend(c, layer, q, out, scale, k, v, pos, m, false, (cudaStream_t)stream);
}

int fkv_decode_step(fkv_cache *c, const void *k, const void *v, const int32_t *pos, const void *q, void *out,
                    float scale, void *stream) {
  if (!c || !k || !v || !q || !out) return FKV_ERR_INVALID_ARG;
  const int batch = c->cfg.max_batch;
  for (int l = 0; l < c->cfg.num_layers; ++l)
    for (int s = 0; s < batch; ++s)
      if (c->h_len[(size_t)l * batch + s] >= c->lay.cap) return FKV_ERR_CAPACITY;
  const size_t kv_stride = (size_t)batch * c->cfg.num_kv_heads * c->cfg.head_dim * 2;
  const size_t q_stride = kv_stride * c->cfg.group_size;
  const SeqMask all = make_mask(c, nullptr);
  for (int l = 0; l < c->cfg.num_layers; ++l) {
    // Layer l's launch may run alongside layer l - 1's: each touches only its own layer's cache state and
    // tensors.  Layer 0's launch is ordered after everything before it on the stream, as usual.
    const int rc = launch_attend(c, l, (const uint8_t *)q + l * q_stride, (uint8_t *)out + l * q_stride, scale,
                                 (const uint8_t *)k + l * kv_stride, (const uint8_t *)v + l * kv_stride, pos, all, l > 0,
                                 (cudaStream_t)stream);
    if (rc) return rc;
  }
  return FKV_OK;
}

int fkv_update_features(fkv_cache *c, int layer, void *stream) {
  if (!c || !layer_ok(c, layer)) return FKV_ERR_INVALID_ARG;
  if (c->cfg.feature_window == 0) return FKV_ERR_NOT_READY;
  if (c->feature_scale == 0.f) return FKV_OK;   // no query has been recorded yet
  const int batch = c->cfg.max_batch, Hkv = c->cfg.num_kv_heads;
  int max_old = 0;
  for (int s = 0; s < batch; ++s) max_old = std::max(max_old, c->h_len[(size_t)layer * batch + s]);
  if (max_old == 0) return FKV_OK;
  cudaStream_t st = (cudaStream_t)stream;
  k_plan<<<1, 1024, 0, st>>>(c->ctx, layer, layer + 1, PLAN_SCORE_ALL, kScorePPS * kPage, nullptr);
  FKV_LAUNCHED(c);
  return launch_features(c, max_old, batch * Hkv, st);
}

int fkv_score_stride(const fkv_cache *c, int32_t *cap) {
  if (!c || !cap) return FKV_ERR_INVALID_ARG;
  *cap = c->lay.cap;
  return FKV_OK;
}

int fkv_score(fkv_cache *c, int layer, float *scores_out, void *stream) {
  if (!c || !layer_ok(c, layer) || !scores_out) return FKV_ERR_INVALID_ARG;
  const int batch = c->cfg.max_batch, Hkv = c->cfg.num_kv_heads;
  for (int h = 0; h < Hkv; ++h)
    if (!c->loaded[(size_t)layer * Hkv + h]) return FKV_ERR_NOT_READY;
  long long tiles = 0;
  for (int s = 0; s < batch; ++s)
    tiles += (long long)Hkv * ((c->h_len[(size_t)layer * batch + s] + kScorePPS * kPage - 1) / (kScorePPS * kPage));
  if (tiles == 0) return FKV_OK;
  cudaStream_t st = (cudaStream_t)stream;
  k_plan<<<1, 1024, 0, st>>>(c->ctx, layer, layer + 1, PLAN_SCORE_ALL, kScorePPS * kPage, nullptr);
  FKV_LAUNCHED(c);
  return launch_score_any(c, scores_out, layer * batch * Hkv, (int)tiles, st);
}

static int select_impl(fkv_cache *c, int layer, const float *scores_in, const float *noise, int noise_stride,
                       int32_t *idx_out, int32_t *kept_count_out, void *stream) {
  if (!c || !layer_ok(c, layer) || !scores_in || !idx_out || !kept_count_out) return FKV_ERR_INVALID_ARG;
  const int batch = c->cfg.max_batch, Hkv = c->cfg.num_kv_heads;
  if (noise)
    for (int s = 0; s < batch; ++s)
      if (sampled_candidates(c->h_len[(size_t)layer * batch + s], c->h_budget[s], c->cfg.recent_keep) > noise_stride)
        return FKV_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  FKV_CUDA(cudaMemsetAsync(kept_count_out, 0, (size_t)batch * Hkv * 4, st));
  k_plan<<<1, 1024, 0, st>>>(c->ctx, layer, layer + 1, PLAN_SELECT, kScorePPS * kPage, nullptr);
  FKV_LAUNCHED(c);
  int max_old = 0;
  for (int s = 0; s < batch; ++s) max_old = std::max(max_old, c->h_len[(size_t)layer * batch + s]);
  const float *sel_in = scores_in;
  if (noise) {   // keep-priorities go to this layer's part of the workspace scratch
    float *prio = c->ctx.scores + (size_t)layer * batch * Hkv * c->lay.cap;
    launch_select(c, 1, max_old, batch * Hkv, scores_in, nullptr, nullptr, layer * batch * Hkv, 0, prio, noise,
                  noise_stride, layer * batch * Hkv, st);
    FKV_LAUNCHED(c);
    sel_in = prio;
  }
  launch_select(c, 0, max_old, batch * Hkv, sel_in, idx_out, kept_count_out, layer * batch * Hkv, 0, nullptr, nullptr, 0,
                0, st);
  FKV_LAUNCHED(c);
  return FKV_OK;
}

int fkv_select(fkv_cache *c, int layer, const float *scores_in, int32_t *idx_out, int32_t *kept_count_out,
               void *stream) {
  return select_impl(c, layer, scores_in, nullptr, 0, idx_out, kept_count_out, stream);
}

int fkv_select_sampled(fkv_cache *c, int layer, const float *scores_in, const float *noise, int32_t noise_stride,
                       int32_t *idx_out, int32_t *kept_count_out, void *stream) {
  if (!noise || noise_stride < 1) return FKV_ERR_INVALID_ARG;
  return select_impl(c, layer, scores_in, noise, noise_stride, idx_out, kept_count_out, stream);
}

int fkv_compact(fkv_cache *c, int layer, const int32_t *idx, const int32_t *kept_count, void *stream) {
  if (!c || !layer_ok(c, layer) || !idx || !kept_count) return FKV_ERR_INVALID_ARG;
  const int batch = c->cfg.max_batch, Hkv = c->cfg.num_kv_heads;
  int maxn = 0;
  for (int s = 0; s < batch; ++s) maxn = std::max(maxn, c->h_len[(size_t)layer * batch + s]);
  if (maxn == 0) return FKV_OK;
  cudaStream_t st = (cudaStream_t)stream;
  k_plan<<<1, 1024, 0, st>>>(c->ctx, layer, layer + 1, PLAN_COMPACT, kScorePPS * kPage, kept_count);
  FKV_LAUNCHED(c);
  k_fill_pt_new<<<batch * Hkv, 256, 0, st>>>(c->ctx, layer * batch * Hkv, batch * Hkv);
  FKV_LAUNCHED(c);
  int rc = launch_compact(c, idx, layer * batch * Hkv, maxn, batch * Hkv, st);
  if (rc) return rc;
  k_commit<<<batch * Hkv, 256, 0, st>>>(c->ctx, layer, layer + 1);
  FKV_LAUNCHED(c);
  FKV_CUDA(cudaMemcpyAsync(&c->h_len[(size_t)layer * batch], c->ctx.len + (size_t)layer * batch, (size_t)batch * 4,
                           cudaMemcpyDeviceToHost, st));
  FKV_CUDA(cudaStreamSynchronize(st));
  return FKV_OK;
}

int fkv_export_head(fkv_cache *c, int layer, int seq, int kv_head, void *k, void *v, float *feat, int32_t *pos,
                    void *stream) {
  if (!c || !layer_ok(c, layer) || seq < 0 || seq >= c->cfg.max_batch || kv_head < 0 || kv_head >= c->cfg.num_kv_heads)
    return FKV_ERR_INVALID_ARG;
  const int n = c->h_len[(size_t)layer * c->cfg.max_batch + seq];
  if (n == 0) return FKV_OK;
  k_export_rows<<<(n + 7) / 8, 256, 0, (cudaStream_t)stream>>>(c->ctx, layer, seq, kv_head, (uint8_t *)k, (uint8_t *)v,
                                                               feat, pos);
  FKV_LAUNCHED(c);
  return FKV_OK;
}

int fkv_get_lengths(const fkv_cache *c, int layer, int32_t *host_out) {
  if (!c || !layer_ok(c, layer) || !host_out) return FKV_ERR_INVALID_ARG;
  for (int s = 0; s < c->cfg.max_batch; ++s) host_out[s] = c->h_len[(size_t)layer * c->cfg.max_batch + s];
  return FKV_OK;
}

int fkv_device_status(fkv_cache *c, uint32_t *status_bits, int32_t *free_pages, void *stream) {
  if (!c) return FKV_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int h[2] = {0, 0};
  FKV_CUDA(cudaMemcpyAsync(h, c->ctx.ctrl, 8, cudaMemcpyDeviceToHost, st));
  FKV_CUDA(cudaStreamSynchronize(st));
  if (h[CTRL_STATUS]) {
    FKV_CUDA(cudaMemsetAsync(c->ctx.ctrl + CTRL_STATUS, 0, 4, st));
    FKV_CUDA(cudaStreamSynchronize(st));
  }
  if (status_bits) *status_bits = (uint32_t)h[CTRL_STATUS];
  if (free_pages) *free_pages = h[CTRL_FREE_TOP];
  return h[CTRL_STATUS] ? FKV_ERR_DEVICE : FKV_OK;
}

int fkv_sync_lengths(fkv_cache *c, void *stream) {
  if (!c) return FKV_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  FKV_CUDA(cudaMemcpyAsync(c->h_len.data(), c->ctx.len, c->h_len.size() * 4, cudaMemcpyDeviceToHost, st));
  FKV_CUDA(cudaStreamSynchronize(st));
  return FKV_OK;
}

int fkv_set_timing(fkv_cache *c, int on) {
  if (!c) return FKV_ERR_INVALID_ARG;
  if (on)
    for (cudaEvent_t &e : c->ev)
      if (!e) FKV_CUDA(cudaEventCreate(&e));
  c->timing = on != 0;
  c->timed = false;
  return FKV_OK;
}

int fkv_get_evict_timing(fkv_cache *c, float ms_out[6]) {
  if (!c || !ms_out) return FKV_ERR_INVALID_ARG;
  if (!c->timed) return FKV_ERR_NOT_READY;
  FKV_CUDA(cudaEventSynchronize(c->ev[5]));
  for (int i = 0; i < 5; ++i) FKV_CUDA(cudaEventElapsedTime(&ms_out[i], c->ev[i], c->ev[i + 1]));
  FKV_CUDA(cudaEventElapsedTime(&ms_out[5], c->ev[6], c->ev[1]));   // feature refresh: after the plan, before the scorer
  ms_out[0] -= ms_out[5];
  return FKV_OK;
}

int fkv_launch_count(const fkv_cache *c, uint64_t *launches) {
  if (!c || !launches) return FKV_ERR_INVALID_ARG;
  *launches = c->launches;
  return FKV_OK;
}

static int golden_select_launch(const float *alpha, int T, int B, int L, int M, int32_t *kept, cudaStream_t st) {
  if (B > 8192) return FKV_ERR_CAPACITY;   // eight cache entries per thread
  const size_t smem = (size_t)B * 4;
  k_golden_select<<<1, 1024, smem, st>>>(alpha, T, B, L, M, kept);
  FKV_CUDA(cudaGetLastError());
  return FKV_OK;
}

int fkv_golden_steps(int32_t T, int32_t B, int32_t L) {
  if (T < 1 || B < 2 || L < 1 || L >= B) return FKV_ERR_INVALID_ARG;
  const int M = (T - B + L - 1) / L - 1;
  return M < 0 ? 0 : M;
}

int fkv_golden_select(const float *alpha, int32_t T, int32_t B, int32_t L, int32_t M, int32_t *kept_out, void *stream) {
  if (!alpha || !kept_out || M < 1 || fkv_golden_steps(T, B, L) < M) return FKV_ERR_INVALID_ARG;
  return golden_select_launch(alpha, T, B, L, M, kept_out, (cudaStream_t)stream);
}

int fkv_golden_eviction(const float *attn, int32_t g, int32_t T, int32_t B, int32_t L, float *alpha_out,
                        int32_t *kept_out, void *stream) {
  if (!attn || !alpha_out || !kept_out || g < 1) return FKV_ERR_INVALID_ARG;
  const int M = fkv_golden_steps(T, B, L);
  if (M < 0) return M;
  if (M == 0) return FKV_OK;
  if (B > 8192) return FKV_ERR_CAPACITY;
  cudaStream_t st = (cudaStream_t)stream;
  k_golden_pool<<<dim3((T + 255) / 256, M), 256, 0, st>>>(attn, g, T, B, L, alpha_out);
  FKV_CUDA(cudaGetLastError());
  k_golden_suffix_max<<<(T + 255) / 256, 256, 0, st>>>(alpha_out, T, M);
  FKV_CUDA(cudaGetLastError());
  return golden_select_launch(alpha_out, T, B, L, M, kept_out, st);
}

const char *fkv_last_cuda_error(void) { return g_cuda_error.c_str(); }

}  // extern "C"
