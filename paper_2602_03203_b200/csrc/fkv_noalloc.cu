// fkv_decode_attn_dense_noalloc: split-K GQA decode attention for callers that
// cannot allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a
// memory pool that has been frozen after start-up, under a serving process
// that accounts every byte of HBM itself, or in a plug-in that is handed a few
// tensors and nothing else.  The regular path keeps its split-K partials in a
// workspace the caller allocates; this entry point needs no workspace at all.
// The partials live in a fixed array that is part of the library image, so
// every GPU that loads the library holds kScratchBytes (about 1.1 MB) until
// the process exits, whether or not this entry point is ever called.
//
// It is the same split-K scheme as the paged kernel (per-split online softmax,
// an (m, l, O) partial per split, the last split to finish merges - by atomic
// ticket, nobody waits), written for dense K and V with plain loads.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <mutex>

#include "../../include/fkv.h"

namespace fkv {
void note_cuda_error(cudaError_t e);   // fkv_api.cu: keeps the text fkv_last_cuda_error returns
}

namespace fkv_noalloc {

constexpr int kMaxHeads = 16;    // KV heads per call
constexpr int kMaxSplits = 16;   // splits per KV head
constexpr int kMaxG = 8;         // query heads per KV head
constexpr int kMaxD = 128;
constexpr int kRowFloats = kMaxD + 2;  // O row, then m and l
constexpr size_t kPartFloats = (size_t)kMaxHeads * kMaxSplits * kMaxG * kRowFloats;
constexpr size_t kScratchBytes = kPartFloats * sizeof(float) + kMaxHeads * sizeof(int);
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for
// cudaGetSymbolAddress; device code may use it directly.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// CPL consecutive bf16 channels (CPL * 2 bytes, aligned to that) as floats.
template <int CPL>
__device__ __forceinline__ void load_channels(const __nv_bfloat16 *p, float (&x)[CPL]) {
  static_assert(CPL == 2 || CPL == 4, "head_dim 64 or 128");
  if (CPL == 2) {
    const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(p));
    x[0] = f.x; x[1] = f.y;
  } else {
    const uint2 u = *reinterpret_cast<const uint2 *>(p);
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&u.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&u.y));
    x[0] = a.x; x[1] = a.y; x[CPL - 2] = b.x; x[CPL - 1] = b.y;
  }
}

// grid (splits, Hkv), 128 threads.  CPL = channels per lane = D / 32.  A service path, not a tuned one: a warp
// reads one row per step (256 bytes), far below the paged kernel's rate for long sequences.
template <int CPL>
__global__ void __launch_bounds__(128) k_attend_dense(const __nv_bfloat16 *q, const __nv_bfloat16 *k,
                                                      const __nv_bfloat16 *v, int n, int G, float scale_log2,
                                                      __nv_bfloat16 *out, float *part, int *tickets) {
  constexpr int D = CPL * 32;
  __shared__ float s_o[4][kMaxG][D];
  __shared__ float s_ml[4][kMaxG][2];
  __shared__ int s_last;
  const int head = blockIdx.y, ns = gridDim.x, split = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int per = (n + ns - 1) / ns, i0 = split * per, i1 = min(n, i0 + per);
  const __nv_bfloat16 *kh = k + (size_t)head * n * D, *vh = v + (size_t)head * n * D;

  float qr[kMaxG][CPL], o[kMaxG][CPL], m[kMaxG], l[kMaxG];
#pragma unroll
  for (int h = 0; h < kMaxG; ++h) {
    m[h] = -INFINITY; l[h] = 0.f;
#pragma unroll
    for (int c = 0; c < CPL; ++c) {
      o[h][c] = 0.f;
      qr[h][c] = h < G ? __bfloat162float(q[((size_t)head * G + h) * D + lane * CPL + c]) : 0.f;
    }
  }
  for (int i = i0 + warp; i < i1; i += 4) {
    float kr[CPL], vr[CPL];
    load_channels<CPL>(kh + (size_t)i * D + lane * CPL, kr);   // one 4- or 8-byte load per lane and tensor
    load_channels<CPL>(vh + (size_t)i * D + lane * CPL, vr);
#pragma unroll
    for (int h = 0; h < kMaxG; ++h) {
      if (h >= G) break;
      float d = 0.f;
#pragma unroll
      for (int c = 0; c < CPL; ++c) d = fmaf(qr[h][c], kr[c], d);
      const float s = warp_sum(d) * scale_log2;
      const float mn = fmaxf(m[h], s), corr = exp2f(m[h] - mn), p = exp2f(s - mn);
      l[h] = l[h] * corr + p;
      m[h] = mn;
#pragma unroll
      for (int c = 0; c < CPL; ++c) o[h][c] = fmaf(p, vr[c], o[h][c] * corr);
    }
  }
  for (int h = 0; h < G; ++h) {
#pragma unroll
    for (int c = 0; c < CPL; ++c) s_o[warp][h][lane * CPL + c] = o[h][c];
    if (lane == 0) { s_ml[warp][h][0] = m[h]; s_ml[warp][h][1] = l[h]; }
  }
  __syncthreads();
  // Merge the four warps into this split's partial.
  float *mypart = part + ((size_t)head * kMaxSplits + split) * kMaxG * kRowFloats;
  for (int e = threadIdx.x; e < G * D; e += blockDim.x) {
    const int h = e / D, ch = e - h * D;
    float M = -INFINITY;
    for (int w = 0; w < 4; ++w) M = fmaxf(M, s_ml[w][h][0]);
    float acc = 0.f, L = 0.f;
    for (int w = 0; w < 4; ++w) {
      const float f = s_ml[w][h][0] == -INFINITY ? 0.f : exp2f(s_ml[w][h][0] - M);
      acc += f * s_o[w][h][ch];
      L += f * s_ml[w][h][1];
    }
    mypart[h * kRowFloats + ch] = acc;
    if (ch == 0) { mypart[h * kRowFloats + D] = M; mypart[h * kRowFloats + D + 1] = L; }
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int t = atomicAdd(&tickets[head], 1);
    s_last = t == ns - 1;
    if (s_last) tickets[head] = 0;  // ready for the next call
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const float *hp = part + (size_t)head * kMaxSplits * kMaxG * kRowFloats;
  for (int e = threadIdx.x; e < G * D; e += blockDim.x) {
    const int h = e / D, ch = e - h * D;
    float M = -INFINITY;
    for (int s = 0; s < ns; ++s) M = fmaxf(M, __ldcg(hp + ((size_t)s * kMaxG + h) * kRowFloats + D));
    float acc = 0.f, L = 0.f;
    for (int s = 0; s < ns; ++s) {
      const float *row = hp + ((size_t)s * kMaxG + h) * kRowFloats;
      const float ms = __ldcg(row + D);
      const float f = ms == -INFINITY ? 0.f : exp2f(ms - M);
      acc += f * __ldcg(row + ch);
      L += f * __ldcg(row + D + 1);
    }
    out[((size_t)head * G + h) * D + ch] = __float2bfloat16(L > 0.f ? acc / L : 0.f);
  }
}

// Device address of g_scratch per device, resolved once per device.
std::mutex g_mu;
void *g_addr[kMaxDevices];

cudaError_t scratch_address(void **out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_addr[dev]) {
    void *p = nullptr;
    e = cudaGetSymbolAddress(&p, g_scratch);  // the current device's copy of the array
    if (e != cudaSuccess) return e;
    g_addr[dev] = p;
  }
  *out = g_addr[dev];
  return cudaSuccess;
}

}  // namespace fkv_noalloc

extern "C" int fkv_decode_attn_dense_noalloc(const void *q, const void *k, const void *v, int32_t n,
                                             int32_t num_kv_heads, int32_t group_size, int32_t head_dim, float scale,
                                             void *out, void *stream) {
  using namespace fkv_noalloc;
  if (!q || !k || !v || !out) return FKV_ERR_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return FKV_ERR_INVALID_ARG;
  if (n < 1 || n > FKV_NOALLOC_MAX_PAIRS) return FKV_ERR_CAPACITY;
  if (num_kv_heads < 1 || num_kv_heads > FKV_NOALLOC_MAX_KV_HEADS) return FKV_ERR_CAPACITY;
  if (group_size < 1 || group_size > kMaxG) return FKV_ERR_CAPACITY;
  static_assert(FKV_NOALLOC_MAX_KV_HEADS == kMaxHeads, "header and kernel disagree");
  // k and v are read with one 8-byte (head_dim 128) or 4-byte (64) load per lane.
  if ((((uintptr_t)k | (uintptr_t)v) & 7u) != 0) return FKV_ERR_INVALID_ARG;
  auto failed = [](cudaError_t e) {
    fkv::note_cuda_error(e);
    return (int)FKV_ERR_CUDA;
  };
  void *base = nullptr;
  cudaError_t err = scratch_address(&base);
  if (err != cudaSuccess) return failed(err);
  float *part = (float *)base;
  int *tickets = (int *)((unsigned char *)base + kPartFloats * sizeof(float));
  cudaStream_t st = (cudaStream_t)stream;
  // The array keeps whatever the last call left; only the tickets must start at zero.
  err = cudaMemsetAsync(tickets, 0, kMaxHeads * sizeof(int), st);
  if (err != cudaSuccess) return failed(err);
  int splits = (n + 255) / 256;
  splits = splits < 1 ? 1 : (splits > kMaxSplits ? kMaxSplits : splits);
  if (scale == 0.f) scale = 1.f / sqrtf((float)head_dim);
  const float scale_log2 = scale * 1.4426950408889634f;
  dim3 grid(splits, num_kv_heads);
  if (head_dim == 128)
    k_attend_dense<4><<<grid, 128, 0, st>>>((const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k,
                                            (const __nv_bfloat16 *)v, n, group_size, scale_log2, (__nv_bfloat16 *)out,
                                            part, tickets);
  else
    k_attend_dense<2><<<grid, 128, 0, st>>>((const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k,
                                            (const __nv_bfloat16 *)v, n, group_size, scale_log2, (__nv_bfloat16 *)out,
                                            part, tickets);
  err = cudaGetLastError();
  return err == cudaSuccess ? (int)FKV_OK : failed(err);
}
