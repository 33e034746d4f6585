// Cache bookkeeping kernels: reset, bulk load, append, dense export, the
// planner that sizes an eviction step on the device, and the commit that
// swaps page tables afterwards.  Pages are handed out from a LIFO free stack
// that lives on the device, so no step needs a host round trip.
#pragma once
#include "fkv_dev.cuh"

namespace fkv {

// ---------------------------------------------------------------- reset
__global__ void k_reset(Ctx c) {
  const int stride = gridDim.x * blockDim.x, t0 = blockIdx.x * blockDim.x + threadIdx.x;
  for (int i = t0; i < c.num_pages; i += stride) c.free_stack[i] = c.num_pages - 1 - i;
  for (int i = t0; i < c.L * c.batch; i += stride) c.len[i] = 0;
  for (int i = t0; i < c.L * c.batch; i += stride) c.seq_tickets[i] = 0;
  for (int i = t0; i < c.L * c.batch * c.Hkv; i += stride) c.att_tickets[i] = 0;
  for (int i = t0; i < c.L * c.batch; i += stride) c.seq_fail[i] = 0;
  if (c.hist_w)
    for (int i = t0; i < c.L * c.batch; i += stride) c.hist_cnt[i] = 0;
  if (t0 == 0) {
    c.ctrl[CTRL_FREE_TOP] = c.num_pages;
    c.ctrl[CTRL_STATUS] = 0;
  }
}

// ---------------------------------------------------------------- prefill
// Takes Hkv * ceil(n/16) pages for one empty (layer, seq) and sets its length.
__global__ void k_prefill_alloc(Ctx c, int layer, int seq, int n) {
  __shared__ int s_top;
  const int cnt = (n + kPage - 1) / kPage, total = cnt * c.Hkv;
  if (threadIdx.x == 0) {
    int top = c.ctrl[CTRL_FREE_TOP];
    if (c.len[layer * c.batch + seq] != 0 || total > top) {
      set_status(c, total > top ? kDevPoolExhausted : kDevCapacity);
      s_top = -1;
    } else {
      s_top = top;
    }
  }
  __syncthreads();
  const int top = s_top;
  if (top < 0) return;
  for (int i = threadIdx.x; i < total; i += blockDim.x) {
    const int h = i / cnt, j = i - h * cnt;
    c.pt[(size_t)seg_of(c, layer, seq, h) * c.max_pages + j] = c.free_stack[top - 1 - i];
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    c.ctrl[CTRL_FREE_TOP] = top - total;
    c.len[layer * c.batch + seq] = n;
  }
}

// grid (ceil(n / 8), Hkv), 256 threads: one warp per pair.  MODE 0: load K, V,
// features, positions; MODE 1: overwrite features only.
template <int MODE>
__global__ void k_prefill_rows(Ctx c, int layer, int seq, int n, const uint8_t *k, const uint8_t *v, const float *feat,
                               const int32_t *pos) {
  if (c.len[layer * c.batch + seq] != n) return;  // allocation failed or wrong length
  const int lane = threadIdx.x & 31, i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), h = blockIdx.y;
  if (i >= n) return;
  const int seg = seg_of(c, layer, seq, h);
  uint8_t *page = c.pool + (size_t)c.pt[(size_t)seg * c.max_pages + i / kPage] * c.page_bytes;
  const size_t row = (size_t)h * n + i;
  if (MODE == 0) {
    move_row<0>(c, page, i % kPage, const_cast<uint8_t *>(k) + row * c.D * 2, const_cast<uint8_t *>(v) + row * c.D * 2,
                feat ? const_cast<float *>(feat) + row * c.F : nullptr, pos ? const_cast<int32_t *>(pos) + i : nullptr,
                lane, i);
  } else {
    float *pf = meta_row(c, page, i % kPage);
    for (int f = lane; f < c.F; f += 32) pf[f] = feat[row * c.F + f];
  }
}

// grid ceil(n / 8): dense copy of one segment.
__global__ void k_export_rows(Ctx c, int layer, int seq, int head, uint8_t *k, uint8_t *v, float *feat, int32_t *pos) {
  const int n = c.len[layer * c.batch + seq];
  const int lane = threadIdx.x & 31, i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (i >= n) return;
  const int seg = seg_of(c, layer, seq, head);
  uint8_t *page = c.pool + (size_t)c.pt[(size_t)seg * c.max_pages + i / kPage] * c.page_bytes;
  move_row<1>(c, page, i % kPage, k ? k + (size_t)i * c.D * 2 : nullptr, v ? v + (size_t)i * c.D * 2 : nullptr,
              feat ? feat + (size_t)i * c.F : nullptr, pos ? pos + i : nullptr, lane, 0);
}

// ---------------------------------------------------------------- append
// grid = batch, block = 32 * Hkv: one warp per KV head writes the new pair at
// slot n; a new page per head is popped from the free stack when n % 16 == 0.
__global__ void k_append(Ctx c, int layer, const uint8_t *k, const uint8_t *v, const int32_t *pos, SeqMask seq_mask) {
  __shared__ int s_top;
  const int seq = blockIdx.x, lane = threadIdx.x & 31, h = threadIdx.x >> 5;
  if (!seq_mask.has(seq)) return;
  const int n = c.len[layer * c.batch + seq];
  if (n >= c.cap) {
    if (threadIdx.x == 0) set_status(c, kDevCapacity);
    return;
  }
  const bool need_page = (n % kPage) == 0;
  if (need_page) {
    if (threadIdx.x == 0) {
      int old = atomicSub(&c.ctrl[CTRL_FREE_TOP], c.Hkv);
      if (old < c.Hkv) {
        atomicAdd(&c.ctrl[CTRL_FREE_TOP], c.Hkv);
        set_status(c, kDevPoolExhausted);
        old = -1;
      }
      s_top = old;
    }
    __syncthreads();
    if (s_top < 0) return;
  }
  const int seg = seg_of(c, layer, seq, h);
  int *ptrow = c.pt + (size_t)seg * c.max_pages;
  int pid;
  if (need_page) {
    pid = c.free_stack[s_top - 1 - h];
    if (lane == 0) ptrow[n / kPage] = pid;
  } else {
    pid = ptrow[n / kPage];
  }
  int32_t pdef = 0;
  if (!pos && n > 0) {
    const uint8_t *prev = c.pool + (size_t)ptrow[(n - 1) / kPage] * c.page_bytes;
    pdef = reinterpret_cast<const int32_t *>(meta_row(c, prev, (n - 1) % kPage))[c.F] + 1;
  }
  const size_t row = (size_t)seq * c.Hkv + h;
  move_row<0>(c, c.pool + (size_t)pid * c.page_bytes, n % kPage, const_cast<uint8_t *>(k) + row * c.D * 2,
              const_cast<uint8_t *>(v) + row * c.D * 2, nullptr, pos ? const_cast<int32_t *>(pos) + seq : nullptr, lane,
              pdef);
  __syncthreads();
  if (threadIdx.x == 0) c.len[layer * c.batch + seq] = n + 1;
}

// ---------------------------------------------------------------- plan
// One block sizes the step for segments of layers [l0, l1): which segments
// take part, their counts, the score-tile prefix, and - when the step
// compacts - one batch of fresh pages per segment, reserved at the top of the
// free stack (offset pad0 of its plan entry).  Everything later kernels need comes from
// here, so the host never reads a length back.
enum { PLAN_EVICT = 0, PLAN_SCORE_ALL = 1, PLAN_SELECT = 2, PLAN_COMPACT = 3 };

__global__ void __launch_bounds__(1024) k_plan(Ctx c, int l0, int l1, int mode, int tile_pairs,
                                                const int32_t *kept_count /* PLAN_COMPACT: [batch][Hkv] */) {
  __shared__ int s_scan[33];
  __shared__ int s_fail;
  const int seg0 = l0 * c.batch * c.Hkv, nseg = (l1 - l0) * c.batch * c.Hkv;
  int carry_work = 0, carry_tiles = 0, carry_new = 0, carry_old = 0;
  if (threadIdx.x == 0) s_fail = 0;
  __syncthreads();
  for (int base = 0; base < nseg; base += blockDim.x) {
    const int i = base + threadIdx.x, seg = seg0 + i;
    int n = 0, n_new = 0, r = 0, k = 0, active = 0, is_work = 0, tiles = 0;
    if (i < nseg) {
      const int ls = seg / c.Hkv, seq = ls % c.batch;
      n = c.len[ls];
      const int B = c.budget[seq];
      n_new = n < B ? n : B;
      if (mode == PLAN_COMPACT) n_new = kept_count[(seq * c.Hkv) + seg % c.Hkv];
      if (n_new > n || n_new < 0) { n_new = n; atomicOr(&s_fail, (int)kDevBadIndex); }
      r = c.R < n_new ? c.R : n_new;
      k = n_new - r;
      active = (mode == PLAN_EVICT || mode == PLAN_COMPACT) && n_new < n;
      is_work = (mode == PLAN_EVICT || mode == PLAN_COMPACT) ? active : n > 0;
      tiles = is_work ? (n + tile_pairs - 1) / tile_pairs : 0;
    }
    const int new_pages = active ? (n_new + kPage - 1) / kPage : 0;
    const int old_pages = active ? (n + kPage - 1) / kPage : 0;
    int tot;
    const int w_off = carry_work + block_excl_scan(is_work, s_scan, tot); carry_work += tot;
    const int t_off = carry_tiles + block_excl_scan(tiles, s_scan, tot); carry_tiles += tot;
    const int n_off = carry_new + block_excl_scan(new_pages, s_scan, tot); carry_new += tot;
    const int o_off = carry_old + block_excl_scan(old_pages, s_scan, tot); carry_old += tot;
    if (i < nseg) {
      SegPlan p;
      p.n_old = n; p.n_new = n_new; p.r = r; p.k_sel = k; p.active = active; p.push_base = o_off;
      p.pad0 = n_off;  // offset of this segment's fresh pages inside the batch taken from the stack
      p.pad1 = 0;
      c.plan[seg] = p;
      if (is_work) { c.work[w_off] = seg; c.tile1_start[w_off] = t_off; }
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) s_scan[0] = c.ctrl[CTRL_FREE_TOP];
  __syncthreads();
  const int top = s_scan[0];
  const bool exhausted = carry_new > top;
  if (exhausted || s_fail) {
    // Not enough pages (or bad counts): make the whole step a no-op.
    if (threadIdx.x == 0) {
      set_status(c, exhausted ? kDevPoolExhausted : (unsigned)s_fail);
      c.planhdr[PH_NWORK] = 0; c.planhdr[PH_TILES1] = 0; c.planhdr[PH_NEW_PAGES] = 0; c.planhdr[PH_OLD_PAGES] = 0;
      c.planhdr[PH_PUSH_START] = top;
    }
    for (int i = threadIdx.x; i < nseg; i += blockDim.x) c.plan[seg0 + i].active = 0;
    return;
  }
  if (threadIdx.x == 0) {
    c.tile1_start[carry_work] = carry_tiles;
    c.planhdr[PH_NWORK] = carry_work; c.planhdr[PH_TILES1] = carry_tiles;
    c.planhdr[PH_NEW_PAGES] = carry_new; c.planhdr[PH_OLD_PAGES] = carry_old;
    c.planhdr[PH_PUSH_START] = top - carry_new;
  }
  // The fresh page ids stay on the stack above the new top until the selection kernel (or
  // k_fill_pt_new) copies each segment's batch into pt_new; the commit pushes old pages only after that.
  if (carry_new > 0 && threadIdx.x == 0) c.ctrl[CTRL_FREE_TOP] = top - carry_new;
}

// ---------------------------------------------------------------- commit
// grid = segments of the call, 256 threads: push the old pages of every
// compacted segment back on the free stack, install its new page table and
// length.  The push region starts where the fresh pages were taken from.
__global__ void k_commit(Ctx c, int l0, int l1) {
  const int nseg = (l1 - l0) * c.batch * c.Hkv, seg = l0 * c.batch * c.Hkv + blockIdx.x;
  if ((int)blockIdx.x >= nseg) return;
  if (blockIdx.x == 0 && threadIdx.x == 0 && c.planhdr[PH_OLD_PAGES] > 0)
    c.ctrl[CTRL_FREE_TOP] = c.planhdr[PH_PUSH_START] + c.planhdr[PH_OLD_PAGES];
  const SegPlan p = c.plan[seg];
  if (!p.active) return;
  const int cnt_old = (p.n_old + kPage - 1) / kPage, cnt_new = (p.n_new + kPage - 1) / kPage;
  const int push = c.planhdr[PH_PUSH_START] + p.push_base;
  int *ptrow = c.pt + (size_t)seg * c.max_pages;
  const int *ptnew = c.pt_new + (size_t)seg * c.max_pages;
  for (int i = threadIdx.x; i < cnt_old; i += blockDim.x) {
    c.free_stack[push + i] = ptrow[i];
    if (i < cnt_new) ptrow[i] = ptnew[i];
  }
  if (threadIdx.x == 0 && seg % c.Hkv == 0) {
    c.len[seg / c.Hkv] = p.n_new;
    if (c.hist_w) c.hist_cnt[seg / c.Hkv] = 0;   // the eviction closed the chunk: its query record starts over
  }
}

}  // namespace fkv
