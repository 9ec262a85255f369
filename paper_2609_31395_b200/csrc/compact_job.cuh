// The plan of a fresh-page compaction (Section 7.2 / Algorithm 4: plan first, then one-shot copies whose
// sources and destinations are disjoint) as a work queue in device memory, and the warp-level routine that
// executes one item of it.  An item is 32 consecutive (slot, head) pairs of one destination page of one
// request in one layer: the K row and the V row of each (16 KB in, 16 KB out at head_dim 128).  Because the copies are order-free and touch nothing the
// score kernels read or write (sources: old pages of layers already scored and selected; destinations:
// pages still on the free list), any warp of any kernel may execute items: the spare warps of the
// tensor-core pooled-score kernel of the NEXT layer group do (it leaves most of the HBM bandwidth idle),
// and a drain kernel takes whatever is left.
#pragma once

#include "common.cuh"

namespace actkv {

struct CompactWs {
  int32_t plan_ok;       // 1 when the copy / finalize kernels may run
  int32_t total_new;     // pages popped
  uint32_t next_item;    // deferred copy: items handed out so far (atomic counter)
  int32_t n_items;       // deferred copy: total_new x layers x parts_per_page; 0 when the job is not deferred
  // the job as the plan kernel recorded it, for whoever executes items
  PoolView pool;
  TablesView tab;
  const int32_t* sel_idx;
  int64_t sel_stride;
  const int32_t* keep_indptr;
  const int32_t* budget;
  int32_t* status;
  int32_t layer_begin, n_layers;
  int32_t vpr_shift;     // log2 of the 16-byte vectors per row (3, 4, 5 for head_dim 64, 128, 256); -1: not deferrable
  int32_t parts_per_page;  // items per destination page: ceil(page_size x heads / 32)
  int32_t role_items;    // items executed by copy roles of other kernels (the rest went to the drain kernel)
  int32_t pad;           // CJ_PLAN_MARK / CJ_INPLACE_MARK once a plan kernel has written this workspace
  uint32_t* src_tab;     // deferred copy: resolved sources, [n_items][32] (see cj_resolve_item)
  uint32_t* dst_tab;     // deferred in-place copy: resolved destinations, [n_items][32]; nullptr for the fresh-page form,
                         // whose destinations follow from the item number
  int32_t items_per_slab;  // items of one layer (>= 1): the layer of an item is item / items_per_slab
  int32_t pad2;
  // followed by int32 new_off[R], push_off[R], item_off[R + 1], new_pages[R * max_pages]
};

__host__ __device__ __forceinline__ int32_t* ws_new_off(CompactWs* w) { return reinterpret_cast<int32_t*>(w + 1); }
__host__ __device__ __forceinline__ int32_t* ws_push_off(CompactWs* w, int R) { return ws_new_off(w) + R; }
__host__ __device__ __forceinline__ int32_t* ws_item_off(CompactWs* w, int R) { return ws_new_off(w) + 2 * R; }
__host__ __device__ __forceinline__ int32_t* ws_new_pages(CompactWs* w, int R) { return ws_new_off(w) + 3 * R + 1; }

constexpr uint32_t CJ_NONE = 0xffffffffu;
constexpr int32_t CJ_PLAN_MARK = 0x414b5650;      // a fresh-page plan
constexpr int32_t CJ_INPLACE_MARK = 0x414b5649;   // an in-place job

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.cs.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Hands out the next item of the queue to this warp: the value every lane returns is the item number, which is
// only valid when below cj_count().  The atomic's round trip is hidden by asking one item ahead.
__device__ __forceinline__ uint32_t cj_pop(CompactWs* w, int lane) {
  uint32_t it = 0;
  if (lane == 0) it = atomicAdd(&w->next_item, 1u);
  return __shfl_sync(0xffffffffu, it, 0);
}
__device__ __forceinline__ uint32_t cj_count(const CompactWs* w) { return w->plan_ok ? (uint32_t)w->n_items : 0u; }

// Where the rows of one item come from, resolved once per job by compact_resolve_kernel so that whoever
// executes the item starts its loads after a single lookup:
//   src_tab[item * 32 + lane] = source of (slot, head) pair lane + 32 * part of the item's destination page, as a
//   16-byte-unit offset within the layer, or CJ_NONE (past the end of the page, or a move that was dropped).
// item = (slab * total_new + page) * parts_per_page + part, page = index into the run of new pages.
__device__ __forceinline__ void cj_resolve_item(CompactWs* w, int item, int lane) {
  const PoolView& pool = w->pool;
  const TablesView& tab = w->tab;
  const int R = tab.n_req, P = pool.page_size, H = pool.n_kv_heads;
  const int jp = w->parts_per_page;
  const int page_item = item / jp, j = item - page_item * jp;
  const int total_new = w->total_new;
  const int slab = page_item / total_new, rem = page_item - slab * total_new;
  const int32_t* item_off = ws_item_off(w, R);
  int lo = 0, hi = R;                                  // item_off[lo] <= rem < item_off[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (item_off[mid] <= rem) lo = mid; else hi = mid;
  }
  const int r = lo, dp = rem - item_off[r];
  const int32_t n = w->budget[r] < 0 ? 0 : w->budget[r];
  const int nsh = min(P, n - dp * P) * H;
  const int32_t L = tab.seq_len[r];
  uint32_t so = CJ_NONE;
  const int i = lane + 32 * j;
  if (i < nsh) {
    const int slot = i / H, h = i - slot * H;
    const int32_t tok = w->sel_idx[((int64_t)slab * H + h) * w->sel_stride + w->keep_indptr[r] + dp * P + slot];
    if ((uint32_t)tok >= (uint32_t)L) {
      report(w->status, ACTKV_E_BADINDEX, r, tok);
    } else {
      const int32_t sp = page_or_neg(tab, pool.n_pages, r, tok / P, w->status);
      if (sp >= 0)
        so = (uint32_t)(((int64_t)sp * pool.stride_page + (int64_t)(tok % P) * pool.stride_slot +
                         (int64_t)h * pool.stride_head) >> 3);
    }
  }
  w->src_tab[(int64_t)item * 32 + lane] = so;
}

// One item, executed by one converged warp: 32 consecutive (slot, head) pairs of one destination page, one
// pair per lane, the K row and the V row of each.  Offsets are kept in 16-byte units relative to the layer
// (the host checked that a layer spans less than 2^32 of them).  NFLY 16-byte loads are in flight per lane:
// the K and the V vector of NFLY / 2 steps.
template <int VPR_SHIFT, int NFLY>
__device__ __forceinline__ void cj_copy_item(CompactWs* w, int item, int lane) {
  const PoolView& pool = w->pool;
  const int ips = w->items_per_slab;
  const int slab = item / ips;
  // the two lookups of an item, independent of each other
  const uint32_t so = w->src_tab[(int64_t)item * 32 + lane];
  uint32_t dof;
  if (w->dst_tab != nullptr) {                         // (uniform over the job) in-place form: resolved destinations
    dof = w->dst_tab[(int64_t)item * 32 + lane];
  } else {
    const int H = pool.n_kv_heads;
    const int jp = w->parts_per_page;                  // items per destination page: ceil(P H / 32)
    const int rem_item = item - slab * ips;
    const int rem = rem_item / jp, j = rem_item - rem * jp;
    const int32_t dst_page = ws_new_pages(w, w->tab.n_req)[rem];
    const int i = lane + 32 * j;
    const int slot = i / H, h = i - slot * H;
    dof = (uint32_t)(((int64_t)dst_page * pool.stride_page + (int64_t)slot * pool.stride_slot +
                      (int64_t)h * pool.stride_head) >> 3);
  }
  uint4* lbase = reinterpret_cast<uint4*>(const_cast<__nv_bfloat16*>(pool.base) +
                                          (int64_t)(w->layer_begin + slab) * pool.stride_layer);
  constexpr int RPS = 32 >> VPR_SHIFT;                 // rows per step (one 16-byte vector per lane): 4, 2, 1
  constexpr int STEPS = 32 / RPS;                      // steps per 32 (slot, head) pairs
  constexpr int NB = NFLY / 2 < STEPS ? NFLY / 2 : STEPS;   // steps per batch
  static_assert(STEPS % NB == 0, "batches");
  const int sub = lane >> VPR_SHIFT;
  const uint32_t dv = (uint32_t)(lane & ((1 << VPR_SHIFT) - 1));
  const uint32_t kvo = (uint32_t)(pool.stride_kv >> 3);
#pragma unroll 1
  for (int t0 = 0; t0 < STEPS; t0 += NB) {
    uint4 val[2 * NB];
    uint32_t d[NB];
#pragma unroll
    for (int k = 0; k < NB; ++k) {
      const int src_lane = (t0 + k) * RPS + sub;       // the lane that holds this step's row
      const uint32_t s = __shfl_sync(0xffffffffu, so, src_lane);
      d[k] = __shfl_sync(0xffffffffu, dof, src_lane);
      if (s == CJ_NONE) d[k] = CJ_NONE;                // a row past the item's end, or a dropped move
      if (d[k] != CJ_NONE) {
        val[2 * k] = ld_stream(lbase + (size_t)s + dv);
        val[2 * k + 1] = ld_stream(lbase + (size_t)s + kvo + dv);
      }
    }
#pragma unroll
    for (int k = 0; k < NB; ++k) {
      if (d[k] != CJ_NONE) {
        st_stream(lbase + (size_t)d[k] + dv, val[2 * k]);
        st_stream(lbase + (size_t)d[k] + kvo + dv, val[2 * k + 1]);
      }
    }
  }
}

// The copy role of a kernel whose other warps do something else: items are taken while `keep_going()` holds
// (the host kernel's own work is still running), so that the CTA retires with its main work.  The item taken
// ahead when the role stops is handed to nobody else, so the role executes it before it leaves.
template <int VPR_SHIFT, int NFLY, class KeepGoing>
__device__ __forceinline__ void cj_copy_role(CompactWs* w, int lane, KeepGoing keep_going) {
  if (w == nullptr || w->vpr_shift != VPR_SHIFT) return;
  const uint32_t n = cj_count(w);
  if (n == 0) return;
  int done = 0;
  uint32_t item = cj_pop(w, lane);
  while (item < n) {
    const bool go = keep_going();
    const uint32_t next = go ? cj_pop(w, lane) : n;    // asked for now, looked at after this item's copies
    cj_copy_item<VPR_SHIFT, NFLY>(w, (int)item, lane);
    ++done;
    item = next;
  }
  if (lane == 0 && done > 0) atomicAdd(&w->role_items, done);
}

// What is left of a deferred copy: every warp takes items until the queue is empty.
template <int VPR_SHIFT>
__global__ void __launch_bounds__(128) compact_drain_kernel(CompactWs* ws) {
  const int lane = threadIdx.x & 31;
  if (ws->vpr_shift != VPR_SHIFT) return;
  const uint32_t n = cj_count(ws);
  if (n == 0) return;
  uint32_t item = cj_pop(ws, lane);
  while (item < n) {
    const uint32_t next = cj_pop(ws, lane);              // asked for now, looked at after this item's copies
    cj_copy_item<VPR_SHIFT, 16>(ws, (int)item, lane);
    item = next;
  }
}

// Launches the drain kernel for a job of at most `items_max` items: at most eight CTAs of four warps per SM.
inline void launch_drain(CompactWs* w, int shift, int64_t items_max, cudaStream_t s) {
  const int64_t want = (items_max + 3) / 4;
  const unsigned grid = (unsigned)(want < 1 ? 1 : (want > 148 * 8 ? 148 * 8 : want));
  if (shift == 3) compact_drain_kernel<3><<<grid, 128, 0, s>>>(w);
  else if (shift == 4) compact_drain_kernel<4><<<grid, 128, 0, s>>>(w);
  else compact_drain_kernel<5><<<grid, 128, 0, s>>>(w);
}

// log2 of the 16-byte vectors per row when the warp-level item copy takes this pool: head_dim 64, 128 or 256,
// a layer (K and V) within 2^32 16-byte units; else -1.
inline int deferrable_shift(const actkv_pool_t* pool) {
  const int vpr = pool->head_dim / 8;
  const int shift = vpr == 8 ? 3 : vpr == 16 ? 4 : vpr == 32 ? 5 : -1;
  if (shift < 0) return -1;
  const int64_t extent = pool->stride_kv + (int64_t)pool->n_pages * pool->stride_page;       // elements, upper bound
  if (pool->stride_kv < 0 || pool->stride_page < 0 || pool->stride_slot < 0 || pool->stride_head < 0) return -1;
  if (extent / 8 >= 0xffffffffLL) return -1;
  return shift;
}

}  // namespace actkv
