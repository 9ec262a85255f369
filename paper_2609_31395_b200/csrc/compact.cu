// actkv_compact: pack survivors into fresh pages, free the old pages (Section 7.2, Algorithm 4:
// plan first, then one-shot parallel copies whose sources and destinations are disjoint, then
// return the freed blocks).  Three kernels on one stream:
//   plan     : per request X_r, offsets into the run of pages popped from the free-list stack,
//              the new page ids; detects a short free list (nothing is modified in that case);
//   copy     : one CTA per (destination page, request, layer) gathers the 16-byte vectors of the
//              K and V rows of the survivors of every head into the page — destination pages are
//              written whole and coalesced, sources are 256-byte row gathers;
//   finalize : new page table / seq_len, pop and push on the free list (only on the call whose
//              layer range ends at the pool's last layer).
#include <algorithm>

#include "compact_job.cuh"

namespace actkv {

// What the host knows of a compaction call, handed to the plan kernel, which records it in the workspace.
struct CompactJobArgs {
  PoolView pool;
  const int32_t* sel_idx;
  int64_t sel_stride;
  const int32_t* keep_indptr;
  int32_t layer_begin, n_layers;
  int32_t vpr_shift;     // >= 0: the copies may be deferred to a work queue (actkv_compact_begin)
  int32_t deferred;
  uint32_t* src_tab;     // deferred: room for the resolved sources of every item
  int64_t src_tab_items; // ... in items (32 entries each)
  const int32_t* tab_page_table;   // the tables of the call (a reused plan must be one of these tables)
};

__global__ void compact_plan_kernel(TablesView tab, int32_t page_size, int32_t n_pages,
                                    const int32_t* __restrict__ budget, int32_t max_keep,
                                    CompactWs* ws, int32_t* status, CompactJobArgs job) {
  const int R = tab.n_req;
  int32_t* new_off = ws_new_off(ws);
  int32_t* push_off = ws_push_off(ws, R);
  int32_t* item_off = ws_item_off(ws, R);
  int32_t* new_pages = ws_new_pages(ws, R);
  __shared__ int32_t s_total, s_ok;
  if (threadIdx.x == 0) {
    int32_t off = 0, poff = 0;
    bool ok = !status_set(status);
    for (int r = 0; r < R; ++r) {
      const int32_t L = tab.seq_len[r];
      int32_t B = budget[r] < 0 ? 0 : budget[r];
      item_off[r] = off;
      if (B < L) {
        new_off[r] = off;
        push_off[r] = poff;
        off += (B + page_size - 1) / page_size;
        poff += (L + page_size - 1) / page_size;
        if ((L + page_size - 1) / page_size > tab.max_pages) { report(status, ACTKV_E_INVALID, r, L); ok = false; }
        if (B > max_keep) { report(status, ACTKV_E_INVALID, r, B); ok = false; }   // host bound too small
      } else {
        new_off[r] = -1;
        push_off[r] = -1;
      }
    }
    const int32_t fc = *tab.free_count;
    if (fc < 0 || fc > n_pages) { report(status, ACTKV_E_INVALID, -1, fc); ok = false; }
    else if (off > fc) { report(status, ACTKV_E_NOFREE, off, fc); ok = false; }
    // the old pages pushed back after the pops must fit on the stack
    else if ((int64_t)fc - off + poff > n_pages) { report(status, ACTKV_E_INVALID, -2, fc - off + poff); ok = false; }
    item_off[R] = off;
    s_total = off;
    s_ok = ok ? 1 : 0;
  }
  __syncthreads();
  // every old page that will be pushed on the free list must be a page id
  if (s_ok) {
    for (int r = 0; r < R; ++r) {
      if (new_off[r] < 0) continue;
      const int Y = (tab.seq_len[r] + page_size - 1) / page_size;
      const int32_t* row = tab.page_table + (int64_t)r * tab.max_pages;
      for (int i0 = threadIdx.x; i0 < Y; i0 += 4 * blockDim.x) {        // four independent loads per thread
        int32_t id[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) { const int i = i0 + k * blockDim.x; id[k] = i < Y ? row[i] : 0; }
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if ((uint32_t)id[k] >= (uint32_t)n_pages) { report(status, ACTKV_E_BADPAGE, r, id[k]); s_ok = 0; }
      }
    }
  }
  __syncthreads();
  const int32_t total = s_total;
  if (s_ok) {
    const int32_t fc = *tab.free_count;
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
      int32_t id = tab.free_list[fc - 1 - i];
      if ((uint32_t)id >= (uint32_t)n_pages) { report(status, ACTKV_E_BADPAGE, -1, id); s_ok = 0; }
      new_pages[i] = id;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    ws->plan_ok = s_ok;
    ws->total_new = total;
    ws->next_item = 0u;
    const int32_t jp = (page_size * job.pool.n_kv_heads + 31) / 32;
    const int64_t items = (int64_t)total * job.n_layers * jp;
    ws->n_items = (s_ok && job.deferred && job.vpr_shift >= 0 && items <= 0x7fffffff && items <= job.src_tab_items)
                      ? (int32_t)items : 0;
    ws->src_tab = job.src_tab;
    ws->pool = job.pool;
    ws->tab = tab;
    ws->sel_idx = job.sel_idx;
    ws->sel_stride = job.sel_stride;
    ws->keep_indptr = job.keep_indptr;
    ws->budget = budget;
    ws->status = status;
    ws->layer_begin = job.layer_begin;
    ws->n_layers = job.n_layers;
    ws->vpr_shift = job.deferred ? job.vpr_shift : -1;
    ws->parts_per_page = jp;
    ws->items_per_slab = (int32_t)max((int64_t)1, min((int64_t)total * jp, (int64_t)0x7fffffff));
    ws->dst_tab = nullptr;
    ws->pad2 = 0;
    ws->role_items = 0;
    ws->pad = CJ_PLAN_MARK;
  }
}

__global__ void compact_stats_kernel(const CompactWs* ws, int32_t* out) {
  out[0] = ws->n_items;
  out[1] = ws->role_items;
}

// A further layer range of a step whose plan is already in the workspace (the plan depends on the tables and
// the budgets only, not on the layers): only the job is recorded anew.
__global__ void compact_rejob_kernel(CompactWs* ws, CompactJobArgs job, int32_t* status) {
  // the workspace must hold a plan of these very tables and this pool (a caller's mistake otherwise: reported,
  // and nothing is copied or finalized from what happens to be in the workspace)
  const bool mine = ws->pad == CJ_PLAN_MARK && ws->pool.base == job.pool.base && ws->tab.page_table == job.tab_page_table &&
                    ws->status == status;
  if (!mine) {
    report(status, ACTKV_E_INVALID, -3, 0);
    ws->pad = CJ_PLAN_MARK;
    ws->plan_ok = 0;
    ws->total_new = 0;
    ws->n_items = 0;
    ws->next_item = 0u;
    ws->role_items = 0;
    ws->vpr_shift = -1;
    ws->parts_per_page = 1;
    ws->items_per_slab = 1;
    ws->dst_tab = nullptr;
    return;
  }
  const bool ok = ws->plan_ok && !status_set(status);
  if (!ok) ws->plan_ok = 0;
  const int64_t items = (int64_t)ws->total_new * job.n_layers * ws->parts_per_page;
  ws->next_item = 0u;
  ws->role_items = 0;
  ws->n_items = (ok && job.deferred && job.vpr_shift >= 0 && items <= 0x7fffffff && items <= job.src_tab_items)
                    ? (int32_t)items : 0;
  ws->src_tab = job.src_tab;
  ws->dst_tab = nullptr;
  ws->sel_idx = job.sel_idx;
  ws->sel_stride = job.sel_stride;
  ws->keep_indptr = job.keep_indptr;
  ws->layer_begin = job.layer_begin;
  ws->n_layers = job.n_layers;
  ws->vpr_shift = job.deferred ? job.vpr_shift : -1;
}

// Resolves the sources of every item of a deferred copy (one warp per item).
__global__ void __launch_bounds__(128) compact_resolve_kernel(CompactWs* ws) {
  const int lane = threadIdx.x & 31;
  const int64_t n = cj_count(ws);
  for (int64_t item = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5); item < n; item += (int64_t)gridDim.x * 4)
    cj_resolve_item(ws, (int)item, lane);
}

constexpr int CP_NT = 128;
constexpr int CP_UNROLL = 8;

// One CTA per (destination page, request, layer).  The (slot, head) -> source / destination row
// offsets are resolved once into shared memory; the copy loop then costs two shared loads and a few
// integer ops per 16-byte vector, with CP_UNROLL independent loads in flight per thread.
// VPR_SHIFT >= 0: 16-byte vectors per row = 1 << VPR_SHIFT (head_dim 64 / 128 / 256); -1: any head_dim.
template <int VPR_SHIFT>
__global__ void __launch_bounds__(CP_NT) compact_copy_kernel(
    PoolView pool, TablesView tab, int32_t layer_begin, const int32_t* __restrict__ sel_idx,
    int64_t sel_stride, const int32_t* __restrict__ keep_indptr, const int32_t* __restrict__ budget,
    CompactWs* ws, int32_t* status) {
  extern __shared__ __align__(16) int64_t cp_smem[];     // [2][P*H]: source offsets, destination offsets
  if (!ws->plan_ok) return;
  const int R = tab.n_req;
  const int r = blockIdx.y, slab = blockIdx.z, dp = blockIdx.x;
  const int32_t noff = ws_new_off(ws)[r];
  if (noff < 0) return;
  const int P = pool.page_size, H = pool.n_kv_heads, D = pool.head_dim;
  const int32_t n = budget[r] < 0 ? 0 : budget[r];
  const int X = (n + P - 1) / P;
  if (dp >= X) return;
  const int32_t L = tab.seq_len[r];
  const int32_t dst_page = ws_new_pages(ws, R)[noff + dp];
  const int n_slots = min(P, n - dp * P);
  const int nsh = n_slots * H;
  int64_t* src_off = cp_smem;
  int64_t* dst_off = cp_smem + P * H;
  const int32_t* sel_base = sel_idx + (int64_t)slab * H * sel_stride + keep_indptr[r] + dp * P;
  for (int i = threadIdx.x; i < nsh; i += CP_NT) {
    const int slot = i / H, h = i - slot * H;
    const int32_t tok = sel_base[(int64_t)h * sel_stride + slot];
    int64_t so = -1;
    if ((uint32_t)tok >= (uint32_t)L) {
      report(status, ACTKV_E_BADINDEX, r, tok);
    } else {
      const int32_t sp = page_or_neg(tab, pool.n_pages, r, tok / P, status);
      if (sp >= 0)
        so = (int64_t)sp * pool.stride_page + (int64_t)(tok % P) * pool.stride_slot + (int64_t)h * pool.stride_head;
    }
    src_off[i] = so;
    dst_off[i] = (int64_t)dst_page * pool.stride_page + (int64_t)slot * pool.stride_slot + (int64_t)h * pool.stride_head;
  }
  __syncthreads();
  __nv_bfloat16* lbase = const_cast<__nv_bfloat16*>(pool.base) + (int64_t)(layer_begin + slab) * pool.stride_layer;
  const int vpr = D / 8;
  const int per_kv = (VPR_SHIFT >= 0) ? (nsh << VPR_SHIFT) : nsh * vpr;
  const int total = 2 * per_kv;
  for (int v0 = threadIdx.x; v0 < total; v0 += CP_NT * CP_UNROLL) {
    uint4 val[CP_UNROLL];
    int64_t doff[CP_UNROLL];
#pragma unroll
    for (int k = 0; k < CP_UNROLL; ++k) {
      const int v = v0 + k * CP_NT;
      doff[k] = -1;
      if (v < total) {
        const int kv = v >= per_kv ? 1 : 0;
        const int rem = v - kv * per_kv;
        const int i = (VPR_SHIFT >= 0) ? (rem >> VPR_SHIFT) : rem / vpr;
        const int dv = (VPR_SHIFT >= 0) ? (rem & ((1 << VPR_SHIFT) - 1)) : rem - i * vpr;
        const int64_t so = src_off[i];
        if (so >= 0) {
          const int64_t kvo = (int64_t)kv * pool.stride_kv + dv * 8;
          val[k] = *reinterpret_cast<const uint4*>(lbase + so + kvo);
          doff[k] = dst_off[i] + kvo;
        }
      }
    }
#pragma unroll
    for (int k = 0; k < CP_UNROLL; ++k)
      if (doff[k] >= 0) *reinterpret_cast<uint4*>(lbase + doff[k]) = val[k];
  }
}

__global__ void compact_finalize_kernel(TablesView tab, int32_t page_size,
                                        const int32_t* __restrict__ budget, CompactWs* ws,
                                        const int32_t* status) {
  // an error met by the copies (bad index, bad page) leaves the tables as they were: the fresh
  // pages that were written are still on the free list
  if (!ws->plan_ok || status_set(status)) return;
  const int R = tab.n_req;
  const int32_t* new_off = ws_new_off(ws);
  const int32_t* push_off = ws_push_off(ws, R);
  const int32_t* new_pages = ws_new_pages(ws, R);
  const int32_t fc_new = *tab.free_count - ws->total_new;
  __shared__ int32_t s_pushed;
  if (threadIdx.x == 0) s_pushed = 0;
  __syncthreads();
  // push the old pages (reads the old table), request by request in ascending order
  for (int r = 0; r < R; ++r) {
    if (new_off[r] < 0) continue;
    const int Y = (tab.seq_len[r] + page_size - 1) / page_size;
    for (int i = threadIdx.x; i < Y; i += blockDim.x)
      tab.free_list[fc_new + push_off[r] + i] = tab.page_table[(int64_t)r * tab.max_pages + i];
    if (threadIdx.x == 0) s_pushed += Y;
  }
  __syncthreads();
  // then rewrite the tables
  for (int r = 0; r < R; ++r) {
    if (new_off[r] < 0) continue;
    const int32_t n = budget[r] < 0 ? 0 : budget[r];
    const int X = (n + page_size - 1) / page_size;
    for (int i = threadIdx.x; i < tab.max_pages; i += blockDim.x)
      tab.page_table[(int64_t)r * tab.max_pages + i] = i < X ? new_pages[new_off[r] + i] : -1;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int r = 0; r < R; ++r)
      if (new_off[r] >= 0) tab.seq_len[r] = budget[r] < 0 ? 0 : budget[r];
    *tab.free_count = fc_new + s_pushed;
  }
}

}  // namespace actkv

extern "C" {

size_t actkv_compact_workspace_bytes(int32_t n_req, int32_t max_pages) {
  if (n_req < 0 || max_pages < 0) return 0;
  return actkv::align_up(sizeof(actkv::CompactWs) +
                         sizeof(int32_t) * ((size_t)3 * n_req + 1 + (size_t)n_req * max_pages), 256);
}

size_t actkv_compact_deferred_workspace_bytes(const actkv_pool_t* pool, int32_t n_req, int32_t max_pages,
                                              int32_t n_layers_sub, int32_t max_keep) {
  if (!pool || n_req < 0 || max_pages < 0 || n_layers_sub < 0 || max_keep < 0 || pool->page_size <= 0) return 0;
  const size_t base = actkv_compact_workspace_bytes(n_req, max_pages);
  int64_t max_x = ((int64_t)max_keep + pool->page_size - 1) / pool->page_size;
  if (max_x > max_pages) max_x = max_pages;
  const int64_t jp = ((int64_t)pool->page_size * pool->n_kv_heads + 31) / 32;
  return base + actkv::align_up((size_t)(max_x * n_req * n_layers_sub * jp) * 32 * sizeof(uint32_t), 256);
}

}  // extern "C"

namespace actkv {

static int compact_check(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin, int32_t layer_end,
                         const int32_t* budget, int32_t max_keep, int64_t sel_stride, void* ws, size_t ws_bytes) {
  if (!pool || !tables || !pool->base) return ACTKV_E_INVALID;
  if (layer_begin < 0 || layer_end > pool->n_layers || layer_begin > layer_end) return ACTKV_E_INVALID;
  if (pool->page_size <= 0 || pool->head_dim <= 0 || pool->head_dim % 8 != 0 || pool->n_kv_heads <= 0)
    return ACTKV_E_INVALID;
  // 16-byte vector moves need every row start 16-byte aligned
  if (((uintptr_t)pool->base & 15) || pool->stride_layer % 8 || pool->stride_kv % 8 || pool->stride_page % 8 ||
      pool->stride_slot % 8 || pool->stride_head % 8)
    return ACTKV_E_INVALID;
  const int R = tables->n_req;
  if (R < 0 || tables->max_pages < 0 || max_keep < 0 || sel_stride < 0) return ACTKV_E_INVALID;
  if (R == 0) return ACTKV_OK;
  if (!tables->page_table || !tables->seq_len || !tables->free_list || !tables->free_count || !budget || !ws)
    return ACTKV_E_INVALID;
  if (ws_bytes < actkv_compact_workspace_bytes(R, tables->max_pages)) return ACTKV_E_WORKSPACE;
  if (R > 65535 || layer_end - layer_begin > 65535) return ACTKV_E_INVALID;
  return ACTKV_OK;
}

static int compact_plan(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin, int32_t layer_end,
                        const int32_t* sel_idx, int64_t sel_stride, const int32_t* keep_indptr, const int32_t* budget,
                        int32_t max_keep, void* ws, size_t ws_bytes, int32_t* status, cudaStream_t s, bool deferred,
                        bool reuse_plan = false) {
  CompactJobArgs job;
  const size_t base = actkv_compact_workspace_bytes(tables->n_req, tables->max_pages);
  // the copies are deferred only when the workspace has room for the resolved sources of the largest job these
  // arguments allow (the same rule decides in actkv_compact_end who copies)
  deferred = deferred && ws_bytes >= actkv_compact_deferred_workspace_bytes(pool, tables->n_req, tables->max_pages,
                                                                             layer_end - layer_begin, max_keep);
  job.src_tab = (uint32_t*)((char*)ws + base);
  job.src_tab_items = deferred ? (int64_t)((ws_bytes - base) / (32 * sizeof(uint32_t))) : 0;
  job.pool = make_view(pool);
  job.tab_page_table = tables->page_table;
  job.sel_idx = sel_idx;
  job.sel_stride = sel_stride;
  job.keep_indptr = keep_indptr;
  job.layer_begin = layer_begin;
  job.n_layers = layer_end - layer_begin;
  job.vpr_shift = deferrable_shift(pool);
  job.deferred = deferred ? 1 : 0;
  if (reuse_plan)
    compact_rejob_kernel<<<1, 1, 0, s>>>((CompactWs*)ws, job, status);
  else
    compact_plan_kernel<<<1, 1024, 0, s>>>(make_view(tables), pool->page_size, pool->n_pages, budget, max_keep,
                                           (CompactWs*)ws, status, job);
  ACTKV_CHECK_LAUNCH();
  if (deferred && job.vpr_shift >= 0 && job.src_tab_items > 0) {
    // one warp per item of the largest job these arguments allow (short, independent chains of lookups)
    int64_t max_x = ((int64_t)max_keep + pool->page_size - 1) / pool->page_size;
    if (max_x > tables->max_pages) max_x = tables->max_pages;
    const int64_t jp = ((int64_t)pool->page_size * pool->n_kv_heads + 31) / 32;
    const int64_t items_max = std::min<int64_t>(max_x * tables->n_req * job.n_layers * jp, job.src_tab_items);
    const int64_t ctas = std::min<int64_t>(std::max<int64_t>(1, (items_max + 3) / 4), 1 << 20);
    compact_resolve_kernel<<<(unsigned)ctas, 128, 0, s>>>((CompactWs*)ws);
    ACTKV_CHECK_LAUNCH();
  }
  return ACTKV_OK;
}

// One CTA per (destination page, request, layer): the whole copy of a call in one launch.
static int compact_copy_all(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin, int32_t layer_end,
                            const int32_t* sel_idx, int64_t sel_stride, const int32_t* keep_indptr, const int32_t* budget,
                            int32_t max_keep, void* ws, int32_t* status, cudaStream_t s) {
  PoolView pv = make_view(pool);
  TablesView tv = make_view(tables);
  CompactWs* w = (CompactWs*)ws;
  const int nl = layer_end - layer_begin, R = tables->n_req;
  int max_x = (max_keep + pool->page_size - 1) / pool->page_size;
  if (max_x > tables->max_pages) max_x = tables->max_pages;
  if (nl <= 0 || max_x <= 0) return ACTKV_OK;
  dim3 grid((unsigned)max_x, (unsigned)R, (unsigned)nl);
  const size_t sm = (size_t)2 * pool->page_size * pool->n_kv_heads * sizeof(int64_t);
  if (sm > 48 * 1024) return ACTKV_E_INVALID;
  const int vpr = pool->head_dim / 8;
  if (vpr == 16)
    compact_copy_kernel<4><<<grid, CP_NT, sm, s>>>(pv, tv, layer_begin, sel_idx, sel_stride, keep_indptr, budget, w, status);
  else if (vpr == 8)
    compact_copy_kernel<3><<<grid, CP_NT, sm, s>>>(pv, tv, layer_begin, sel_idx, sel_stride, keep_indptr, budget, w, status);
  else if (vpr == 32)
    compact_copy_kernel<5><<<grid, CP_NT, sm, s>>>(pv, tv, layer_begin, sel_idx, sel_stride, keep_indptr, budget, w, status);
  else
    compact_copy_kernel<-1><<<grid, CP_NT, sm, s>>>(pv, tv, layer_begin, sel_idx, sel_stride, keep_indptr, budget, w, status);
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

static int compact_finalize(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_end, const int32_t* budget,
                            void* ws, int32_t* status, cudaStream_t s) {
  if (layer_end != pool->n_layers) return ACTKV_OK;
  compact_finalize_kernel<<<1, 1024, 0, s>>>(make_view(tables), pool->page_size, budget, (CompactWs*)ws, status);
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

}  // namespace actkv

extern "C" {

int actkv_compact(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                  int32_t layer_end, const int32_t* sel_idx, int64_t sel_stride,
                  const int32_t* keep_indptr, const int32_t* budget, int32_t max_keep,
                  void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream) {
  using namespace actkv;
  int rc = compact_check(pool, tables, layer_begin, layer_end, budget, max_keep, sel_stride, ws, ws_bytes);
  if (rc != ACTKV_OK || tables->n_req == 0) return rc;
  if (!keep_indptr || !sel_idx) return ACTKV_E_INVALID;
  cudaStream_t s = (cudaStream_t)stream;
  rc = compact_plan(pool, tables, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr, budget, max_keep, ws, ws_bytes,
                    status, s, false);
  if (rc != ACTKV_OK) return rc;
  rc = compact_copy_all(pool, tables, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr, budget, max_keep, ws, status, s);
  if (rc != ACTKV_OK) return rc;
  return compact_finalize(pool, tables, layer_end, budget, ws, status, s);
}

int actkv_compact_begin(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                        int32_t layer_end, const int32_t* sel_idx, int64_t sel_stride,
                        const int32_t* keep_indptr, const int32_t* budget, int32_t max_keep, int32_t reuse_plan,
                        void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream) {
  using namespace actkv;
  int rc = compact_check(pool, tables, layer_begin, layer_end, budget, max_keep, sel_stride, ws, ws_bytes);
  if (rc != ACTKV_OK || tables->n_req == 0) return rc;
  if (!keep_indptr || !sel_idx) return ACTKV_E_INVALID;
  return compact_plan(pool, tables, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr, budget, max_keep, ws, ws_bytes,
                      status, (cudaStream_t)stream, true, reuse_plan != 0);
}

int actkv_compact_stats(const void* ws, int32_t* stats, actkv_stream_t stream) {
  if (!ws || !stats) return ACTKV_E_INVALID;
  actkv::compact_stats_kernel<<<1, 1, 0, (cudaStream_t)stream>>>((const actkv::CompactWs*)ws, stats);
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

int actkv_compact_end(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                      int32_t layer_end, const int32_t* sel_idx, int64_t sel_stride,
                      const int32_t* keep_indptr, const int32_t* budget, int32_t max_keep,
                      void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream) {
  using namespace actkv;
  int rc = compact_check(pool, tables, layer_begin, layer_end, budget, max_keep, sel_stride, ws, ws_bytes);
  if (rc != ACTKV_OK || tables->n_req == 0) return rc;
  if (!keep_indptr || !sel_idx) return ACTKV_E_INVALID;
  cudaStream_t s = (cudaStream_t)stream;
  const int shift = deferrable_shift(pool);
  const size_t need = actkv_compact_deferred_workspace_bytes(pool, tables->n_req, tables->max_pages, layer_end - layer_begin,
                                                             max_keep);
  if (shift < 0 || ws_bytes < need) {
    // a pool shape the item copy does not take: nothing was deferred (the queue is empty), the copy runs here
    rc = compact_copy_all(pool, tables, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr, budget, max_keep, ws, status, s);
    if (rc != ACTKV_OK) return rc;
  } else {
    // every warp takes items until the queue is empty
    const int64_t max_x = std::min<int64_t>((max_keep + pool->page_size - 1) / pool->page_size, tables->max_pages);
    const int64_t jp = ((int64_t)pool->page_size * pool->n_kv_heads + 31) / 32;
    launch_drain((CompactWs*)ws, shift, max_x * tables->n_req * (layer_end - layer_begin) * jp, s);
    ACTKV_CHECK_LAUNCH();
  }
  return compact_finalize(pool, tables, layer_end, budget, ws, status, s);
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// actkv_compact_noalloc: the same compaction for callers that have no device allocator to ask
// for the plan scratch.  The scratch is a fixed array in the library's own device image.

#include <mutex>

// Plan scratch of actkv_compact_noalloc.  One copy lives on every GPU that loads the library, from
// load until the process exits.  Device code could name it directly; host code may only use the
// address that cudaGetSymbolAddress returns for the current device (the host-side symbol is a
// stand-in, not a device pointer).
static __device__ __align__(256) unsigned char g_compact_scratch[ACTKV_COMPACT_NOALLOC_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};
}  // namespace

extern "C" {

size_t actkv_compact_noalloc_max_bytes(void) { return ACTKV_COMPACT_NOALLOC_BYTES; }

int actkv_compact_noalloc(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                          int32_t layer_end, const int32_t* sel_idx, int64_t sel_stride,
                          const int32_t* keep_indptr, const int32_t* budget, int32_t max_keep,
                          int32_t* status, actkv_stream_t stream) {
  if (!tables) return ACTKV_E_INVALID;
  if (tables->n_req < 0 || tables->max_pages < 0) return ACTKV_E_INVALID;
  if (actkv_compact_workspace_bytes(tables->n_req, tables->max_pages) > ACTKV_COMPACT_NOALLOC_BYTES)
    return ACTKV_E_TOOBIG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ACTKV_E_CUDA;
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (g_scratch_addr[dev] == nullptr) {
      // once per device, with that device current: resolve the array's address on THIS device
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_compact_scratch) != cudaSuccess || p == nullptr) return ACTKV_E_CUDA;
      g_scratch_addr[dev] = p;
    }
    scratch = g_scratch_addr[dev];
  }
  // Every word of the plan that the copy and table-update kernels read is rewritten by the plan
  // kernel of this same call (flags, per-request offsets, the page ids it pops), so what an earlier
  // call left in the array is never read and nothing needs clearing.
  return actkv_compact(pool, tables, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr, budget, max_keep,
                       scratch, ACTKV_COMPACT_NOALLOC_BYTES, status, stream);
}

}  // extern "C"
