// actkv_compact_inplace: in-place compaction into the last X logical blocks of every request
// (Section 7.2 region equations; Algorithm 4), one keep mask per (layer, KV head).
//
// For a request with L used slots in Y = ceil(L/BS) blocks and budget B < L:  X = ceil(B/BS),
// Start = (Y-X)*BS, End = Start + B.  Holes of the region (slots of [Start, End) that are not kept,
// including allocated-but-unused slots past L) are the destinations, survivors outside the region are
// the sources, both in ascending order, zipped.  With the keep mask given as the ascending index list
// sel[0..B) the plan needs no scan and no scratch:
//     a = #kept below Start, c = #kept below End,
//     hole p has rank j = (p - Start) - (#kept in [Start, p)),
//     its source is the j-th survivor outside the region: sel[j] if j < a, else sel[c + j - a].
// Two kernels on one stream:
//   copy     : one CTA per (256 region slots, request, layer x head): every thread classifies one slot
//              by binary search in the CTA's window of the index list, the CTA's moves are packed in
//              shared memory and copied as 16-byte vectors, several loads in flight per thread.
//              Sources lie outside the region and destinations inside it, so one pass is conflict-free.
//   finalize : page_table[r] <- its last X pages, seq_len[r] <- B, the first Y-X pages are pushed on
//              the free-list stack (only on the call whose layer range ends at the pool's last layer).
// On a device-detected error the tables stay as they were; only dead slots (holes) were written.
// The copy can also be deferred (actkv_compact_inplace_begin / _end): the moves of a layer group are resolved
// once into a table of (source, destination) row offsets, 32 region slots per item, and published as the work
// queue of compact_job.cuh, so that the spare warps of the pooled-score kernel of the NEXT layer group execute
// them (sources and destinations lie in layers that kernel does not touch) and a drain kernel what is left.
#include "compact_job.cuh"

namespace actkv {

constexpr int CI_NT = 128;
constexpr int CI_UNROLL = 8;

__device__ __forceinline__ int lower_bound_i32(const int32_t* __restrict__ a, int n, int32_t key) {
  int lo = 0, hi = n;                                        // first index with a[idx] >= key
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (a[mid] < key) lo = mid + 1; else hi = mid;
  }
  return lo;
}

template <int VPR_SHIFT>
__global__ void __launch_bounds__(CI_NT) compact_inplace_copy_kernel(
    PoolView pool, TablesView tab, int32_t layer_begin, const int32_t* __restrict__ sel_idx, int64_t sel_stride,
    const int32_t* __restrict__ keep_indptr, const int32_t* __restrict__ budget, int32_t max_keep,
    int32_t* __restrict__ new_order, int32_t* status) {
  __shared__ int32_t s_win[CI_NT];                           // kept indices that can fall in this CTA's slots
  __shared__ int64_t s_src[CI_NT], s_dst[CI_NT];
  __shared__ int32_t s_a, s_c, s_lb0, s_cnt;

  if (status_set(status)) return;
  const int r = blockIdx.y;
  const int H = pool.n_kv_heads, P = pool.page_size, D = pool.head_dim;
  const int slab = blockIdx.z / H, h = blockIdx.z - slab * H;
  const int tid = threadIdx.x, lane = tid & 31;
  const int32_t L = tab.seq_len[r];
  const int32_t B = budget[r] < 0 ? 0 : budget[r];
  const int32_t* sel = sel_idx + (int64_t)blockIdx.z * sel_stride + keep_indptr[r];
  int32_t* ord = new_order ? new_order + (int64_t)blockIdx.z * sel_stride + keep_indptr[r] : nullptr;
  const int32_t i0 = blockIdx.x * CI_NT;                     // first region slot of this CTA, relative to Start

  if (B >= L) {                                              // not compacting: the order is the identity list
    if (ord && i0 + tid < L) ord[i0 + tid] = sel[i0 + tid];
    return;
  }
  if (i0 >= B) return;
  const int Y = (L + P - 1) / P, X = (B + P - 1) / P;
  if (Y > tab.max_pages || B > max_keep) {
    if (tid == 0) report(status, ACTKV_E_INVALID, r, Y > tab.max_pages ? L : B);
    return;
  }
  const int32_t start = (Y - X) * P, end = start + B;
  const int32_t p0 = start + i0;

  if (tid == 0) s_a = lower_bound_i32(sel, B, start);
  if (tid == 32) s_c = lower_bound_i32(sel, B, end);
  if (tid == 64) s_lb0 = lower_bound_i32(sel, B, p0);
  if (tid == 96) s_cnt = 0;
  __syncthreads();
  const int a = s_a, c = s_c, lb0 = s_lb0;
  const int m = a + (B - c);                                 // survivors outside the region = holes inside it
  // at most CI_NT kept indices fall in this CTA's CI_NT slots: they all sit in sel[lb0 .. lb0 + CI_NT)
  const int wn = min(CI_NT, B - lb0);
  if (tid < wn) s_win[tid] = sel[lb0 + tid];
  __syncthreads();
  // the list must be strictly ascending for the plan to be conflict-free
  if (tid + 1 < wn && s_win[tid + 1] <= s_win[tid]) report(status, ACTKV_E_BADINDEX, r, s_win[tid + 1]);

  const int32_t p = p0 + tid;
  bool hole = false;
  int32_t src_pos = -1;
  if (p < end) {
    const int w = lower_bound_i32(s_win, wn, p);             // #kept in [p0, p)
    const bool kept = w < wn && s_win[w] == p;
    if (kept) {
      if (ord) ord[p - start] = p;
    } else {
      const int j = (p - start) - (lb0 + w - a);             // rank of this hole
      if (j < 0 || j >= m) {
        report(status, ACTKV_E_BADINDEX, r, p);
      } else {
        src_pos = j < a ? sel[j] : sel[c + (j - a)];
        if ((uint32_t)src_pos >= (uint32_t)L || (src_pos >= start && src_pos < end)) {
          report(status, ACTKV_E_BADINDEX, r, src_pos);
        } else {
          hole = true;
          if (ord) ord[p - start] = src_pos;
        }
      }
    }
  }
  // a move whose source or destination page id is out of range is dropped (and reported): nothing is read
  // from or written to a page the request does not own
  int32_t sp = -1, dp = -1;
  if (hole) {
    sp = page_or_neg(tab, pool.n_pages, r, src_pos / P, status);
    dp = page_or_neg(tab, pool.n_pages, r, p / P, status);
    if (sp < 0 || dp < 0) hole = false;
  }
  // pack this CTA's moves (their order within the CTA does not matter)
  const uint32_t bal = __ballot_sync(0xffffffffu, hole);
  int wbase = 0;
  if (lane == 0 && bal) wbase = atomicAdd(&s_cnt, __popc(bal));
  wbase = __shfl_sync(0xffffffffu, wbase, 0);
  if (hole) {
    const int k = wbase + __popc(bal & ((1u << lane) - 1u));
    s_src[k] = (int64_t)sp * pool.stride_page + (int64_t)(src_pos % P) * pool.stride_slot + (int64_t)h * pool.stride_head;
    s_dst[k] = (int64_t)dp * pool.stride_page + (int64_t)(p % P) * pool.stride_slot + (int64_t)h * pool.stride_head;
  }
  __syncthreads();
  const int cnt = s_cnt;
  __nv_bfloat16* lbase = const_cast<__nv_bfloat16*>(pool.base) + (int64_t)(layer_begin + slab) * pool.stride_layer;
  const int vpr = D / 8;
  const int per_kv = (VPR_SHIFT >= 0) ? (cnt << VPR_SHIFT) : cnt * vpr;
  const int total = 2 * per_kv;
  for (int v0 = tid; v0 < total; v0 += CI_NT * CI_UNROLL) {
    uint4 val[CI_UNROLL];
    int64_t doff[CI_UNROLL];
#pragma unroll
    for (int k = 0; k < CI_UNROLL; ++k) {
      const int v = v0 + k * CI_NT;
      doff[k] = -1;
      if (v < total) {
        const int kv = v >= per_kv ? 1 : 0;
        const int rem = v - kv * per_kv;
        const int i = (VPR_SHIFT >= 0) ? (rem >> VPR_SHIFT) : rem / vpr;
        const int dv = (VPR_SHIFT >= 0) ? (rem & ((1 << VPR_SHIFT) - 1)) : rem - i * vpr;
        const int64_t kvo = (int64_t)kv * pool.stride_kv + dv * 8;
        val[k] = *reinterpret_cast<const uint4*>(lbase + s_src[i] + kvo);
        doff[k] = s_dst[i] + kvo;
      }
    }
#pragma unroll
    for (int k = 0; k < CI_UNROLL; ++k)
      if (doff[k] >= 0) *reinterpret_cast<uint4*>(lbase + doff[k]) = val[k];
  }
}

// ---- deferred form --------------------------------------------------------------------------------
// Plan: items per request (32 region slots each; with an order output also the requests that are not
// compacted, whose order is the identity list), their prefix sums, and the job record.
__global__ void compact_inplace_plan_kernel(TablesView tab, PoolView pool, const int32_t* __restrict__ budget,
                                            int32_t max_keep, int32_t want_order, int32_t layer_begin, int32_t n_layers,
                                            int32_t vpr_shift, uint32_t* src_tab, uint32_t* dst_tab, int64_t tab_items,
                                            CompactWs* ws, int32_t* status) {
  if (threadIdx.x != 0) return;
  const int R = tab.n_req, P = pool.page_size;
  int32_t* item_off = ws_item_off(ws, R);
  bool ok = !status_set(status);
  int64_t off = 0;
  for (int r = 0; r < R; ++r) {
    item_off[r] = (int32_t)off;
    const int32_t L = tab.seq_len[r];
    const int32_t B = budget[r] < 0 ? 0 : budget[r];
    if (L < 0) { report(status, ACTKV_E_INVALID, r, L); ok = false; continue; }
    if (B >= L) {
      if (want_order) off += (L + 31) / 32;
      continue;
    }
    const int Y = (L + P - 1) / P;
    if (Y > tab.max_pages || B > max_keep) { report(status, ACTKV_E_INVALID, r, Y > tab.max_pages ? L : B); ok = false; continue; }
    off += (B + 31) / 32;
  }
  item_off[R] = (int32_t)off;
  const int64_t per_slab = off * pool.n_kv_heads;
  const int64_t items = per_slab * n_layers;
  if (items > 0x7fffffff || items > tab_items) {         // (the host sized the tables for max_keep)
    if (ok) report(status, ACTKV_E_WORKSPACE, -1, (int32_t)min(items, (int64_t)0x7fffffff));
    ok = false;
  }
  ws->plan_ok = ok ? 1 : 0;
  ws->total_new = (int32_t)off;                 // items of one (layer, head)
  ws->next_item = 0u;
  ws->n_items = ok ? (int32_t)items : 0;
  ws->pool = pool;
  ws->tab = tab;
  ws->sel_idx = nullptr;
  ws->sel_stride = 0;
  ws->keep_indptr = nullptr;
  ws->budget = budget;
  ws->status = status;
  ws->layer_begin = layer_begin;
  ws->n_layers = n_layers;
  ws->vpr_shift = vpr_shift;
  ws->parts_per_page = 1;
  ws->role_items = 0;
  ws->pad = CJ_INPLACE_MARK;
  ws->src_tab = src_tab;
  ws->dst_tab = dst_tab;
  ws->items_per_slab = (int32_t)max((int64_t)1, min(per_slab, (int64_t)0x7fffffff));
  ws->pad2 = 0;
}

// One warp per item: the 32 region slots [32 chunk, 32 chunk + 32) of one (layer, head, request), classified as
// in the one-launch kernel above; a hole's move goes into the table as (source, destination) offsets in 16-byte
// units within the layer, everything else as CJ_NONE.
__global__ void __launch_bounds__(128) compact_inplace_resolve_kernel(
    CompactWs* ws, const int32_t* __restrict__ sel_idx, int64_t sel_stride, const int32_t* __restrict__ keep_indptr,
    int32_t* __restrict__ new_order) {
  const int lane = threadIdx.x & 31;
  const int64_t n = cj_count(ws);
  const PoolView& pool = ws->pool;
  const TablesView& tab = ws->tab;
  const int R = tab.n_req, H = pool.n_kv_heads, P = pool.page_size;
  const int32_t* item_off = ws_item_off(ws, R);
  const int per_head = ws->total_new, per_slab = ws->items_per_slab;
  int32_t* status = ws->status;
  for (int64_t item = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5); item < n; item += (int64_t)gridDim.x * 4) {
    const int slab = (int)(item / per_slab), rem = (int)(item - (int64_t)slab * per_slab);
    const int h = rem / per_head, rem2 = rem - h * per_head;
    int lo = 0, hi = R;                                  // item_off[lo] <= rem2 < item_off[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (item_off[mid] <= rem2) lo = mid; else hi = mid;
    }
    const int r = lo, chunk = rem2 - item_off[r];
    const int z = slab * H + h;
    const int32_t L = tab.seq_len[r];
    const int32_t B = ws->budget[r] < 0 ? 0 : ws->budget[r];
    const int32_t* sel = sel_idx + (int64_t)z * sel_stride + keep_indptr[r];
    int32_t* ord = new_order ? new_order + (int64_t)z * sel_stride + keep_indptr[r] : nullptr;
    uint32_t so = CJ_NONE, dof = CJ_NONE;
    if (B >= L) {                                        // not compacting: the order is the identity list
      const int i = chunk * 32 + lane;
      if (ord && i < L) ord[i] = sel[i];
    } else {
      const int Y = (L + P - 1) / P, X = (B + P - 1) / P;
      const int32_t start = (Y - X) * P, end = start + B;
      const int32_t p0 = start + chunk * 32, p = p0 + lane;
      int v = 0;
      if (lane == 0) v = lower_bound_i32(sel, B, start);
      if (lane == 1) v = lower_bound_i32(sel, B, end);
      if (lane == 2) v = lower_bound_i32(sel, B, p0);
      const int a = __shfl_sync(0xffffffffu, v, 0), c = __shfl_sync(0xffffffffu, v, 1), lb0 = __shfl_sync(0xffffffffu, v, 2);
      const int m = a + (B - c);                         // survivors outside the region = holes inside it
      // at most 32 kept indices fall in these 32 slots: they all sit in sel[lb0 .. lb0 + 32)
      const int wn = min(32, B - lb0);
      const int32_t win = lane < wn ? sel[lb0 + lane] : 0x7fffffff;
      const int32_t nxt = __shfl_down_sync(0xffffffffu, win, 1);
      if (lane + 1 < wn && nxt <= win) report(status, ACTKV_E_BADINDEX, r, nxt);      // must be strictly ascending
      int w = 0;                                         // #kept in [p0, p)
      bool kept = false;
#pragma unroll
      for (int k = 0; k < 32; ++k) {
        const int32_t x = __shfl_sync(0xffffffffu, win, k);
        w += (k < wn && x < p) ? 1 : 0;
        kept = kept || (k < wn && x == p);
      }
      if (p < end) {
        if (kept) {
          if (ord) ord[p - start] = p;
        } else {
          const int j = (p - start) - (lb0 + w - a);     // rank of this hole
          if (j < 0 || j >= m) {
            report(status, ACTKV_E_BADINDEX, r, p);
          } else {
            const int32_t src_pos = j < a ? sel[j] : sel[c + (j - a)];
            if ((uint32_t)src_pos >= (uint32_t)L || (src_pos >= start && src_pos < end)) {
              report(status, ACTKV_E_BADINDEX, r, src_pos);
            } else {
              if (ord) ord[p - start] = src_pos;
              // a move whose source or destination page id is out of range is dropped (and reported)
              const int32_t sp = page_or_neg(tab, pool.n_pages, r, src_pos / P, status);
              const int32_t dp = page_or_neg(tab, pool.n_pages, r, p / P, status);
              if (sp >= 0 && dp >= 0) {
                so = (uint32_t)(((int64_t)sp * pool.stride_page + (int64_t)(src_pos % P) * pool.stride_slot +
                                 (int64_t)h * pool.stride_head) >> 3);
                dof = (uint32_t)(((int64_t)dp * pool.stride_page + (int64_t)(p % P) * pool.stride_slot +
                                  (int64_t)h * pool.stride_head) >> 3);
              }
            }
          }
        }
      }
    }
    ws->src_tab[item * 32 + lane] = so;
    ws->dst_tab[item * 32 + lane] = dof;
  }
}

__global__ void compact_inplace_finalize_kernel(TablesView tab, int32_t page_size, int32_t n_pages,
                                                const int32_t* __restrict__ budget, int32_t* status) {
  if (status_set(status)) return;
  const int R = tab.n_req;
  __shared__ int32_t s_fc, s_ok;
  if (threadIdx.x == 0) {
    // every dropped page must fit on the free-list stack
    int64_t fc = *tab.free_count;
    bool ok = fc >= 0 && fc <= n_pages;
    for (int r = 0; r < R && ok; ++r) {
      const int32_t L = tab.seq_len[r];
      const int32_t B = budget[r] < 0 ? 0 : budget[r];
      if (B < L) fc += (L + page_size - 1) / page_size - (B + page_size - 1) / page_size;
    }
    if (!ok || fc > n_pages) { report(status, ACTKV_E_INVALID, -1, (int32_t)fc); ok = false; }
    s_ok = ok ? 1 : 0;
    s_fc = *tab.free_count;
  }
  __syncthreads();
  if (!s_ok) return;
  for (int r = 0; r < R; ++r) {
    const int32_t L = tab.seq_len[r];
    const int32_t B = budget[r] < 0 ? 0 : budget[r];
    if (B >= L) continue;                                    // uniform over the CTA
    const int Y = (L + page_size - 1) / page_size, X = (B + page_size - 1) / page_size;
    const int drop = Y - X;
    int32_t* row = tab.page_table + (int64_t)r * tab.max_pages;
    const int32_t fc = s_fc;
    for (int i = threadIdx.x; i < drop; i += blockDim.x) tab.free_list[fc + i] = row[i];
    __syncthreads();
    // shift the row left by `drop`, chunk by chunk in ascending order: a chunk reads at or above where
    // it writes and earlier chunks wrote strictly below, so reading before the barrier is safe
    for (int i0 = 0; i0 < tab.max_pages; i0 += blockDim.x) {
      const int i = i0 + threadIdx.x;
      int32_t v = -1;
      if (i < X) v = row[i + drop];
      __syncthreads();
      if (i < tab.max_pages) row[i] = v;
      __syncthreads();
    }
    if (threadIdx.x == 0) {
      tab.seq_len[r] = B;
      s_fc = fc + drop;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) *tab.free_count = s_fc;
}

}  // namespace actkv

namespace actkv {

static int inplace_check(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin, int32_t layer_end,
                         const int32_t* sel_idx, int64_t sel_stride, const int32_t* keep_indptr, const int32_t* budget,
                         int32_t max_keep) {
  if (!pool || !tables || !pool->base) return ACTKV_E_INVALID;
  if (layer_begin < 0 || layer_end > pool->n_layers || layer_begin > layer_end) return ACTKV_E_INVALID;
  if (pool->page_size <= 0 || pool->head_dim <= 0 || pool->head_dim % 8 != 0 || pool->n_kv_heads <= 0)
    return ACTKV_E_INVALID;
  if (((uintptr_t)pool->base & 15) || pool->stride_layer % 8 || pool->stride_kv % 8 || pool->stride_page % 8 ||
      pool->stride_slot % 8 || pool->stride_head % 8)
    return ACTKV_E_INVALID;
  const int R = tables->n_req;
  if (R < 0 || tables->max_pages < 0 || max_keep < 0 || sel_stride < 0) return ACTKV_E_INVALID;
  if (R == 0) return ACTKV_OK;
  if (!tables->page_table || !tables->seq_len || !tables->free_list || !tables->free_count || !budget ||
      !keep_indptr || !sel_idx)
    return ACTKV_E_INVALID;
  const int64_t nz = (int64_t)(layer_end - layer_begin) * pool->n_kv_heads;
  if (R > 65535 || nz > 65535) return ACTKV_E_INVALID;
  return ACTKV_OK;
}

// The whole copy of a call in one launch.
static int inplace_copy_all(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin, int32_t layer_end,
                            const int32_t* sel_idx, int64_t sel_stride, const int32_t* keep_indptr, const int32_t* budget,
                            int32_t max_keep, int32_t* new_order, int32_t* status, cudaStream_t s) {
  const int R = tables->n_req;
  const int64_t nz = (int64_t)(layer_end - layer_begin) * pool->n_kv_heads;
  PoolView pv = make_view(pool);
  TablesView tv = make_view(tables);
  if (nz > 0 && max_keep > 0) {
    dim3 grid((unsigned)((max_keep + CI_NT - 1) / CI_NT), (unsigned)R, (unsigned)nz);
    const int vpr = pool->head_dim / 8;
    if (vpr == 16)
      compact_inplace_copy_kernel<4><<<grid, CI_NT, 0, s>>>(pv, tv, layer_begin, sel_idx, sel_stride, keep_indptr, budget,
                                                            max_keep, new_order, status);
    else if (vpr == 8)
      compact_inplace_copy_kernel<3><<<grid, CI_NT, 0, s>>>(pv, tv, layer_begin, sel_idx, sel_stride, keep_indptr, budget,
                                                            max_keep, new_order, status);
    else if (vpr == 32)
      compact_inplace_copy_kernel<5><<<grid, CI_NT, 0, s>>>(pv, tv, layer_begin, sel_idx, sel_stride, keep_indptr, budget,
                                                            max_keep, new_order, status);
    else
      compact_inplace_copy_kernel<-1><<<grid, CI_NT, 0, s>>>(pv, tv, layer_begin, sel_idx, sel_stride, keep_indptr, budget,
                                                             max_keep, new_order, status);
    ACTKV_CHECK_LAUNCH();
  }
  return ACTKV_OK;
}

static int inplace_finalize(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_end, const int32_t* budget,
                            int32_t* status, cudaStream_t s) {
  if (layer_end == pool->n_layers) {
    compact_inplace_finalize_kernel<<<1, 1024, 0, s>>>(make_view(tables), pool->page_size, pool->n_pages, budget, status);
    ACTKV_CHECK_LAUNCH();
  }
  return ACTKV_OK;
}

// Items of the largest job these arguments allow, per layer.
static int64_t inplace_items_per_layer(const actkv_pool_t* pool, int32_t n_req, int32_t max_keep) {
  return (int64_t)pool->n_kv_heads * n_req * (((int64_t)max_keep + 31) / 32);
}
static size_t inplace_ws_base(int32_t n_req) {
  return align_up(sizeof(CompactWs) + sizeof(int32_t) * ((size_t)3 * n_req + 1), 256);
}

}  // namespace actkv

extern "C" {

int actkv_compact_inplace(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                          int32_t layer_end, const int32_t* sel_idx, int64_t sel_stride,
                          const int32_t* keep_indptr, const int32_t* budget, int32_t max_keep,
                          int32_t* new_order, int32_t* status, actkv_stream_t stream) {
  using namespace actkv;
  int rc = inplace_check(pool, tables, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr, budget, max_keep);
  if (rc != ACTKV_OK || tables->n_req == 0) return rc;
  cudaStream_t s = (cudaStream_t)stream;
  rc = inplace_copy_all(pool, tables, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr, budget, max_keep, new_order,
                        status, s);
  if (rc != ACTKV_OK) return rc;
  return inplace_finalize(pool, tables, layer_end, budget, status, s);
}

size_t actkv_compact_inplace_deferred_workspace_bytes(const actkv_pool_t* pool, int32_t n_req, int32_t n_layers_sub,
                                                      int32_t max_keep) {
  if (!pool || n_req < 0 || n_layers_sub < 0 || max_keep < 0 || pool->n_kv_heads <= 0) return 0;
  const int64_t items = actkv::inplace_items_per_layer(pool, n_req, max_keep) * n_layers_sub;
  return actkv::inplace_ws_base(n_req) + 2 * actkv::align_up((size_t)items * 32 * sizeof(uint32_t), 256);
}

int actkv_compact_inplace_begin(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                                int32_t layer_end, const int32_t* sel_idx, int64_t sel_stride,
                                const int32_t* keep_indptr, const int32_t* budget, int32_t max_keep,
                                int32_t* new_order, void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream) {
  using namespace actkv;
  int rc = inplace_check(pool, tables, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr, budget, max_keep);
  if (rc != ACTKV_OK || tables->n_req == 0) return rc;
  if (!ws || ws_bytes < inplace_ws_base(tables->n_req)) return ACTKV_E_WORKSPACE;
  cudaStream_t s = (cudaStream_t)stream;
  const int nl = layer_end - layer_begin;
  const int shift = deferrable_shift(pool);
  const int64_t items_max = inplace_items_per_layer(pool, tables->n_req, max_keep) * nl;
  const bool deferred = shift >= 0 && items_max <= 0x7fffffff &&
                        ws_bytes >= actkv_compact_inplace_deferred_workspace_bytes(pool, tables->n_req, nl, max_keep);
  const size_t base = inplace_ws_base(tables->n_req);
  const size_t tab_bytes = align_up((size_t)(deferred ? items_max : 0) * 32 * sizeof(uint32_t), 256);
  uint32_t* src_tab = (uint32_t*)((char*)ws + base);
  uint32_t* dst_tab = (uint32_t*)((char*)ws + base + tab_bytes);
  // (not deferred: an empty job, so that a score call given this workspace finds nothing to do; actkv_compact_inplace_end
  //  then copies everything itself)
  compact_inplace_plan_kernel<<<1, 32, 0, s>>>(make_view(tables), make_view(pool), budget, max_keep,
                                               new_order != nullptr ? 1 : 0, layer_begin, deferred ? nl : 0,
                                               deferred ? shift : -1, src_tab, dst_tab, deferred ? items_max : 0,
                                               (CompactWs*)ws, status);
  ACTKV_CHECK_LAUNCH();
  if (deferred && items_max > 0) {
    const int64_t ctas = std::min<int64_t>(std::max<int64_t>(1, (items_max + 3) / 4), 1 << 20);
    compact_inplace_resolve_kernel<<<(unsigned)ctas, 128, 0, s>>>((CompactWs*)ws, sel_idx, sel_stride, keep_indptr, new_order);
    ACTKV_CHECK_LAUNCH();
  }
  return ACTKV_OK;
}

int actkv_compact_inplace_end(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                              int32_t layer_end, const int32_t* sel_idx, int64_t sel_stride,
                              const int32_t* keep_indptr, const int32_t* budget, int32_t max_keep,
                              int32_t* new_order, void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream) {
  using namespace actkv;
  int rc = inplace_check(pool, tables, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr, budget, max_keep);
  if (rc != ACTKV_OK || tables->n_req == 0) return rc;
  if (!ws || ws_bytes < inplace_ws_base(tables->n_req)) return ACTKV_E_WORKSPACE;
  cudaStream_t s = (cudaStream_t)stream;
  const int nl = layer_end - layer_begin;
  const int shift = deferrable_shift(pool);
  const int64_t items_max = inplace_items_per_layer(pool, tables->n_req, max_keep) * nl;
  const bool deferred = shift >= 0 && items_max <= 0x7fffffff &&
                        ws_bytes >= actkv_compact_inplace_deferred_workspace_bytes(pool, tables->n_req, nl, max_keep);
  if (!deferred) {
    rc = inplace_copy_all(pool, tables, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr, budget, max_keep, new_order,
                          status, s);
    if (rc != ACTKV_OK) return rc;
  } else if (items_max > 0) {
    launch_drain((CompactWs*)ws, shift, items_max, s);
    ACTKV_CHECK_LAUNCH();
  }
  return inplace_finalize(pool, tables, layer_end, budget, status, s);
}

}  // extern "C"
