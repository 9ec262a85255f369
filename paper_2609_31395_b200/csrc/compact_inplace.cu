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
#include "common.cuh"

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

extern "C" {

int actkv_compact_inplace(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                          int32_t layer_end, const int32_t* sel_idx, int64_t sel_stride,
                          const int32_t* keep_indptr, const int32_t* budget, int32_t max_keep,
                          int32_t* new_order, int32_t* status, actkv_stream_t stream) {
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
  cudaStream_t s = (cudaStream_t)stream;
  actkv::PoolView pv = actkv::make_view(pool);
  actkv::TablesView tv = actkv::make_view(tables);
  if (nz > 0 && max_keep > 0) {
    dim3 grid((unsigned)((max_keep + actkv::CI_NT - 1) / actkv::CI_NT), (unsigned)R, (unsigned)nz);
    const int vpr = pool->head_dim / 8;
    if (vpr == 16)
      actkv::compact_inplace_copy_kernel<4><<<grid, actkv::CI_NT, 0, s>>>(pv, tv, layer_begin, sel_idx, sel_stride,
                                                                          keep_indptr, budget, max_keep, new_order, status);
    else if (vpr == 8)
      actkv::compact_inplace_copy_kernel<3><<<grid, actkv::CI_NT, 0, s>>>(pv, tv, layer_begin, sel_idx, sel_stride,
                                                                          keep_indptr, budget, max_keep, new_order, status);
    else if (vpr == 32)
      actkv::compact_inplace_copy_kernel<5><<<grid, actkv::CI_NT, 0, s>>>(pv, tv, layer_begin, sel_idx, sel_stride,
                                                                          keep_indptr, budget, max_keep, new_order, status);
    else
      actkv::compact_inplace_copy_kernel<-1><<<grid, actkv::CI_NT, 0, s>>>(pv, tv, layer_begin, sel_idx, sel_stride,
                                                                           keep_indptr, budget, max_keep, new_order, status);
    ACTKV_CHECK_LAUNCH();
  }
  if (layer_end == pool->n_layers) {
    actkv::compact_inplace_finalize_kernel<<<1, 1024, 0, s>>>(tv, pool->page_size, pool->n_pages, budget, status);
    ACTKV_CHECK_LAUNCH();
  }
  return ACTKV_OK;
}

}  // extern "C"
