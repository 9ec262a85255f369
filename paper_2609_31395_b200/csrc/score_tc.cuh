// Tensor-core path of actkv_score for sm_100a: tcgen05.mma with TMEM accumulators, operands
// staged by TMA (cp.async.bulk.tensor, 128-byte swizzle) straight from the paged pool through the
// block table, one TMA box per (page, half of the head dimension).
//
// Two kernels, both warp-specialised (warp 0: TMA producer, warp 1: MMA issuer + TMEM owner,
// the other warps: epilogue reading TMEM with tcgen05.ld):
//
//  * LSE pass (score_tc_lse.cuh; Section 7.1, LSE equation).  D[row, key] = Q K^T with the window x
//    group rows on the TMEM lanes (Q as the A operand from tensor memory), so every epilogue thread
//    owns one row per 128-row block and keeps its running (max, sum of exp2) in registers: no shuffles.
//  * Pooled-score pass (score_tc_pool.cuh; Section 7.1 recovery identity, Algorithm 3 steps 3-5).
//    The transposed product D[key, row] = K Q^T with the keys on the lanes and row = w*G + g on the
//    columns, so the max over the GQA group and the sum over the action tokens run inside one
//    thread.  Because exp is monotone the max over the group is taken on (s - lse) BEFORE the exp:
//    W exps per key instead of W*G.
//
// Every wait on an mbarrier is bounded (wall-clock limit); on give-up the kernel records
// ACTKV_E_TIMEOUT in the status word, every role leaves its loop, outstanding MMAs are drained,
// TMEM is freed and the CTA returns.
//
// This file: tensor-map creation and launch configuration (host side).
#pragma once

#include <algorithm>
#include <atomic>

#include "score_tc_lse.cuh"
#include "score_tc_pool.cuh"

namespace actkv {
namespace tc {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is looked up through the runtime, so the library does not link libcuda.
inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return (EncodeTiledFn)p;
  }();
  return fn;
}

// The four-dimensional K map needs the slots of consecutive pages to continue at the slot stride.
inline bool pool_needs_5d(const actkv_pool_t* pool) { return pool->stride_page != (int64_t)pool->page_size * pool->stride_slot; }

inline int pow2_at_least(int g) { int p = 1; while (p < g) p <<= 1; return p; }

// CTAs per unit for a launch over `units` units of `tiles` key tiles each.  One CTA is resident per SM, so a
// launch runs in rounds of 148 CTAs and the last round is partly empty; more CTAs make that round
// cheaper, but every CTA pays a fixed cost (operand set-up, pipeline fill and drain) of about `ovh` key
// tiles' worth.  Returns the count in [1, n_max] with the best product of the two, preferring fewer CTAs
// unless more are clearly better.
inline int best_split(int64_t units, int tiles, int ovh, int n_max) {
  int best = 1;
  double best_eff = 0.0;
  if (units < 1) units = 1;
  for (int n = 1; n <= n_max; ++n) {
    const int tpc = (tiles + n - 1) / n;
    if (tpc < 1) break;
    const int64_t grid = units * ((tiles + tpc - 1) / tpc);
    const int64_t rounds = (grid + 147) / 148;
    const double eff = (double)grid / (double)(rounds * 148) * (double)tpc / (double)(tpc + ovh);
    if (eff > best_eff * 1.005) { best_eff = eff; best = n; }
  }
  return best;
}

inline bool make_maps(const actkv_pool_t* pool, const void* q, int nls, int sum_win, int n_q_heads, int G,
                      CUtensorMap* kmap, CUtensorMap* qmap) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  {
    // K half of the pool.  Slot-major pages whose slots continue across pages: [layer][slot (page*16 + s)]
    // [head][dim], four dimensions (measured 13 % faster than five on the K stream).  Any other page layout
    // (head-major pages): [layer][page][head][slot][dim] with the caller's strides.  A box is one page of
    // one head, 64 dims: page_size rows of 128 B.
    CUresult res;
    if (!pool_needs_5d(pool)) {
      cuuint64_t dims[4] = {(cuuint64_t)pool->head_dim, (cuuint64_t)pool->n_kv_heads, (cuuint64_t)pool->n_pages * pool->page_size,
                            (cuuint64_t)pool->n_layers};
      cuuint64_t strides[3] = {(cuuint64_t)pool->stride_head * 2, (cuuint64_t)pool->stride_slot * 2,
                               (cuuint64_t)pool->stride_layer * 2};
      cuuint32_t box[4] = {64, 1, (cuuint32_t)pool->page_size, 1};
      cuuint32_t es[4] = {1, 1, 1, 1};
      res = enc(kmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, pool->base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
      cuuint64_t dims[5] = {(cuuint64_t)pool->head_dim, (cuuint64_t)pool->page_size, (cuuint64_t)pool->n_kv_heads,
                            (cuuint64_t)pool->n_pages, (cuuint64_t)pool->n_layers};
      cuuint64_t strides[4] = {(cuuint64_t)pool->stride_slot * 2, (cuuint64_t)pool->stride_head * 2,
                               (cuuint64_t)pool->stride_page * 2, (cuuint64_t)pool->stride_layer * 2};
      cuuint32_t box[5] = {64, (cuuint32_t)pool->page_size, 1, 1, 1};
      cuuint32_t es[5] = {1, 1, 1, 1, 1};
      res = enc(kmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, pool->base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (res != CUDA_SUCCESS) return false;
  }
  {
    // q: [slab*sum_win + w][q head][128]; a box is (64 dims, the G heads of one group, 128/G window rows)
    const cuuint64_t D = (cuuint64_t)pool->head_dim;
    cuuint64_t dims[3] = {D, (cuuint64_t)n_q_heads, (cuuint64_t)nls * sum_win};
    cuuint64_t strides[2] = {D * 2, (cuuint64_t)n_q_heads * D * 2};
    const int Gp = pow2_at_least(G);                 // the pooled-score kernel pads a group to a power of two
    cuuint32_t box[3] = {64, (cuuint32_t)Gp, (cuuint32_t)(128 / Gp)};
    cuuint32_t es[3] = {1, 1, 1};
    if (enc(qmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  return true;
}

constexpr size_t SMEM_LIMIT = 232448;        // 227 KB of dynamic shared memory per CTA

// Fault-injection hook of the bounded waits (actkv_debug_inject_stall): while stall_tile >= 0 the K-tile
// producers of every tensor-core score launch issue no tile from that one on, and every wait gives up after
// `wait_cycles`.  Process-wide, read at launch.
struct StallHook {
  std::atomic<int32_t> stall_tile{-1};
  std::atomic<long long> wait_cycles{WAIT_LIMIT_CYCLES};
};
inline StallHook& stall_hook() { static StallHook h; return h; }
inline void apply_hook(TcArgs& ta) {
  ta.stall_tile = stall_hook().stall_tile.load();
  ta.wait_cycles = stall_hook().wait_cycles.load();
}

}  // namespace tc

// The tensor-core path takes: pages of 16, 32, 64 or 128 tokens, head_dim 128 or 64, slot-major or head-major pages (any strides that are
// multiples of 16 bytes), 128-byte aligned
// base, group size <= 32 (padded to a power of two in the pooled-score pass), min_rows <= window x group rows <= 4096 (a CTA handles up to 512;
// more are taken in groups of 512 rows), positive softmax scale.
// The full score (LSE + pooled pass) takes it from 64 rows up; the streaming update, which runs the
// pooled pass alone and is bound by the K reads, from a single row.
inline bool score_tc_supported(const actkv_pool_t* p, int G, int max_win, float sm_scale, const void* q,
                               int min_rows = 64) {
  if (p->page_size != 16 && p->page_size != 32 && p->page_size != 64 && p->page_size != 128) return false;
  if (p->head_dim != 128 && p->head_dim != 64) return false;
  // TMA: every stride a positive multiple of 16 bytes (any page layout with contiguous head dimensions)
  if (p->stride_head <= 0 || p->stride_slot <= 0 || p->stride_page <= 0 || p->stride_layer <= 0) return false;
  if ((p->stride_head % 8) || (p->stride_slot % 8) || (p->stride_page % 8) || (p->stride_layer % 8)) return false;
  if (((uintptr_t)p->base & 127) || ((uintptr_t)q & 127)) return false;
  if (G < 1 || G > 32) return false;
  if (max_win * G < min_rows) return false;
  const int rows = max_win * tc::pow2_at_least(G);     // rows of the pooled-score pass (groups padded to a power of two)
  if (rows > tc::MAX_ROWS_TOTAL) return false;
  if (!(sm_scale > 0.f)) return false;
  return tc::encode_fn() != nullptr;
}

inline int score_tc_launch_lse_c(const CUtensorMap& kmap, const tc::TcArgs& ta, unsigned grid, size_t smem, cudaStream_t s) {
  constexpr int NPOLY = tc::LSE_NPOLY;
  const bool rgs = ta.n_rg > 1, d64 = ta.a.pool.head_dim == 64;
  const bool win = ta.a.win_left > 0;
  auto kern = win ? (rgs ? (d64 ? tc::score_tc_lse_kernel<NPOLY, true, 1, true> : tc::score_tc_lse_kernel<NPOLY, true, 2, true>)
                         : (d64 ? tc::score_tc_lse_kernel<NPOLY, false, 1, true> : tc::score_tc_lse_kernel<NPOLY, false, 2, true>))
                  : (rgs ? (d64 ? tc::score_tc_lse_kernel<NPOLY, true, 1, false> : tc::score_tc_lse_kernel<NPOLY, true, 2, false>)
                         : (d64 ? tc::score_tc_lse_kernel<NPOLY, false, 1, false> : tc::score_tc_lse_kernel<NPOLY, false, 2, false>));
  if (ensure_dyn_smem(kern, smem) != cudaSuccess) return ACTKV_E_CUDA;
  kern<<<grid, tc::LSE_THREADS, smem, s>>>(kmap, ta);
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

inline int score_tc_launch_lse(ScoreArgs& a, const actkv_pool_t* pool, int max_tok, int max_win, cudaStream_t s) {
  (void)max_tok;
  CUtensorMap kmap, qmap;
  if (!tc::make_maps(pool, a.q, a.n_layers_sub, a.sum_win, a.n_q_heads, a.group, &kmap, &qmap)) return ACTKV_E_CUDA;
  tc::TcArgs ta;
  ta.a = a;
  ta.n_rg = (max_win * a.group + tc::MAX_ROWS - 1) / tc::MAX_ROWS;
  ta.row_begin = 0;
  ta.k5 = tc::pool_needs_5d(pool) ? 1 : 0;
  ta.n_stages = 6;
  ta.tiles_per_cta = 0;
  ta.n_kchunks = 0;
  ta.copy_ws = nullptr;              // (this kernel has no copy role)
  tc::apply_hook(ta);
  const int64_t units = (int64_t)a.n_layers_sub * a.pool.n_kv_heads * a.tab.n_req;
  const int64_t grid = units * a.n_chunks * ta.n_rg;
  if (grid > 0x7fffffffLL) return ACTKV_E_INVALID;
  const size_t smem = (size_t)ta.n_stages * tc::KTILE_BYTES + sizeof(tc::LseBarriers);
  return score_tc_launch_lse_c(kmap, ta, (unsigned)grid, smem, s);
}

template <int G>
inline int score_tc_launch_pool_g(const CUtensorMap& kmap, const CUtensorMap& qmap, const tc::TcArgs& ta, unsigned grid,
                                  size_t smem, cudaStream_t s) {
  auto kern = ta.a.pool.head_dim == 64 ? tc::score_tc_pool_kernel<G, 1> : tc::score_tc_pool_kernel<G, 2>;
  // The warpgroups of this kernel re-divide the registers the launch allocates; the epilogue warpgroups would
  // wait for ever for registers that a smaller allocation does not have, so the allocation is checked first.
  if (kernel_num_regs(kern) < tc::POOL_REGS_ENTRY) return ACTKV_E_CUDA;
  if (ensure_dyn_smem(kern, smem) != cudaSuccess) return ACTKV_E_CUDA;
  kern<<<grid, tc::POOL_THREADS, smem, s>>>(kmap, qmap, ta);
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

inline int score_tc_launch_score(ScoreArgs& a, const actkv_pool_t* pool, int max_tok, int max_win, cudaStream_t s,
                                 CompactWs* copy_ws) {
  CUtensorMap kmap, qmap;
  if (!tc::make_maps(pool, a.q, a.n_layers_sub, a.sum_win, a.n_q_heads, a.group, &kmap, &qmap)) return ACTKV_E_CUDA;
  tc::TcArgs ta;
  ta.a = a;
  const int Gp = tc::pow2_at_least(a.group);
  const int rows_all = max_win * Gp;
  const int rows_pad = (std::min(rows_all, tc::MAX_ROWS) + 127) & ~127;      // per launch
  const int n_rc = (rows_pad + 255) / 256;
  const size_t q_bytes = (size_t)n_rc * 2 * tc::QBLK_BYTES;
  const size_t fixed = q_bytes + tc::MAX_ROWS * 4 + sizeof(tc::PoolBarriers);
  int stages = (int)((tc::SMEM_LIMIT - fixed) / tc::KTILE_BYTES);
  if (stages > 6) stages = 6;
  if (stages < 2) return ACTKV_E_INVALID;
  ta.n_stages = stages;
  ta.n_rg = 0;
  ta.k5 = tc::pool_needs_5d(pool) ? 1 : 0;
  ta.copy_ws = copy_ws;
  tc::apply_hook(ta);
  const int64_t units = (int64_t)a.n_layers_sub * a.pool.n_kv_heads * a.tab.n_req;
  const int max_tiles = (max_tok + tc::TK - 1) / tc::TK;
  // CTAs per unit: one CTA per SM is resident, so the launch runs in rounds of 148 CTAs and the last round
  // is partly empty; more CTAs make that round cheaper, but every CTA pays for its Q load and its pipeline
  // fill (about three key tiles' worth).  Take the count with the best product of the two.
  ta.n_kchunks = tc::best_split(units, max_tiles, 3, std::min(64, std::max(1, max_tiles / 4)));
  ta.tiles_per_cta = (max_tiles + ta.n_kchunks - 1) / ta.n_kchunks;
  ta.n_kchunks = (max_tiles + ta.tiles_per_cta - 1) / ta.tiles_per_cta;
  const int64_t grid = units * ta.n_kchunks;
  if (grid > 0x7fffffffLL) return ACTKV_E_INVALID;
  const size_t smem = fixed + (size_t)stages * tc::KTILE_BYTES;
  // a window of more than MAX_ROWS rows: one launch per group of MAX_ROWS rows (whole action tokens), in
  // stream order; the first writes the score, the others add their share of the mean
  for (int row_begin = 0; row_begin < rows_all; row_begin += tc::MAX_ROWS) {
    ta.row_begin = row_begin;
    int rc = ACTKV_E_INVALID;
    switch (Gp) {
      case 1: rc = score_tc_launch_pool_g<1>(kmap, qmap, ta, (unsigned)grid, smem, s); break;
      case 2: rc = score_tc_launch_pool_g<2>(kmap, qmap, ta, (unsigned)grid, smem, s); break;
      case 4: rc = score_tc_launch_pool_g<4>(kmap, qmap, ta, (unsigned)grid, smem, s); break;
      case 8: rc = score_tc_launch_pool_g<8>(kmap, qmap, ta, (unsigned)grid, smem, s); break;
      case 16: rc = score_tc_launch_pool_g<16>(kmap, qmap, ta, (unsigned)grid, smem, s); break;
      case 32: rc = score_tc_launch_pool_g<32>(kmap, qmap, ta, (unsigned)grid, smem, s); break;
      default: break;
    }
    if (rc != ACTKV_OK) return rc;
  }
  return ACTKV_OK;
}

}  // namespace actkv
