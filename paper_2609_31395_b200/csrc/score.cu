// actkv_score: host entry point and path selection.
//   tensor-core path (score_tc.cuh): window x group rows >= 64 (any row count for the streaming update),
//   page 16, head_dim 128, packed pool;
//   FMA path (score_fma.cuh): everything else.
// actkv_score_accumulate (streaming, Algorithm 3 per decode step) runs the pooled-score pass alone against
// the supplied LSE and folds its result into the running mean held in the score array.
// Both write per-chunk (max, sum) partials of the LSE pass into the caller's workspace, merge them
// with lse_combine_kernel, then run the pooled-score pass against the merged (or supplied) LSE.
#include "score_fma.cuh"
#include "score_tc.cuh"

namespace actkv {

struct ScoreWsLayout {
  size_t lse_off, lse_bytes, part_off, part_bytes, total;
  int32_t rows_max, n_chunks;
};

static ScoreWsLayout score_ws_layout(int32_t n_kv_heads, int32_t n_req, int32_t nls, int32_t n_q_heads,
                                     int32_t sum_win, int32_t max_win, int32_t max_tok) {
  ScoreWsLayout l;
  const int G = n_q_heads / (n_kv_heads > 0 ? n_kv_heads : 1);
  l.rows_max = max_win * G;
  // Chunks per unit of a launch over `units` units: enough for LSE_ITEMS work items of at least
  // LSE_CHUNK_LONG keys, or for LSE_ITEMS_MIN items of at least LSE_CHUNK keys when that leaves SMs idle.  units x n_chunks <= LSE_ITEMS + 2 units, and that bound grows with the unit count,
  // so a workspace sized for a layer range also serves every call on fewer layers.
  const int64_t units = (int64_t)nls * n_kv_heads * n_req;
  const int64_t by_len = max_tok > 0 ? (max_tok + LSE_CHUNK - 1) / LSE_CHUNK : 1;
  const int64_t by_len_long = max_tok > 0 ? (max_tok + LSE_CHUNK_LONG - 1) / LSE_CHUNK_LONG : 1;
  int64_t nc = units > 0 ? (LSE_ITEMS + units - 1) / units : 1;
  if (nc > by_len_long) nc = by_len_long;
  if (units > 0 && units * nc < LSE_ITEMS_MIN) {   // a small problem: shorter chunks, so that every SM has work
    nc = (LSE_ITEMS_MIN + units - 1) / units;
    if (nc > by_len) nc = by_len;
  }
  if (nc < 1) nc = 1;
  l.n_chunks = (int32_t)nc;
  int64_t slots = units * by_len;
  if (slots > LSE_ITEMS + 2 * units) slots = LSE_ITEMS + 2 * units;
  l.lse_off = 0;
  l.lse_bytes = align_up((size_t)nls * sum_win * n_q_heads * 4, 256);
  l.part_off = l.lse_bytes;
  l.part_bytes = align_up((size_t)slots * l.rows_max * sizeof(float2), 256);
  l.total = l.part_off + l.part_bytes;
  return l;
}

}  // namespace actkv

extern "C" {

size_t actkv_score_workspace_bytes(const actkv_pool_t* pool, int32_t n_req, int32_t n_layers_sub,
                                   int32_t n_q_heads, int32_t sum_win, int32_t max_win, int32_t max_tok) {
  if (!pool || n_req < 0 || n_layers_sub < 0 || n_q_heads <= 0 || sum_win < 0 || max_win < 0 || max_tok < 0)
    return 0;
  return actkv::score_ws_layout(pool->n_kv_heads, n_req, n_layers_sub, n_q_heads, sum_win, max_win, max_tok).total;
}

// mode bit 0: run the LSE pass (+ merge) into `lse_dst`; bit 1: run the pooled-score pass with `lse_src`.
static int score_impl(int mode, const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                      int32_t layer_end, const void* q, const int32_t* win_indptr, int32_t n_q_heads,
                      const float* lse_in, float sm_scale, int32_t causal, const int32_t* tok_indptr,
                      float* score_out, float* lse_out, int32_t sum_win, int32_t max_win, int32_t sum_tok,
                      int32_t max_tok, void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream,
                      const int32_t* acc_steps = nullptr, void* copy_ws = nullptr, int32_t window_left = 0) {
  using namespace actkv;
  if (!pool || !tables || !pool->base) return ACTKV_E_INVALID;
  if (layer_begin < 0 || layer_end > pool->n_layers || layer_begin > layer_end) return ACTKV_E_INVALID;
  const int D = pool->head_dim, Hkv = pool->n_kv_heads, R = tables->n_req;
  if (D <= 0 || D % 8 != 0 || D > 256 || Hkv <= 0 || pool->page_size <= 0) return ACTKV_E_INVALID;
  if (n_q_heads <= 0 || n_q_heads % Hkv != 0) return ACTKV_E_INVALID;
  const int G = n_q_heads / Hkv;
  if (G > FMA_RQ) return ACTKV_E_INVALID;
  if (R < 0 || sum_win < 0 || max_win < 0 || sum_tok < 0 || max_tok < 0 || window_left < 0) return ACTKV_E_INVALID;
  if (((uintptr_t)pool->base & 15) || pool->stride_layer % 8 || pool->stride_page % 8 || pool->stride_slot % 8 ||
      pool->stride_head % 8 || ((uintptr_t)q & 15))
    return ACTKV_E_INVALID;
  const int nls = layer_end - layer_begin;
  if (R == 0 || nls == 0 || sum_tok == 0 || max_tok == 0) return ACTKV_OK;
  if (!q || !win_indptr || !tok_indptr || !tables->page_table || !tables->seq_len) return ACTKV_E_INVALID;
  if ((mode & 2) && !score_out) return ACTKV_E_INVALID;
  if (mode == 1 && !lse_out) return ACTKV_E_INVALID;
  if (acc_steps != nullptr && sum_win == 0) return ACTKV_OK;      // no request is inside an action region
  if (max_win <= 0 || sum_win <= 0) return ACTKV_E_INVALID;
  const ScoreWsLayout lay = score_ws_layout(Hkv, R, nls, n_q_heads, sum_win, max_win, max_tok);
  if (!ws || ws_bytes < lay.total) return ACTKV_E_WORKSPACE;
  cudaStream_t s = (cudaStream_t)stream;

  ScoreArgs a;
  a.pool = make_view(pool);
  a.tab = make_view(tables);
  a.q = (const __nv_bfloat16*)q;
  a.win_indptr = win_indptr;
  a.tok_indptr = tok_indptr;
  a.lse = nullptr;
  a.partials = (float2*)((char*)ws + lay.part_off);
  a.score_out = score_out;
  a.status = status;
  a.layer_begin = layer_begin;
  a.n_layers_sub = nls;
  a.n_q_heads = n_q_heads;
  a.group = G;
  a.sum_win = sum_win;
  a.sum_tok = sum_tok;
  a.rows_max = lay.rows_max;
  // Keys per LSE partial.  A CTA pays a fixed cost (operand set-up, pipeline fill and drain), so chunks
  // are as long as they can be while there are still many CTAs per SM (the last wave of a launch is
  // partly empty): whole key tiles, about equal, the chunk count of the workspace layout (a CTA covers
  // all rows of its unit).
  const bool use_tc = actkv_score_path(pool, n_q_heads, max_win, sm_scale, q, acc_steps != nullptr) == 1;
  {
    int n_chunks = lay.n_chunks;
    // tensor-core kernel: one CTA per SM is resident, so the launch runs in rounds of 148 CTAs; of the chunk
    // counts the workspace allows, take the one that wastes least (partly empty last round against a fixed
    // cost per CTA of about four key tiles: the Q blocks go to tensor memory, the pipeline fills and drains)
    if (use_tc && (mode & 1))
      n_chunks = tc::best_split((int64_t)nls * Hkv * R, (max_tok + tc::TK - 1) / tc::TK, 4, lay.n_chunks);
    int chunk = (max_tok + n_chunks - 1) / n_chunks;
    chunk = (chunk + 127) / 128 * 128;
    if (chunk < LSE_CHUNK) chunk = LSE_CHUNK;
    a.lse_chunk = chunk;
    a.n_chunks = (max_tok + chunk - 1) / chunk;    // <= lay.n_chunks
  }
  a.n_tiles = (max_tok + FMA_TK - 1) / FMA_TK;
  a.scale_log2 = sm_scale * kLog2e;
  a.causal = causal;
  a.win_left = window_left;
  a.acc_steps = acc_steps;
  const int64_t units = (int64_t)nls * Hkv * R;
  const float* lse = lse_in;
  if (mode & 1) {
    float* lse_buf = lse_out ? lse_out : (float*)((char*)ws + lay.lse_off);
    if (use_tc) {
      int rc = score_tc_launch_lse(a, pool, max_tok, max_win, s);
      if (rc != ACTKV_OK) return rc;
    } else {
      const int64_t grid1 = units * a.n_chunks;
      if (grid1 > 0x7fffffffLL) return ACTKV_E_INVALID;
      const size_t sm1 = score_fma_smem_bytes(D, lay.rows_max, 1);
      if (sm1 > 200 * 1024) return ACTKV_E_INVALID;
      if (ensure_dyn_smem(score_fma_kernel<1>, sm1) != cudaSuccess)
        return ACTKV_E_CUDA;
      score_fma_kernel<1><<<(unsigned)grid1, FMA_NT, sm1, s>>>(a);
      ACTKV_CHECK_LAUNCH();
    }
    const int64_t n_rows_all = units * lay.rows_max;
    lse_combine_kernel<<<(unsigned)((n_rows_all + 255) / 256), 256, 0, s>>>(a, lse_buf, nullptr);
    ACTKV_CHECK_LAUNCH();
    lse = lse_buf;
  } else if (lse_out != nullptr && lse_in != nullptr && lse_out != lse_in) {
    if (cudaMemcpyAsync(lse_out, lse_in, (size_t)nls * sum_win * n_q_heads * 4, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
      return ACTKV_E_CUDA;
  }
  if (!(mode & 2)) return ACTKV_OK;
  if (!lse) return ACTKV_E_INVALID;
  a.lse = lse;
  if (use_tc) return score_tc_launch_score(a, pool, max_tok, max_win, s, (CompactWs*)copy_ws);
  const int64_t grid2 = units * a.n_tiles;
  if (grid2 > 0x7fffffffLL) return ACTKV_E_INVALID;
  const size_t sm2 = score_fma_smem_bytes(D, lay.rows_max, 2);
  if (ensure_dyn_smem(score_fma_kernel<2>, sm2) != cudaSuccess)
    return ACTKV_E_CUDA;
  score_fma_kernel<2><<<(unsigned)grid2, FMA_NT, sm2, s>>>(a);
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

int actkv_score(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                int32_t layer_end, const void* q, const int32_t* win_indptr, int32_t n_q_heads,
                const float* lse_in, float sm_scale, int32_t causal, const int32_t* tok_indptr,
                float* score_out, float* lse_out, int32_t sum_win, int32_t max_win, int32_t sum_tok,
                int32_t max_tok, void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream) {
  return score_impl(lse_in ? 2 : 3, pool, tables, layer_begin, layer_end, q, win_indptr, n_q_heads, lse_in, sm_scale,
                    causal, tok_indptr, score_out, lse_out, sum_win, max_win, sum_tok, max_tok, ws, ws_bytes, status,
                    stream);
}

int actkv_score_overlap(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                        int32_t layer_end, const void* q, const int32_t* win_indptr, int32_t n_q_heads,
                        const float* lse_in, float sm_scale, int32_t causal, const int32_t* tok_indptr,
                        float* score_out, float* lse_out, int32_t sum_win, int32_t max_win, int32_t sum_tok,
                        int32_t max_tok, void* ws, size_t ws_bytes, void* pending_compact_ws, int32_t* status,
                        actkv_stream_t stream) {
  return score_impl(lse_in ? 2 : 3, pool, tables, layer_begin, layer_end, q, win_indptr, n_q_heads, lse_in, sm_scale,
                    causal, tok_indptr, score_out, lse_out, sum_win, max_win, sum_tok, max_tok, ws, ws_bytes, status,
                    stream, nullptr, pending_compact_ws);
}

int actkv_score_sliding(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                        int32_t layer_end, const void* q, const int32_t* win_indptr, int32_t n_q_heads,
                        const float* lse_in, float sm_scale, int32_t causal, int32_t window_left,
                        const int32_t* tok_indptr, float* score_out, float* lse_out, int32_t sum_win,
                        int32_t max_win, int32_t sum_tok, int32_t max_tok, void* ws, size_t ws_bytes,
                        int32_t* status, actkv_stream_t stream) {
  return score_impl(lse_in ? 2 : 3, pool, tables, layer_begin, layer_end, q, win_indptr, n_q_heads, lse_in, sm_scale,
                    causal, tok_indptr, score_out, lse_out, sum_win, max_win, sum_tok, max_tok, ws, ws_bytes, status,
                    stream, nullptr, nullptr, window_left);
}

int actkv_score_lse(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                    int32_t layer_end, const void* q, const int32_t* win_indptr, int32_t n_q_heads,
                    float sm_scale, int32_t causal, const int32_t* tok_indptr, float* lse_out,
                    int32_t sum_win, int32_t max_win, int32_t sum_tok, int32_t max_tok,
                    void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream) {
  return score_impl(1, pool, tables, layer_begin, layer_end, q, win_indptr, n_q_heads, nullptr, sm_scale, causal,
                    tok_indptr, nullptr, lse_out, sum_win, max_win, sum_tok, max_tok, ws, ws_bytes, status, stream);
}

int actkv_score_accumulate(const actkv_pool_t* pool, const actkv_tables_t* tables, int32_t layer_begin,
                           int32_t layer_end, const void* q, const int32_t* win_indptr, int32_t n_q_heads,
                           const float* lse_in, float sm_scale, int32_t causal, const int32_t* tok_indptr,
                           const int32_t* acc_steps, float* score_io, int32_t sum_win, int32_t max_win,
                           int32_t sum_tok, int32_t max_tok, void* ws, size_t ws_bytes, int32_t* status,
                           actkv_stream_t stream) {
  if (!lse_in || !acc_steps) return ACTKV_E_INVALID;
  return score_impl(2, pool, tables, layer_begin, layer_end, q, win_indptr, n_q_heads, lse_in, sm_scale, causal,
                    tok_indptr, score_io, nullptr, sum_win, max_win, sum_tok, max_tok, ws, ws_bytes, status, stream,
                    acc_steps);
}

int actkv_score_path(const actkv_pool_t* pool, int32_t n_q_heads, int32_t max_win, float sm_scale, const void* q,
                     int32_t streaming) {
  if (!pool || pool->n_kv_heads <= 0 || n_q_heads <= 0 || n_q_heads % pool->n_kv_heads != 0) return ACTKV_E_INVALID;
  const int G = n_q_heads / pool->n_kv_heads;
  return actkv::score_tc_supported(pool, G, max_win, sm_scale, q, streaming ? 1 : 64) ? 1 : 0;
}

int actkv_debug_inject_stall(int32_t after_tile, int32_t wait_limit_us) {
  auto& h = actkv::tc::stall_hook();
  if (after_tile < 0) {
    h.stall_tile.store(-1);
    h.wait_cycles.store(actkv::tc::WAIT_LIMIT_CYCLES);
    return ACTKV_OK;
  }
  if (wait_limit_us <= 0) return ACTKV_E_INVALID;
  h.wait_cycles.store((long long)wait_limit_us * 2100ll);       // cycles at the highest SM clock
  h.stall_tile.store(after_tile);
  return ACTKV_OK;
}

const char* actkv_version(void) { return "actkv-b200 0.2 (sm_100a)"; }

}  // extern "C"
