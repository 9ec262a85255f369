// actkv_step_host: one whole compression step for a caller whose per-step inputs live in HOST memory.
// Copies queries, logits, index arrays, budgets and tables to the caller's device staging buffers,
// runs budget -> keep_indptr -> (lse, score, select, compact) per layer group through the library's
// own entry points, copies the new tables / budgets / status back and synchronises the stream.
// The KV pool itself stays in HBM: it is the cache being compressed.
#include "common.cuh"

#define ACTKV_TRY(expr)            \
  do {                             \
    int rc__ = (expr);             \
    if (rc__ != ACTKV_OK) return rc__; \
  } while (0)

static int h2d(void* dst, const void* src, size_t n, cudaStream_t s) {
  if (n == 0) return ACTKV_OK;
  if (!dst || !src) return ACTKV_E_INVALID;
  return cudaMemcpyAsync(dst, src, n, cudaMemcpyHostToDevice, s) == cudaSuccess ? ACTKV_OK : ACTKV_E_CUDA;
}
static int d2h(void* dst, const void* src, size_t n, cudaStream_t s) {
  if (n == 0 || !dst) return ACTKV_OK;
  if (!src) return ACTKV_E_INVALID;
  return cudaMemcpyAsync(dst, src, n, cudaMemcpyDeviceToHost, s) == cudaSuccess ? ACTKV_OK : ACTKV_E_CUDA;
}

extern "C" int actkv_step_host(const actkv_pool_t* pool, const actkv_tables_t* tab,
                               const actkv_budget_params_t* params, const actkv_host_step_t* io,
                               actkv_stream_t stream) {
  if (!pool || !tab || !io) return ACTKV_E_INVALID;
  cudaStream_t s = (cudaStream_t)stream;
  const int R = tab->n_req, NL = pool->n_layers, Hkv = pool->n_kv_heads;
  if (R <= 0 || NL <= 0 || io->sum_win <= 0 || io->sum_tok <= 0) return ACTKV_E_INVALID;
  const size_t q_bytes = (size_t)NL * io->sum_win * io->n_q_heads * pool->head_dim * 2;
  const size_t tbl_bytes = (size_t)R * tab->max_pages * 4;

  // ---- host -> device: this step's inputs ----
  ACTKV_TRY(h2d(io->q_dev, io->q_host, q_bytes, s));
  ACTKV_TRY(h2d(io->win_indptr_dev, io->win_indptr_host, (size_t)(R + 1) * 4, s));
  ACTKV_TRY(h2d(io->tok_indptr_dev, io->tok_indptr_host, (size_t)(R + 1) * 4, s));
  ACTKV_TRY(h2d(io->budget_dev, io->budget_in_host, (size_t)R * 4, s));
  ACTKV_TRY(h2d(tab->page_table, io->page_table_host, tbl_bytes, s));
  ACTKV_TRY(h2d(tab->seq_len, io->seq_len_host, (size_t)R * 4, s));
  ACTKV_TRY(h2d(tab->free_list, io->free_list_host, (size_t)pool->n_pages * 4, s));
  ACTKV_TRY(h2d(tab->free_count, io->free_count_host, 4, s));
  if (cudaMemsetAsync(io->status_dev, 0, 16, s) != cudaSuccess) return ACTKV_E_CUDA;

  // ---- the path ----
  if (io->logits_host != nullptr && io->n_rows > 0) {
    if (!params) return ACTKV_E_INVALID;
    ACTKV_TRY(h2d(io->logits_dev, io->logits_host, (size_t)io->n_rows * io->vocab * 4, s));
    ACTKV_TRY(h2d(io->logit_indptr_dev, io->logit_indptr_host, (size_t)(R + 1) * 4, s));
    ACTKV_TRY(actkv_budget(io->logits_dev, io->logit_indptr_dev, io->n_rows, io->vocab, io->conf_hist_dev,
                           io->hist_len_dev, io->hist_cap, params, tab->seq_len, io->budget_dev, io->budget_dev,
                           nullptr, R, io->ws_budget, io->ws_budget_bytes, io->status_dev, stream));
  }
  ACTKV_TRY(actkv_keep_indptr(tab->seq_len, io->budget_dev, R, io->keep_indptr_dev, stream));
  const int lpc = io->layers_per_call > 0 ? (io->layers_per_call < NL ? io->layers_per_call : NL) : NL;
  for (int l0 = 0; l0 < NL; l0 += lpc) {
    const int l1 = l0 + lpc < NL ? l0 + lpc : NL;
    const char* q_l = (const char*)io->q_dev + (size_t)l0 * io->sum_win * io->n_q_heads * pool->head_dim * 2;
    float* lse_l = io->lse_dev + (size_t)l0 * io->sum_win * io->n_q_heads;
    ACTKV_TRY(actkv_score_lse(pool, tab, l0, l1, q_l, io->win_indptr_dev, io->n_q_heads, io->sm_scale, io->causal,
                              io->tok_indptr_dev, lse_l, io->sum_win, io->max_win, io->sum_tok, io->max_tok,
                              io->ws_score, io->ws_score_bytes, io->status_dev, stream));
    ACTKV_TRY(actkv_score(pool, tab, l0, l1, q_l, io->win_indptr_dev, io->n_q_heads, lse_l, io->sm_scale, io->causal,
                          io->tok_indptr_dev, io->score_dev, nullptr, io->sum_win, io->max_win, io->sum_tok,
                          io->max_tok, io->ws_score, io->ws_score_bytes, io->status_dev, stream));
    ACTKV_TRY(actkv_select(io->score_dev, io->tok_indptr_dev, io->sum_tok, io->budget_dev, (l1 - l0) * Hkv, R,
                           io->keep_indptr_dev, io->sel_idx_dev, io->sel_stride, nullptr, nullptr, nullptr, 0,
                           io->status_dev, stream));
    ACTKV_TRY(actkv_compact(pool, tab, l0, l1, io->sel_idx_dev, io->sel_stride, io->keep_indptr_dev, io->budget_dev,
                            io->max_keep, io->ws_compact, io->ws_compact_bytes, io->status_dev, stream));
  }

  // ---- device -> host: the step's results ----
  ACTKV_TRY(d2h(io->page_table_out_host, tab->page_table, tbl_bytes, s));
  ACTKV_TRY(d2h(io->seq_len_out_host, tab->seq_len, (size_t)R * 4, s));
  ACTKV_TRY(d2h(io->free_list_out_host, tab->free_list, (size_t)pool->n_pages * 4, s));
  ACTKV_TRY(d2h(io->free_count_out_host, tab->free_count, 4, s));
  ACTKV_TRY(d2h(io->budget_out_host, io->budget_dev, (size_t)R * 4, s));
  ACTKV_TRY(d2h(io->status_out_host, io->status_dev, 16, s));
  if (cudaStreamSynchronize(s) != cudaSuccess) return ACTKV_E_CUDA;
  return ACTKV_OK;
}
