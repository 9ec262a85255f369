// actkv_step_host: one whole compression step for a caller whose per-step inputs live in HOST memory.
// Copies queries, logits, index arrays, budgets and tables to the caller's device staging buffers,
// runs budget -> keep_indptr -> (lse, score, select, compact) per layer group through the library's
// own entry points, copies the new tables / budgets / status back and synchronises the stream.
// The KV pool itself stays in HBM: it is the cache being compressed.
//
// The large inputs (queries, logits) cross the host link on a copy stream of the library while the
// score kernels already run: the queries go first, one layer group at a time, and the LSE pass of a
// group starts as soon as its queries have landed (the first group is short, so that this is soon);
// the logits follow, the budget monitor runs on a side stream when they are in, and the first select,
// which is the first kernel to need the budgets, comes after the last LSE pass and the first
// pooled-score pass.  All side work is joined into the caller's stream before the results are copied
// back.
#include <mutex>

#include "common.cuh"

#define ACTKV_TRY(expr)            \
  do {                             \
    int rc__ = (expr);             \
    if (rc__ != ACTKV_OK) return rc__; \
  } while (0)

namespace {

constexpr int kMaxDevices = 64;
constexpr int kMaxGroups = 64;
constexpr int kDefaultGroupLayers = 16;      // layer-group size when the caller leaves it open

struct StepStreams {
  bool ready = false;
  cudaStream_t copy = nullptr, side = nullptr;
  cudaEvent_t start = nullptr, small = nullptr, logits = nullptr, budget = nullptr, q[kMaxGroups] = {nullptr};
};
std::mutex g_mutex;
StepStreams g_streams[kMaxDevices];

// Streams and events of the current device, created on first use.
StepStreams* step_streams() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_mutex);
  StepStreams& st = g_streams[dev];
  if (!st.ready) {
    if (cudaStreamCreateWithFlags(&st.copy, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithFlags(&st.side, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    cudaEvent_t* evs[4] = {&st.start, &st.small, &st.logits, &st.budget};
    for (cudaEvent_t* e : evs)
      if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    for (int g = 0; g < kMaxGroups; ++g)
      if (cudaEventCreateWithFlags(&st.q[g], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    st.ready = true;
  }
  return &st;
}

int h2d(void* dst, const void* src, size_t n, cudaStream_t s) {
  if (n == 0) return ACTKV_OK;
  if (!dst || !src) return ACTKV_E_INVALID;
  return cudaMemcpyAsync(dst, src, n, cudaMemcpyHostToDevice, s) == cudaSuccess ? ACTKV_OK : ACTKV_E_CUDA;
}
int d2h(void* dst, const void* src, size_t n, cudaStream_t s) {
  if (n == 0 || !dst) return ACTKV_OK;
  if (!src) return ACTKV_E_INVALID;
  return cudaMemcpyAsync(dst, src, n, cudaMemcpyDeviceToHost, s) == cudaSuccess ? ACTKV_OK : ACTKV_E_CUDA;
}
int record(cudaEvent_t e, cudaStream_t s) { return cudaEventRecord(e, s) == cudaSuccess ? ACTKV_OK : ACTKV_E_CUDA; }
int wait(cudaStream_t s, cudaEvent_t e) { return cudaStreamWaitEvent(s, e, 0) == cudaSuccess ? ACTKV_OK : ACTKV_E_CUDA; }

}  // namespace

// The passes that follow the LSE pass, in layer groups of layers_per_call layers: pooled score, select, compaction.
// The budgets are first needed by the first select (`budget_ready`: an event to wait for before it, or nullptr).
// With several layer groups the copies of group g run inside the pooled-score kernel of group g + 1
// (actkv_compact_begin / actkv_score_overlap / actkv_compact_end); one index buffer suffices because the copies of
// g are closed before the select of g + 1.
static int step_groups(const actkv_pool_t* pool, const actkv_tables_t* tab, const actkv_host_step_t* io,
                       actkv_stream_t stream, cudaEvent_t budget_ready) {
  cudaStream_t s = (cudaStream_t)stream;
  const int R = tab->n_req, NL = pool->n_layers, Hkv = pool->n_kv_heads;
  const int lpc_post = io->layers_per_call > 0 && io->layers_per_call < NL ? io->layers_per_call : NL;
  const int n_groups = (NL + lpc_post - 1) / lpc_post;
  const size_t q_layer_bytes = (size_t)io->sum_win * io->n_q_heads * pool->head_dim * 2;
  int pl0 = -1, pl1 = -1;                      // the group whose compaction is pending
  for (int g = 0; g < n_groups; ++g) {
    const int l0 = g * lpc_post, l1 = l0 + lpc_post < NL ? l0 + lpc_post : NL;
    ACTKV_TRY(actkv_score_overlap(pool, tab, l0, l1, (const char*)io->q_dev + (size_t)l0 * q_layer_bytes, io->win_indptr_dev,
                                  io->n_q_heads, io->lse_dev + (size_t)l0 * io->sum_win * io->n_q_heads, io->sm_scale,
                                  io->causal, io->tok_indptr_dev, io->score_dev, nullptr, io->sum_win, io->max_win,
                                  io->sum_tok, io->max_tok, io->ws_score, io->ws_score_bytes,
                                  pl0 >= 0 ? io->ws_compact : nullptr, io->status_dev, stream));
    if (pl0 >= 0)
      ACTKV_TRY(actkv_compact_end(pool, tab, pl0, pl1, io->sel_idx_dev, io->sel_stride, io->keep_indptr_dev, io->budget_dev,
                                  io->max_keep, io->ws_compact, io->ws_compact_bytes, io->status_dev, stream));
    if (g == 0) {
      if (budget_ready != nullptr) ACTKV_TRY(wait(s, budget_ready));
      ACTKV_TRY(actkv_keep_indptr(tab->seq_len, io->budget_dev, R, io->keep_indptr_dev, stream));
    }
    ACTKV_TRY(actkv_select(io->score_dev, io->tok_indptr_dev, io->sum_tok, io->budget_dev, (l1 - l0) * Hkv, R,
                           io->keep_indptr_dev, io->sel_idx_dev, io->sel_stride, nullptr, nullptr, nullptr, 0,
                           io->status_dev, stream));
    if (g == n_groups - 1) {
      // nothing follows the last group that could carry its copies: the one-launch copy
      ACTKV_TRY(actkv_compact(pool, tab, l0, l1, io->sel_idx_dev, io->sel_stride, io->keep_indptr_dev, io->budget_dev,
                              io->max_keep, io->ws_compact, io->ws_compact_bytes, io->status_dev, stream));
      pl0 = pl1 = -1;
    } else {
      ACTKV_TRY(actkv_compact_begin(pool, tab, l0, l1, io->sel_idx_dev, io->sel_stride, io->keep_indptr_dev, io->budget_dev,
                                    io->max_keep, g > 0 ? 1 : 0, io->ws_compact, io->ws_compact_bytes, io->status_dev,
                                    stream));
      pl0 = l0;
      pl1 = l1;
    }
  }
  return ACTKV_OK;
}

static int step_enqueue(const actkv_pool_t* pool, const actkv_tables_t* tab, const actkv_budget_params_t* params,
                        const actkv_host_step_t* io, actkv_stream_t stream, StepStreams* st) {
  cudaStream_t s = (cudaStream_t)stream;
  const int R = tab->n_req, NL = pool->n_layers;
  const bool with_budget = io->logits_host != nullptr && io->n_rows > 0;
  int lpc = io->layers_per_call > 0 && io->layers_per_call < kDefaultGroupLayers ? io->layers_per_call
                                                                                 : kDefaultGroupLayers;
  if (lpc > NL) lpc = NL;
  if ((NL + lpc - 1) / lpc + 1 > kMaxGroups) return ACTKV_E_INVALID;
  // (The passes that follow the LSE work on resident queries: as many layers per call as the caller's score
  // and index buffers hold: step_groups.)
  // Groups of the query copies and LSE passes: a short first group, so that the first kernel starts
  // after a quarter of a group's transfer time, then groups of lpc layers.
  int lse_bound[kMaxGroups + 1];
  int n_lse_groups = 0;
  lse_bound[0] = 0;
  {
    const int first = lpc >= 4 && NL > lpc / 4 ? lpc / 4 : (lpc < NL ? lpc : NL);
    for (int l = first; ; l += lpc) {
      lse_bound[++n_lse_groups] = l < NL ? l : NL;
      if (l >= NL) break;
    }
  }
  const size_t q_layer_bytes = (size_t)io->sum_win * io->n_q_heads * pool->head_dim * 2;
  const size_t tbl_bytes = (size_t)R * tab->max_pages * 4;

  // ---- copy stream (after whatever the caller queued on `stream`): the small inputs first, then the
  // queries group by group, then the logits.  The caller's stream carries no copy of its own until the
  // results go back: measured on B200, kernels of a stream that had issued host-to-device copies itself
  // did not start until the copy engine had drained the other stream's large copies as well (no overlap
  // at all, 26.8 ms per step instead of 19.5 at the benchmark shape). ----
  cudaStream_t c = st->copy;
  ACTKV_TRY(record(st->start, s));
  ACTKV_TRY(wait(c, st->start));
  ACTKV_TRY(h2d(io->win_indptr_dev, io->win_indptr_host, (size_t)(R + 1) * 4, c));
  ACTKV_TRY(h2d(io->tok_indptr_dev, io->tok_indptr_host, (size_t)(R + 1) * 4, c));
  ACTKV_TRY(h2d(io->budget_dev, io->budget_in_host, (size_t)R * 4, c));
  ACTKV_TRY(h2d(tab->page_table, io->page_table_host, tbl_bytes, c));
  ACTKV_TRY(h2d(tab->seq_len, io->seq_len_host, (size_t)R * 4, c));
  ACTKV_TRY(h2d(tab->free_list, io->free_list_host, (size_t)pool->n_pages * 4, c));
  ACTKV_TRY(h2d(tab->free_count, io->free_count_host, 4, c));
  if (with_budget) ACTKV_TRY(h2d(io->logit_indptr_dev, io->logit_indptr_host, (size_t)(R + 1) * 4, c));
  if (cudaMemsetAsync(io->status_dev, 0, 16, c) != cudaSuccess) return ACTKV_E_CUDA;
  ACTKV_TRY(record(st->small, c));
  for (int g = 0; g < n_lse_groups; ++g) {
    const int l0 = lse_bound[g], l1 = lse_bound[g + 1];
    ACTKV_TRY(h2d((char*)io->q_dev + (size_t)l0 * q_layer_bytes, (const char*)io->q_host + (size_t)l0 * q_layer_bytes,
                  (size_t)(l1 - l0) * q_layer_bytes, st->copy));
    ACTKV_TRY(record(st->q[g], st->copy));
  }
  if (with_budget) {
    ACTKV_TRY(h2d(io->logits_dev, io->logits_host, (size_t)io->n_rows * io->vocab * 4, st->copy));
    ACTKV_TRY(record(st->logits, st->copy));
  }

  // ---- side stream: the budget monitor, as soon as the logits are in ----
  if (with_budget) {
    ACTKV_TRY(wait(st->side, st->logits));
    ACTKV_TRY(actkv_budget(io->logits_dev, io->logit_indptr_dev, io->n_rows, io->vocab, io->conf_hist_dev,
                           io->hist_len_dev, io->hist_cap, params, tab->seq_len, io->budget_dev, io->budget_dev,
                           nullptr, R, io->ws_budget, io->ws_budget_bytes, io->status_dev, (actkv_stream_t)st->side));
    ACTKV_TRY(record(st->budget, st->side));
  }

  // ---- caller's stream: LSE pass of every group while the rest of the input arrives ----
  for (int g = 0; g < n_lse_groups; ++g) {
    const int l0 = lse_bound[g], l1 = lse_bound[g + 1];
    ACTKV_TRY(wait(s, st->q[g]));
    ACTKV_TRY(actkv_score_lse(pool, tab, l0, l1, (const char*)io->q_dev + (size_t)l0 * q_layer_bytes, io->win_indptr_dev,
                              io->n_q_heads, io->sm_scale, io->causal, io->tok_indptr_dev,
                              io->lse_dev + (size_t)l0 * io->sum_win * io->n_q_heads, io->sum_win, io->max_win,
                              io->sum_tok, io->max_tok, io->ws_score, io->ws_score_bytes, io->status_dev, stream));
  }
  ACTKV_TRY(step_groups(pool, tab, io, stream, with_budget ? st->budget : nullptr));

  // ---- device -> host: the step's results ----
  ACTKV_TRY(d2h(io->page_table_out_host, tab->page_table, tbl_bytes, s));
  ACTKV_TRY(d2h(io->seq_len_out_host, tab->seq_len, (size_t)R * 4, s));
  ACTKV_TRY(d2h(io->free_list_out_host, tab->free_list, (size_t)pool->n_pages * 4, s));
  ACTKV_TRY(d2h(io->free_count_out_host, tab->free_count, 4, s));
  ACTKV_TRY(d2h(io->budget_out_host, io->budget_dev, (size_t)R * 4, s));
  ACTKV_TRY(d2h(io->status_out_host, io->status_dev, 16, s));
  return ACTKV_OK;
}

extern "C" int actkv_step_host(const actkv_pool_t* pool, const actkv_tables_t* tab,
                               const actkv_budget_params_t* params, const actkv_host_step_t* io,
                               actkv_stream_t stream) {
  if (!pool || !tab || !io) return ACTKV_E_INVALID;
  if (tab->n_req <= 0 || pool->n_layers <= 0 || io->sum_win <= 0 || io->sum_tok <= 0) return ACTKV_E_INVALID;
  if (io->logits_host != nullptr && io->n_rows > 0 && !params) return ACTKV_E_INVALID;
  StepStreams* st = step_streams();
  if (!st) return ACTKV_E_CUDA;
  const int rc = step_enqueue(pool, tab, params, io, stream, st);
  // whatever was queued is waited for, also when a later call failed: the library's streams are shared
  // by every call on this device and the caller's host buffers must be free again on return
  bool ok = cudaStreamSynchronize(st->copy) == cudaSuccess;
  ok = (cudaStreamSynchronize(st->side) == cudaSuccess) && ok;
  ok = (cudaStreamSynchronize((cudaStream_t)stream) == cudaSuccess) && ok;
  if (rc != ACTKV_OK) return rc;
  return ok ? ACTKV_OK : ACTKV_E_CUDA;
}

// The same step for inputs that are already in device memory: nothing is copied, no stream of the library's own is
// used and the call does not synchronise.
extern "C" int actkv_step_device(const actkv_pool_t* pool, const actkv_tables_t* tab,
                                 const actkv_budget_params_t* params, const actkv_host_step_t* io,
                                 int32_t lse_supplied, actkv_stream_t stream) {
  if (!pool || !tab || !io) return ACTKV_E_INVALID;
  if (tab->n_req <= 0 || pool->n_layers <= 0 || io->sum_win <= 0 || io->sum_tok <= 0) return ACTKV_E_INVALID;
  const bool with_budget = io->logits_dev != nullptr && io->n_rows > 0;
  if (with_budget && !params) return ACTKV_E_INVALID;
  if (!io->lse_dev || !io->q_dev || !io->budget_dev) return ACTKV_E_INVALID;
  const int R = tab->n_req, NL = pool->n_layers;
  if (with_budget)
    ACTKV_TRY(actkv_budget(io->logits_dev, io->logit_indptr_dev, io->n_rows, io->vocab, io->conf_hist_dev,
                           io->hist_len_dev, io->hist_cap, params, tab->seq_len, io->budget_dev, io->budget_dev, nullptr,
                           R, io->ws_budget, io->ws_budget_bytes, io->status_dev, stream));
  if (!lse_supplied) {
    // as many layers per LSE launch as the score workspace holds (fewer, larger launches waste less)
    int per = NL;
    for (int parts = 1; parts <= NL; ++parts) {
      per = (NL + parts - 1) / parts;
      if (actkv_score_workspace_bytes(pool, R, per, io->n_q_heads, io->sum_win, io->max_win, io->max_tok) <= io->ws_score_bytes)
        break;
    }
    const size_t q_layer_bytes = (size_t)io->sum_win * io->n_q_heads * pool->head_dim * 2;
    for (int l0 = 0; l0 < NL; l0 += per) {
      const int l1 = l0 + per < NL ? l0 + per : NL;
      ACTKV_TRY(actkv_score_lse(pool, tab, l0, l1, (const char*)io->q_dev + (size_t)l0 * q_layer_bytes, io->win_indptr_dev,
                                io->n_q_heads, io->sm_scale, io->causal, io->tok_indptr_dev,
                                io->lse_dev + (size_t)l0 * io->sum_win * io->n_q_heads, io->sum_win, io->max_win,
                                io->sum_tok, io->max_tok, io->ws_score, io->ws_score_bytes, io->status_dev, stream));
    }
  }
  return step_groups(pool, tab, io, stream, nullptr);
}
