/*
 * actkv.h — C ABI of the action-guided KV-cache compression hot path (ActKV) for one B200.
 *
 * The library runs the three page-aware primitives the paper distils every eviction method
 * into (Section 3.3: CalAttn -> Eviction -> Compaction) plus the confidence monitor that sets
 * the budget (Section 6, Algorithm 2), directly on a paged bf16 KV cache
 * PagedKVCache[2, B, BS, H, D] addressed through a block table (Section 2.5).
 *
 * Conventions that hold for every entry point
 *   - `extern "C"`, plain pointers and sizes.  Unless a parameter says "host", a pointer is a
 *     DEVICE pointer owned by the caller.  The two descriptor structs and the parameter struct
 *     are HOST structs (passed by pointer, read during the call) that hold device pointers.
 *   - Every call is asynchronous on `stream`, never synchronises, never allocates or frees
 *     device memory.  Scratch comes from the caller: `ws` of at least
 *     `actkv_*_workspace_bytes(...)` bytes, 256-byte aligned.  The one exception is
 *     actkv_step_host, whose outputs are host memory: it creates two streams and a few events
 *     per device on first use, and synchronises `stream` before it returns.
 *   - Return value: ACTKV_OK or a negative code for what the host can see (bad argument,
 *     workspace too small, launch failure).  What only the device can see (a page id out of
 *     range, a free list that is too short) is written to the caller's `status[4]` int32 words:
 *     status[0] = first error code (0 while clean), status[1..2] = where (request / unit,
 *     offending value).  Kernels never trap.  An out-of-range page id met by a score kernel is
 *     replaced by page 0 for the read and reported; a copy whose source or destination page id is
 *     out of range is dropped and reported (nothing is read from or written to a page the request
 *     does not own).  Once status[0] is set, actkv_select and the compaction calls of the same
 *     step do nothing.  When the plan step of actkv_compact reports ACTKV_E_NOFREE the copy and
 *     table-update steps of that call do nothing, so pool and tables stay unmodified.
 *   - All indices are int32.  Strides are in ELEMENTS (bf16), the head dimension is contiguous.
 *   - "unit" = one (layer, KV head, request); units are independent in score and select.
 *   - Arrays with a leading layer axis are RELATIVE to `layer_begin`: slab 0 belongs to layer
 *     `layer_begin`.  Only the pool is indexed by absolute layer.
 */
#ifndef ACTKV_H_
#define ACTKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ACTKV_OK            0
#define ACTKV_E_INVALID    -1   /* bad argument / unsupported shape (host-detected)              */
#define ACTKV_E_WORKSPACE  -2   /* `ws_bytes` smaller than the matching *_workspace_bytes()     */
#define ACTKV_E_CUDA       -3   /* a CUDA runtime call or launch failed                          */
#define ACTKV_E_BADPAGE    -4   /* device: page id outside [0, n_pages) met in a page table      */
#define ACTKV_E_NOFREE     -5   /* device: free list holds fewer pages than compaction needs     */
#define ACTKV_E_BADINDEX   -6   /* device: selected token index outside [0, seq_len)             */
#define ACTKV_E_TIMEOUT    -7   /* device: a bounded wait inside a kernel gave up                */
#define ACTKV_E_TOOBIG     -8   /* sizes beyond the fixed scratch of a *_noalloc entry point    */

/* CUDA stream handle (identical to cudaStream_t; spelled out so the header needs no CUDA). */
typedef struct CUstream_st* actkv_stream_t;

/*
 * The paged pool, Section 2.5: PagedKVCache[2, B, BS, H, D] per layer.
 * Element (layer l, kv in {0 = K, 1 = V}, page p, slot s, head h, dim d) lives at
 *   base + l*stride_layer + kv*stride_kv + p*stride_page + s*stride_slot + h*stride_head + d.
 * Any strides with contiguous head dimensions describe a pool (slot-major [page][slot][head][dim]
 * pages as well as head-major [page][head][slot][dim] ones).  The tensor-core score path needs
 * page_size 16, 32, 64 or 128, head_dim 64 or 128, strides that are multiples of 8 elements and a
 * 128-byte aligned base; other shapes take the (much slower) FMA path.
 */
typedef struct {
  void*   base;                 /* device, bf16 */
  int32_t n_layers, n_pages, page_size, n_kv_heads, head_dim;
  int64_t stride_layer, stride_kv, stride_page, stride_slot, stride_head;
} actkv_pool_t;

/*
 * Block table and allocator state, Section 2.5 (block_table, seqused_k) plus the free list the
 * freed blocks go back to (Section 7.2, last paragraph).  Logical token j of request r sits in
 * physical slot page_table[r][j / page_size] * page_size + j % page_size.
 * free_list is a LIFO stack of page ids, the top at free_list[*free_count - 1].
 */
typedef struct {
  int32_t  n_req, max_pages;
  int32_t* page_table;          /* [n_req, max_pages], unused entries -1 */
  int32_t* seq_len;             /* [n_req] */
  int32_t* free_list;           /* [n_pages] */
  int32_t* free_count;          /* [1] */
} actkv_tables_t;

/*
 * Parameters of the confidence monitor, Section 6.1 and Algorithm 2; defaults of Section 8.1
 * (Configuration): k=20, w=64, s=8, b=10, scale_up=1.75, B_upper=30000.
 * The clamp is an addition of this library (off when clamp_hi_ppm <= 0): after the update,
 * B' = min(max(B', ceil(L*clamp_lo_ppm/1e6)), floor(L*clamp_hi_ppm/1e6)), L = seq_len, in
 * exact integer arithmetic.
 */
typedef struct {
  int32_t k;                    /* top-k tokens per distribution                         */
  int32_t w, s;                 /* min-pooling window and stride                         */
  double  b_percent;            /* bottom-b% of the pooled sequence is kept               */
  double  scale_up;             /* B' = floor(B*scale_up) when the fitted slope is < 0    */
  int32_t B_upper;              /* cap on B'                                              */
  int32_t clamp_lo_ppm, clamp_hi_ppm;
} actkv_budget_params_t;

/* Per-unit report of actkv_select: the n-th largest score and how ties at it were resolved. */
typedef struct {
  float   threshold;            /* score of the last entry kept (0 if none kept)          */
  int32_t n_equal_kept;         /* entries equal to threshold that were kept              */
  int32_t n_equal_total;        /* entries equal to threshold in the unit                 */
  int32_t n_keep;               /* min(budget, seq_len)                                   */
} actkv_tie_t;

/* ---------------------------------------------------------------------------------------
 * actkv_budget — confidence monitor and budget update (Section 6.1 equations, Algorithm 2).
 *
 * For every new token i of request r (rows tok_indptr[r] .. tok_indptr[r+1] of `logits`):
 *   T_i = -(1/k) sum_{j<=k} log P_i(j)  over the k most probable tokens
 *       = logsumexp(z_i) - mean(top-k z_i),
 * appended (as float32) to the request's history conf_hist[r][hist_len[r] ...].  Then over the
 * whole history (length Lh): R'_m = min T[m*s .. m*s+w), m = 0..floor((Lh-w)/s); R = the values
 * of R' not above its b-th percentile (nearest rank: the max(1, ceil(b/100*M))-th smallest), in
 * time order; alpha = least-squares slope of R against 0..|R|-1 (0 when |R| < 2 or Lh < w);
 *   B' = alpha < 0 ? min(floor(B*scale_up), B_upper) : B,   then the optional clamp.
 * logits     float32 [n_rows, vocab] row-major, n_rows = tok_indptr[n_req] (passed as n_rows).
 * tok_indptr int32 [n_req+1].  conf_hist float32 [n_req, hist_cap]; hist_len int32 [n_req]
 *            (updated).  Tokens that do not fit in hist_cap are dropped and reported as
 *            ACTKV_E_INVALID in status.
 * seq_len    int32 [n_req] (only read when the clamp is on; may be NULL otherwise).
 * budget_in / budget_out int32 [n_req] (may alias).  slope_out double [n_req] or NULL.
 * logits == NULL with n_rows == 0 runs only the trend / update step on the stored history.
 * hist_cap <= 65536.
 */
size_t actkv_budget_workspace_bytes(int32_t n_rows, int32_t n_req, int32_t hist_cap);
int actkv_budget(const float* logits, const int32_t* tok_indptr, int32_t n_rows, int32_t vocab,
                 float* conf_hist, int32_t* hist_len, int32_t hist_cap,
                 const actkv_budget_params_t* params /* host */,
                 const int32_t* seq_len, const int32_t* budget_in, int32_t* budget_out,
                 double* slope_out, int32_t n_req, void* ws, size_t ws_bytes,
                 int32_t* status, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_score — action-region attention score of every cached entry
 * (Section 2.3 attention definition; Section 7.1 LSE identity; Algorithm 3 pooling).
 *
 * For layer l, request r, KV head h, key j < L_r, window row w < W_r and q-head
 * qh = h*G + g (G = n_q_heads / n_kv_heads, contiguous GQA groups):
 *   s      = sm_scale * <q[l, win_indptr[r]+w, qh, :], K[l, slot(r, j), h, :]>
 *   lse    = log sum_{j visible} exp(s)              (or lse_in when supplied)
 *   a      = exp(s - lse)                            (Section 7.1: A = exp(s - LSE))
 *   score[l, h, tok_indptr[r]+j] = (1/W_r) * sum_w max_g a      (Algorithm 3 steps 4-5)
 * causal == 0: every row sees every key.  causal != 0: the window is the last W_r cached
 * tokens, row w sees keys j <= L_r - W_r + w; a masked (w, j) pair contributes 0 and the
 * divisor stays W_r.
 * q          bf16 [NLs, sum_win, n_q_heads, head_dim], NLs = layer_end - layer_begin.
 * win_indptr int32 [n_req+1]; tok_indptr int32 [n_req+1] (exclusive prefix sums of W_r, L_r).
 * lse_in     float32 [NLs, sum_win, n_q_heads] natural-log units of the scaled logits, or NULL
 *            to compute it here (one extra pass over K).  lse_out: same shape or NULL.
 * score_out  float32 [NLs, n_kv_heads, sum_tok].
 * sum_win, max_win, sum_tok, max_tok: host copies of win_indptr[n_req], max W_r,
 *            tok_indptr[n_req], max L_r (upper bounds are accepted for the two maxima).
 * W_r == 0 for a request with L_r > 0 is reported as ACTKV_E_INVALID in status.
 * Workspace: the size for n_layers_sub layers also serves every call on fewer layers with the
 * same other arguments.
 */
size_t actkv_score_workspace_bytes(const actkv_pool_t* pool /* host */, int32_t n_req,
                                   int32_t n_layers_sub, int32_t n_q_heads, int32_t sum_win,
                                   int32_t max_win, int32_t max_tok);
int actkv_score(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                int32_t layer_begin, int32_t layer_end,
                const void* q, const int32_t* win_indptr, int32_t n_q_heads,
                const float* lse_in, float sm_scale, int32_t causal,
                const int32_t* tok_indptr, float* score_out, float* lse_out,
                int32_t sum_win, int32_t max_win, int32_t sum_tok, int32_t max_tok,
                void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_score_sliding — actkv_score for sliding-window attention layers (Section 8.2 names models
 * that interleave such layers with full-attention ones; the paper does not say how they are scored,
 * this is the reading taken here).
 *
 * window_left = S > 0: a query at cache position p attends to the S keys p - S < j <= p only.  With
 * causal != 0 row w sits at p = L_r - W_r + w; with causal == 0 every row is taken to sit at the end
 * of the cache, p = L_r - 1.  The LSE (computed here or supplied) runs over the same visible set.
 * Keys no row sees score 0; whole key tiles of them are neither fetched nor multiplied.
 * S = 0 is actkv_score.  One S per call: a model that alternates layer kinds hands each kind over as
 * a pool view whose stride_layer skips the other.  All other arguments as actkv_score.
 */
int actkv_score_sliding(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                        int32_t layer_begin, int32_t layer_end,
                        const void* q, const int32_t* win_indptr, int32_t n_q_heads,
                        const float* lse_in, float sm_scale, int32_t causal, int32_t window_left,
                        const int32_t* tok_indptr, float* score_out, float* lse_out,
                        int32_t sum_win, int32_t max_win, int32_t sum_tok, int32_t max_tok,
                        void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_score_path — which kernels actkv_score (streaming == 0) or actkv_score_accumulate
 * (streaming != 0) would run for this pool, group size, window bound, scale and query pointer:
 * 1 = the tensor-core kernels (tcgen05), 0 = the FMA kernels, negative = bad argument.
 * Launches nothing.  (Section 7.1 / Algorithm 3 are the same arithmetic on both paths.)
 */
int actkv_score_path(const actkv_pool_t* pool /* host */, int32_t n_q_heads, int32_t max_win,
                     float sm_scale, const void* q, int32_t streaming);

/* ---------------------------------------------------------------------------------------
 * actkv_score_lse — only the log-sum-exp of actkv_score (Section 7.1, LSE equation): what a
 * paged attention backend would hand over as a by-product.  Same arguments and workspace as
 * actkv_score; writes lse_out float32 [NLs, sum_win, n_q_heads] (required) and no score.
 * actkv_score_lse followed by actkv_score(lse_in = that) equals actkv_score(lse_in = NULL).
 */
int actkv_score_lse(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                    int32_t layer_begin, int32_t layer_end,
                    const void* q, const int32_t* win_indptr, int32_t n_q_heads,
                    float sm_scale, int32_t causal, const int32_t* tok_indptr, float* lse_out,
                    int32_t sum_win, int32_t max_win, int32_t sum_tok, int32_t max_tok,
                    void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_score_accumulate — the streaming form of actkv_score: Algorithm 3 as it is triggered
 * at every decode step of an action region, with the LSE handed over by the attention backend
 * (Section 7.1) and the running mean over the action queries kept in score_io (Algorithm 3
 * step 5; the state restarts from zero at region entry).
 *
 * Per call every request contributes its W_r newest action queries (W_r = 1 per decode step;
 * W_r = 0: the request is outside an action region and is skipped).  With n_r = acc_steps[r]
 * action queries already folded in, and S_j = sum_w max_g exp(s - lse_in) as in actkv_score:
 *   score_io[l, h, tok_indptr[r]+j] <- (n_r * score_io[..] + S_j) / (n_r + W_r),   j < L_r.
 * n_r == 0 (region entry): the old content is not read, the value is S_j / W_r.  For n_r > 0
 * the entries of keys cached since the previous call must hold 0 (zero the request's segment at
 * region entry).  The caller adds W_r to acc_steps[r] after the call (same stream).
 * tok_indptr gives the OFFSET of each request's segment in score_io; segments may be longer than
 * L_r (capacity), L_r is read from tables->seq_len.  causal as in actkv_score (within the call's
 * W_r queries; irrelevant for W_r = 1).  lse_in and acc_steps (int32 [n_req], device) are
 * required.  Other arguments, workspace and errors as actkv_score.
 * After the last query of a region score_io equals actkv_score's result for the whole window
 * (causal != 0) up to float32 rounding of the running mean.
 */
int actkv_score_accumulate(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                           int32_t layer_begin, int32_t layer_end,
                           const void* q, const int32_t* win_indptr, int32_t n_q_heads,
                           const float* lse_in, float sm_scale, int32_t causal,
                           const int32_t* tok_indptr, const int32_t* acc_steps, float* score_io,
                           int32_t sum_win, int32_t max_win, int32_t sum_tok, int32_t max_tok,
                           void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_keep_indptr — helper: keep_indptr[r] = sum_{r'<r} min(budget[r'], seq_len[r']),
 * keep_indptr[n_req] = total (Algorithm 1 step 5 keeps min(B, L) entries).  One tiny kernel.
 */
int actkv_keep_indptr(const int32_t* seq_len, const int32_t* budget, int32_t n_req,
                      int32_t* keep_indptr, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_keepscore — attention-aware LRFU keep-score (Section 5.1 equation; Algorithm 1 steps 2-4),
 * an optional stage between actkv_score and actkv_select.
 *
 * Per unit (o, r) over score[o, tok_indptr[r] .. tok_indptr[r+1]):
 *   hit_i  = 1 iff entry i falls within the top-p set of the unit: the shortest prefix of the
 *            entries ordered by (score descending, index ascending) whose mass reaches p of the
 *            unit's total mass, the crossing entry included.  Mass is counted exactly:
 *            m_i = floor(clip(score_i, 0, 256) * 2^32), mark = ceil(round(p*10000) * sum m / 10000).
 *   KS_i   = lambda * KS_i + score_i * hit_i        (float32, one rounding per operation)
 *   score_i is then OVERWRITTEN with the key actkv_select should rank: KS_i, or +inf for the
 *            first n_protect[r] entries (system prompt / task description, Section 8.1), which are
 *            therefore always retained while the budget allows.
 * keep_score float32 [n_outer, sum_tok], same layout as score, in/out.  Entries appended since the
 *            last compression must hold 0 (Algorithm 1 step 2).
 * n_protect  int32 [n_req] or NULL.  hit_mask optional bitmap [n_outer, ceil(sum_tok/32)], zeroed
 *            by the caller.  Scores are expected in [0, 1] (pooled probabilities).
 */
int actkv_keepscore(float* score, const int32_t* tok_indptr, int32_t sum_tok, int32_t n_outer,
                    int32_t n_req, float top_p, float lambda, const int32_t* n_protect,
                    float* keep_score, uint32_t* hit_mask, int32_t* status, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_keepscore_select — actkv_keepscore and actkv_select in one launch (Algorithm 1 steps 2-5):
 * the ranking keys (updated keep-scores, +inf on the protected prefix) go straight into TopK
 * without passing through memory, so the scores are read once.  Same results as the two calls
 * (keep_score, hit_mask, sel_idx, keep_mask, tie_report), except that `score` is left as it was
 * when every unit fits in shared memory (max_tok <= 45568 tokens); longer units run the two
 * stages as two kernels and `score` then holds the ranking keys as after actkv_keepscore.
 * max_tok: host upper bound on the unit lengths.  Other arguments as the two calls.
 */
int actkv_keepscore_select(float* score, const int32_t* tok_indptr, int32_t sum_tok, int32_t max_tok,
                           int32_t n_outer, int32_t n_req, float top_p, float lambda,
                           const int32_t* n_protect, float* keep_score, uint32_t* hit_mask,
                           const int32_t* budget, const int32_t* keep_indptr, int32_t* sel_idx,
                           int64_t sel_stride, uint32_t* keep_mask, actkv_tie_t* tie_report,
                           int32_t* status, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_gather_f32 — the survivors' keep-scores move with them (Algorithm 1 step 5 returns KS'):
 *   dst[o, keep_indptr[r] + i] = src[o, tok_indptr[r] + sel_idx[o, keep_indptr[r] + i]].
 * src float32 [n_outer, src_stride]; dst float32 [n_outer, dst_stride]; max_total_keep: host upper
 * bound on keep_indptr[n_req].
 */
int actkv_gather_f32(const float* src, int64_t src_stride, const int32_t* tok_indptr,
                     const int32_t* sel_idx, int64_t sel_stride, const int32_t* keep_indptr,
                     int32_t n_outer, int32_t n_req, int32_t max_total_keep,
                     float* dst, int64_t dst_stride, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_select — TopK(score, k = B) per unit (Algorithm 1 step 5, applied to the pooled
 * score, independently per layer and KV head).
 *
 * For unit (o, r), o < n_outer (= layers * KV heads), over score[o, tok_indptr[r] ..
 * tok_indptr[r+1]): keep the n_r = min(budget[r], L_r) largest float32 scores; among equal
 * scores the lower token index wins; emit the kept token indices (0-based within the
 * request) in ascending order to sel_idx[o*sel_stride + keep_indptr[r] ...].
 * score      float32 [n_outer, sum_tok] (values must be >= 0, as pooled probabilities are;
 *            -0.0 and NaN are treated by their bit pattern order).
 * keep_mask  optional uint32 bitmap [n_outer, ceil(sum_tok/32)]: bit (tok_indptr[r]+j) set
 *            iff kept; must be zero-filled by the caller.  NULL to skip.
 * tie_report optional [n_outer, n_req].
 */
size_t actkv_select_workspace_bytes(int32_t n_outer, int32_t n_req, int32_t max_tok);
int actkv_select(const float* score, const int32_t* tok_indptr, int32_t sum_tok,
                 const int32_t* budget, int32_t n_outer, int32_t n_req,
                 const int32_t* keep_indptr, int32_t* sel_idx, int64_t sel_stride,
                 uint32_t* keep_mask, actkv_tie_t* tie_report,
                 void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_compact — pack the survivors into fresh pages and free the old ones
 * (Section 7.2 / Algorithm 4: survivors packed contiguously, pure copy, freed blocks returned;
 *  here into pages popped from the free list instead of the tail of the old ones).
 *
 * Requests with budget[r] >= seq_len[r] are left untouched.  For the others, in ascending r,
 * n_r = budget[r], X_r = ceil(n_r / page_size), off_r = sum of X over earlier compacting
 * requests:  new_page[r][i] = free_list[free_count - 1 - (off_r + i)],  i < X_r.
 * For every layer in [layer_begin, layer_end), head h, i < n_r: the K row and the V row of
 * token sel_idx[(l-layer_begin)*H + h][keep_indptr[r] + i] move to logical slot i of the new
 * pages.  When layer_end == pool->n_layers the tables are updated after the copies:
 * page_table[r] = new pages then -1, seq_len[r] = n_r, free_count -= sum X, then for r
 * ascending and i ascending free_list[free_count++] = old page i of r.
 * Calls on layer sub-ranges recompute the same plan from the still-unchanged tables.
 * max_keep: host upper bound on n_r (<= max_pages*page_size).
 */
size_t actkv_compact_workspace_bytes(int32_t n_req, int32_t max_pages);
int actkv_compact(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                  int32_t layer_begin, int32_t layer_end,
                  const int32_t* sel_idx, int64_t sel_stride, const int32_t* keep_indptr,
                  const int32_t* budget, int32_t max_keep,
                  void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_compact_begin / actkv_score_overlap / actkv_compact_end — the compaction of one layer
 * group hidden under the score kernels of the next one.
 * (Section 3.3: the three primitives are independent per layer; Section 7.2 / Algorithm 4: the
 *  copies of a planned compaction are order-free, their sources and destinations disjoint.)
 *
 * The pooled-score kernel is bound by the tensor pipe and leaves most of the HBM bandwidth idle; the
 * copy of a compaction is bound by HBM and needs no tensor pipe.  A step over many layers can
 * therefore run, for layer groups g = 0, 1, ...:
 *     actkv_score_overlap(group g, pending = ws)   score of g; spare warps of its pooled-score kernel copy rows of g-1
 *     actkv_compact_end(group g-1, ws)             copies whatever is left of g-1 (+ tables after the last layer)
 *     actkv_select(group g)
 *     actkv_compact_begin(group g, ws)             plan of g, published as a work queue in ws; copies nothing
 * and after the last group actkv_compact_end for it.  All calls on one stream; one workspace and
 * one index buffer suffice, because actkv_compact_end(g-1) precedes actkv_select(g).
 *
 * actkv_compact_begin: arguments as actkv_compact.  Runs the plan (fresh pages for
 *   [layer_begin, layer_end), errors as actkv_compact), resolves the source of every row once into a
 *   table and records the job in `ws`, which must stay untouched, like sel_idx / keep_indptr /
 *   budget / the tables, until the matching actkv_compact_end has run.  `ws` must have
 *   actkv_compact_deferred_workspace_bytes(pool, n_req, max_pages, layer_end - layer_begin, max_keep)
 *   bytes for the copies to be deferred; with only actkv_compact_workspace_bytes nothing is deferred
 *   and actkv_compact_end copies everything.  reuse_plan != 0: `ws` still holds the plan of an earlier
 *   actkv_compact_begin of the same step (same tables, budgets and max_keep, nothing finalized in
 *   between; the plan does not depend on the layers), so only the job of this layer range is recorded.
 *   A workspace that holds no plan of this pool and these tables is reported (status ACTKV_E_INVALID) and
 *   nothing is copied or finalized from it.
 * actkv_score_overlap: actkv_score with one more argument, pending_compact_ws: the workspace of a
 *   begun compaction of OTHER layers of the same pool, or NULL (then it is actkv_score).  The
 *   result of the score does not depend on it.  On the tensor-core path four spare warps per CTA of the
 *   pooled-score kernel take items (32 (slot, head) pairs of one destination page of one request and
 *   layer) of the pending job from a queue for as long as their CTA is scoring; the LSE kernel (whose
 *   epilogue needs every register of the SM) and the FMA path take none.
 * actkv_compact_end: the same arguments as the actkv_compact_begin it closes.  Copies every item
 *   not yet taken, then, when layer_end == pool->n_layers, updates the tables as actkv_compact does.
 * begin + end without a score call in between equals actkv_compact.  Pools the item copy does not
 * take (head_dim other than 64 / 128 / 256, more than 128 (slot, head) pairs per page) are copied
 * entirely by actkv_compact_end.
 */
size_t actkv_compact_deferred_workspace_bytes(const actkv_pool_t* pool /* host */, int32_t n_req, int32_t max_pages,
                                              int32_t n_layers_sub, int32_t max_keep);
int actkv_compact_begin(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                        int32_t layer_begin, int32_t layer_end,
                        const int32_t* sel_idx, int64_t sel_stride, const int32_t* keep_indptr,
                        const int32_t* budget, int32_t max_keep, int32_t reuse_plan,
                        void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream);
int actkv_compact_end(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                      int32_t layer_begin, int32_t layer_end,
                      const int32_t* sel_idx, int64_t sel_stride, const int32_t* keep_indptr,
                      const int32_t* budget, int32_t max_keep,
                      void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream);
/* stats (device, int32[2]) <- { items of the job begun in ws, items that score kernels executed };
 * an item is 32 (slot, head) pairs of one destination page.  Valid from actkv_compact_begin until
 * the next one on the same ws. */
int actkv_compact_stats(const void* ws, int32_t* stats, actkv_stream_t stream);
int actkv_score_overlap(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                        int32_t layer_begin, int32_t layer_end,
                        const void* q, const int32_t* win_indptr, int32_t n_q_heads,
                        const float* lse_in, float sm_scale, int32_t causal,
                        const int32_t* tok_indptr, float* score_out, float* lse_out,
                        int32_t sum_win, int32_t max_win, int32_t sum_tok, int32_t max_tok,
                        void* ws, size_t ws_bytes, void* pending_compact_ws,
                        int32_t* status, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_compact_inplace — compaction into the last X logical blocks of each request, without
 * fresh pages (Section 7.2 region equations; Algorithm 4 steps 1-6), one keep mask per
 * (layer, KV head), given as the ascending index lists actkv_select writes.
 *
 * Requests with budget[r] >= seq_len[r] are left untouched.  For the others, with L = seq_len[r],
 * B = budget[r], Y = ceil(L / page_size), X = ceil(B / page_size):
 *     Start = (Y - X) * page_size,  End = Start + B        (logical slots; End may pass L inside
 *                                                           the last block: unused slots are holes)
 * For every layer in [layer_begin, layer_end) and head: the holes of [Start, End) (slots not in
 * the list) in ascending order receive, pairwise, the K and V rows of the listed slots outside
 * [Start, End) in ascending order.  Sources and destinations are disjoint, nothing else is
 * written.  When layer_end == pool->n_layers the tables are updated after the copies, r ascending:
 * free_list[free_count++] = page i of r for i < Y - X ascending, page_table[r] = its last X pages
 * then -1, seq_len[r] = B.  No page is popped, so the call cannot run short of free pages.
 * Survivors do not keep ascending order: new_order (optional, int32, same layout as sel_idx)
 * receives at [.., keep_indptr[r] + i] the original token index of what now sits at logical slot
 * i (for untouched requests: the list itself), e.g. for actkv_gather_f32.
 * On a device-detected error the tables stay as they were; only holes were overwritten.
 * max_keep: host upper bound on min(budget[r], seq_len[r]).  No workspace.
 */
int actkv_compact_inplace(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                          int32_t layer_begin, int32_t layer_end,
                          const int32_t* sel_idx, int64_t sel_stride, const int32_t* keep_indptr,
                          const int32_t* budget, int32_t max_keep, int32_t* new_order,
                          int32_t* status, actkv_stream_t stream);

/* actkv_compact_inplace_begin / actkv_compact_inplace_end — the same in-place compaction with the
 * copies of one layer group hidden under the pooled-score kernel of the next one, as
 * actkv_compact_begin / actkv_compact_end do for the fresh-page form (Section 3.3: the primitives
 * are independent per layer; Algorithm 4: the moves of a plan are conflict-free, sources outside
 * the region, destinations inside it, so their order is free).
 *   begin: resolves every move of [layer_begin, layer_end) once into a table of (source,
 *          destination) rows, 32 region slots per item, and publishes it in `ws` as the work queue
 *          that actkv_score_overlap(pending_compact_ws = ws) serves; writes new_order (optional) as
 *          actkv_compact_inplace does; copies nothing, leaves the tables alone.  sel_idx may be
 *          reused once begin has run on the stream.
 *   end:   the same arguments; copies every item not yet taken and, when layer_end ==
 *          pool->n_layers, updates the tables as actkv_compact_inplace does.
 * begin + end without a score call in between equals actkv_compact_inplace.  `ws` must have
 * actkv_compact_inplace_deferred_workspace_bytes(pool, n_req, layer_end - layer_begin, max_keep)
 * bytes for the copies to be deferred (8 bytes per kept row and layer); with less (at least the
 * bytes of that call with max_keep = 0), or for a pool the item copy does not take (head_dim other
 * than 64 / 128 / 256), nothing is deferred and end runs the one-launch copy itself, for which
 * sel_idx must then still hold the lists. */
size_t actkv_compact_inplace_deferred_workspace_bytes(const actkv_pool_t* pool /* host */, int32_t n_req,
                                                      int32_t n_layers_sub, int32_t max_keep);
int actkv_compact_inplace_begin(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                                int32_t layer_begin, int32_t layer_end,
                                const int32_t* sel_idx, int64_t sel_stride, const int32_t* keep_indptr,
                                const int32_t* budget, int32_t max_keep, int32_t* new_order,
                                void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream);
int actkv_compact_inplace_end(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                              int32_t layer_begin, int32_t layer_end,
                              const int32_t* sel_idx, int64_t sel_stride, const int32_t* keep_indptr,
                              const int32_t* budget, int32_t max_keep, int32_t* new_order,
                              void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_step_host — one whole compression step (Algorithm 1 steps 1, 5, 6 with Algorithm 2 in
 * front) for a caller whose per-step inputs live in HOST memory.
 *
 * Copies this step's queries, action-token logits, index arrays, budgets and tables from the host
 * (pinned memory recommended) into the caller's device staging buffers, runs actkv_score_lse per
 * group of layers, actkv_budget (when logits are given) -> actkv_keep_indptr, then per group:
 * actkv_score_overlap, actkv_select, actkv_compact_begin / _end (the copies of a group run inside the
 * score kernels of the next one when ws_compact has actkv_compact_deferred_workspace_bytes for
 * layers_per_call layers), copies the new page table, seq_len, free list, free
 * count, budgets and the status words back to the host, and SYNCHRONISES the stream before
 * returning (the one entry point that does: its outputs are host memory).  The KV pool stays in
 * device memory — it is the cache being compressed.
 * The queries and logits are copied on a stream of the library's own (created on first use, one per
 * device), ordered after the work already queued on `stream`, so that the transfers overlap the LSE
 * kernels; everything is joined into `stream` before the results are copied back.  Those streams
 * are shared by all calls on a device: host threads must not run this entry point concurrently on
 * the same device.
 * layers_per_call: capacity of score_dev / sel_idx_dev / the score workspace in layers (0: all
 * layers).  The LSE passes run in groups of at most min(layers_per_call, 16) layers (the first one
 * shorter) while the queries arrive; the passes after them in groups of layers_per_call layers.
 * Every pointer named *_host is host memory, every other pointer device memory owned by the caller
 * and sized as the corresponding argument of the per-stage calls (score_dev:
 * [layers_per_call, n_kv_heads, sum_tok]; sel_idx_dev: [layers_per_call*n_kv_heads, sel_stride];
 * lse_dev: [n_layers, sum_win, n_q_heads]; q_dev: [n_layers, sum_win, n_q_heads, head_dim]).
 * `tables` holds the DEVICE copies of the tables; they are overwritten from the *_host inputs.
 * Output host pointers may be NULL to skip that copy.  budget_dev holds budget_in on entry of the
 * path and the budget that was applied on exit.
 */
typedef struct {
  const void*    q_host;
  const float*   logits_host;          /* [n_rows, vocab] or NULL: no budget update */
  const int32_t* win_indptr_host;      /* [n_req+1] */
  const int32_t* tok_indptr_host;      /* [n_req+1] */
  const int32_t* logit_indptr_host;    /* [n_req+1] (with logits) */
  const int32_t* budget_in_host;       /* [n_req] */
  const int32_t* page_table_host;      /* [n_req, max_pages] */
  const int32_t* seq_len_host;         /* [n_req] */
  const int32_t* free_list_host;       /* [n_pages] */
  const int32_t* free_count_host;      /* [1] */
  int32_t* page_table_out_host; int32_t* seq_len_out_host; int32_t* free_list_out_host;
  int32_t* free_count_out_host; int32_t* budget_out_host; int32_t* status_out_host /* [4] */;
  int32_t n_q_heads, sum_win, max_win, sum_tok, max_tok, n_rows, vocab, hist_cap, max_keep;
  int32_t causal, layers_per_call;
  float   sm_scale;
  int64_t sel_stride;
  void* q_dev; float* logits_dev;
  int32_t* win_indptr_dev; int32_t* tok_indptr_dev; int32_t* logit_indptr_dev;
  int32_t* budget_dev; int32_t* keep_indptr_dev;
  float* conf_hist_dev; int32_t* hist_len_dev; float* lse_dev; float* score_dev; int32_t* sel_idx_dev;
  void* ws_budget; size_t ws_budget_bytes; void* ws_score; size_t ws_score_bytes;
  void* ws_compact; size_t ws_compact_bytes;
  int32_t* status_dev;                 /* [4] */
} actkv_host_step_t;
int actkv_step_host(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                    const actkv_budget_params_t* params /* host, may be NULL without logits */,
                    const actkv_host_step_t* io /* host */, actkv_stream_t stream);

/* actkv_step_device — the same whole step in one call for inputs that are ALREADY in device memory:
 * the *_host members of `io` are ignored, q_dev / win_indptr_dev / tok_indptr_dev / budget_dev (and
 * logits_dev / logit_indptr_dev for a budget update: logits_dev == NULL or n_rows == 0 skips it) and
 * `tables` hold this step's inputs.  Runs actkv_budget, then (lse_supplied == 0) actkv_score_lse over
 * all layers in as few launches as ws_score allows, writing lse_dev, or (lse_supplied != 0) takes
 * lse_dev as the attention backend's LSE; then the layer groups as actkv_step_host does.  Everything
 * is queued on `stream`; like the per-stage calls it neither synchronises nor copies, and status_dev
 * is the caller's to clear and read. */
int actkv_step_device(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                      const actkv_budget_params_t* params /* host, may be NULL without logits */,
                      const actkv_host_step_t* io /* host */, int32_t lse_supplied, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_compact_noalloc — actkv_compact without a caller-supplied workspace.
 * (The paper has no counterpart; this is a convenience of the library.)
 *
 * Who it is for: a serving engine normally claims almost all of HBM for its KV block pool when
 * it starts, so a later cudaMalloc for a few hundred KB of plan scratch can fail outright, and
 * even when it succeeds cudaMalloc stalls the whole device, which a decode loop cannot afford
 * between two steps.  Plug-in style callers (a C host without torch's caching allocator) are in
 * the same position: they have device pointers to the pool and the tables and nothing to
 * allocate with.  For them the plan scratch lives in a fixed array inside the library's device
 * image (ACTKV_COMPACT_NOALLOC_BYTES on every GPU that loads the library, held until exit).
 *
 * Same arguments, semantics, status reporting and result as actkv_compact, minus ws/ws_bytes.
 * Limits and rules:
 *   - actkv_compact_workspace_bytes(n_req, max_pages) must not exceed
 *     ACTKV_COMPACT_NOALLOC_BYTES (about n_req*(max_pages+2) <= 262 000 table entries, e.g.
 *     64 requests x 4000 pages); larger tables return ACTKV_E_TOOBIG and launch nothing.
 *   - The first call on each device looks up the array's device address (once, with that device
 *     current) before launching; make that first call outside any stream capture.
 *   - It calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - All calls on a device share the one array.  The plan kernel of a call rewrites every word
 *     the later kernels of that call read, so stale contents are harmless, but two calls whose
 *     kernels overlap on the GPU (different streams without an ordering between them) race on
 *     it: serialise them, or give the second one actkv_compact with its own workspace.
 */
#define ACTKV_COMPACT_NOALLOC_BYTES (1u << 20)
size_t actkv_compact_noalloc_max_bytes(void);
int actkv_compact_noalloc(const actkv_pool_t* pool /* host */, const actkv_tables_t* tables /* host */,
                          int32_t layer_begin, int32_t layer_end,
                          const int32_t* sel_idx, int64_t sel_stride, const int32_t* keep_indptr,
                          const int32_t* budget, int32_t max_keep,
                          int32_t* status, actkv_stream_t stream);

/* ---------------------------------------------------------------------------------------
 * actkv_debug_inject_stall — fault-injection hook for the bounded waits of the tensor-core score
 * kernels (the paper has no counterpart).  Every wait inside those kernels (on a shared-memory
 * barrier) has a limit, after which the kernel writes ACTKV_E_TIMEOUT to status, all its roles
 * leave, outstanding tensor-core work is drained, tensor memory is freed and the kernel returns;
 * later stages of the step see the status and do nothing.  This hook makes that happen without a
 * real fault: while after_tile >= 0, the K-tile producers of every such launch of this process
 * issue no key tile with index >= after_tile of their CTA (nothing is left in flight: the loads are
 * simply not issued), and every wait gives up after about wait_limit_us microseconds instead of the
 * default two seconds.  after_tile < 0 restores normal operation.  Host-side, process-wide, takes
 * effect at the next launch; not for production use.
 */
int actkv_debug_inject_stall(int32_t after_tile, int32_t wait_limit_us);

/* Library version string (host pointer to static storage). */
const char* actkv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ACTKV_H_ */
