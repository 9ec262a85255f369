// actkv_budget: confidence monitor and budget update (Section 6.1, Algorithm 2).
//
// token_conf_kernel — one CTA per logits row.  T = logsumexp(z) - mean(top-k z).  The row is
//   streamed once from HBM (max + 11-bit digit histogram of the order-preserving integer image
//   of the floats) and twice more from L2 (sum of exp with the next 11-bit digit, then the last
//   10-bit digit with the sum of everything above the 22-bit prefix): a 3-pass radix select that
//   finds the k-th largest logit exactly, so the top-k sum is exact whatever the distribution
//   (all-equal rows included) and needs no sort.
// trend_kernel — one CTA per request: append, window-min pooling, nearest-rank bottom-b%,
//   least-squares slope in float64, budget update with the optional integer clamp.
#include "common.cuh"

namespace actkv {

constexpr int TC_NT = 1024;

__device__ __forceinline__ uint32_t okey(float x) {
  uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float okey_inv(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

__device__ __forceinline__ float block_reduce_max(float v, float* sm) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if (lane == 0) sm[warp] = v;
  __syncthreads();
  float r = sm[0];
  for (int w = 1; w < (int)(blockDim.x >> 5); ++w) r = fmaxf(r, sm[w]);
  return r;
}

// Fixed-order tree: deterministic for a given block size.
__device__ __forceinline__ double block_reduce_sum(double v, double* sm) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) sm[warp] = v;
  __syncthreads();
  double r = 0.0;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) r += sm[w];
  return r;
}

// Finds the digit d with  #(digit > d) < remaining <= #(digit >= d)  in hist[0..nbins).
// All threads call it; results land in shared s_out[0] = d, s_out[1] = remaining - #(digit > d),
// s_out[2] = hist[d].
__device__ __forceinline__ void pick_digit(const uint32_t* hist, int nbins, uint32_t remaining,
                                           uint32_t* warp_tot, uint32_t* s_out) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // nbins <= 2048 = 2 * TC_NT: each thread owns two adjacent reversed bins
  const int b0 = nbins - 1 - 2 * tid, b1 = b0 - 1;
  const uint32_t v0 = (b0 >= 0) ? hist[b0] : 0u, v1 = (b1 >= 0) ? hist[b1] : 0u;
  uint32_t incl = v0 + v1;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    uint32_t t = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += t;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  uint32_t add = 0;
  for (int w = 0; w < warp; ++w) add += warp_tot[w];
  incl += add;                                   // #(digit >= b1)
  const uint32_t ge0 = incl - v1;                // #(digit >= b0)
  const uint32_t gt0 = ge0 - v0;                 // #(digit >  b0)
  if (b0 >= 0 && ge0 >= remaining && gt0 < remaining) { s_out[0] = (uint32_t)b0; s_out[1] = remaining - gt0; s_out[2] = v0; }
  if (b1 >= 0 && incl >= remaining && ge0 < remaining) { s_out[0] = (uint32_t)b1; s_out[1] = remaining - ge0; s_out[2] = v1; }
  __syncthreads();
}

__global__ void __launch_bounds__(TC_NT) token_conf_kernel(
    const float* __restrict__ logits, const int32_t* __restrict__ tok_indptr, int32_t vocab,
    int32_t n_req, int32_t k_top, float* __restrict__ conf_hist, const int32_t* __restrict__ hist_len,
    int32_t hist_cap, const int32_t* __restrict__ redo, int32_t* status) {
  // three-sweep form: runs only for the rows the single-sweep kernel gave up on
  if (redo != nullptr && redo[blockIdx.x] == 0) return;
  __shared__ uint32_t hist[2048];
  __shared__ uint32_t warp_tot[TC_NT / 32];
  __shared__ uint32_t s_pick[3];
  __shared__ float red_f[TC_NT / 32];
  __shared__ double red_d[TC_NT / 32];
  const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
  const float* z = logits + (int64_t)row * vocab;
  const int k = min(k_top, vocab);

  // ---- pass 1 (HBM): max, histogram of key bits 31..21 ------------------------------------
  for (int i = tid; i < 2048; i += TC_NT) hist[i] = 0;
  __syncthreads();
  float mx = -INFINITY;
  for (int i0 = 0; i0 < vocab; i0 += TC_NT) {
    const int i = i0 + tid;
    const bool in = i < vocab;
    const float x = in ? z[i] : 0.f;
    const uint32_t voters = __ballot_sync(0xffffffffu, in);
    if (in) {
      mx = fmaxf(mx, x);
      const uint32_t bin = okey(x) >> 21;
      const uint32_t peers = __match_any_sync(voters, bin);
      if (lane == (__ffs(peers) - 1)) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
    }
  }
  mx = block_reduce_max(mx, red_f);             // includes the barrier that completes hist
  pick_digit(hist, 2048, (uint32_t)k, warp_tot, s_pick);
  const uint32_t d1 = s_pick[0];
  uint32_t remaining = s_pick[1];
  __syncthreads();

  // ---- pass 2 (L2): sum exp(z - max), histogram of bits 20..10 among keys with digit d1 -----
  for (int i = tid; i < 2048; i += TC_NT) hist[i] = 0;
  __syncthreads();
  double se = 0.0;
  {
    float se_f = 0.f;
    const float mx2 = mx * kLog2e;
    for (int i0 = 0; i0 < vocab; i0 += TC_NT) {
      const int i = i0 + tid;
      const bool in = i < vocab;
      const float x = in ? z[i] : 0.f;
      const uint32_t key = okey(x);
      const bool cand = in && (key >> 21) == d1;
      const uint32_t voters = __ballot_sync(0xffffffffu, cand);
      if (in) se_f += exp2f(fmaf(x, kLog2e, -mx2));
      if (cand) {
        const uint32_t bin = (key >> 10) & 2047u;
        const uint32_t peers = __match_any_sync(voters, bin);
        if (lane == (__ffs(peers) - 1)) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
      }
    }
    se = (double)se_f;
  }
  se = block_reduce_sum(se, red_d);
  pick_digit(hist, 2048, remaining, warp_tot, s_pick);
  const uint32_t d2 = s_pick[0];
  remaining = s_pick[1];
  const uint32_t prefix22 = (d1 << 11) | d2;
  __syncthreads();

  // ---- pass 3 (L2): sum of logits above the 22-bit prefix, histogram of the last 10 bits ----
  for (int i = tid; i < 1024; i += TC_NT) hist[i] = 0;
  __syncthreads();
  double top = 0.0;
  for (int i0 = 0; i0 < vocab; i0 += TC_NT) {
    const int i = i0 + tid;
    const bool in = i < vocab;
    const float x = in ? z[i] : 0.f;
    const uint32_t key = okey(x);
    const uint32_t p22 = key >> 10;
    const bool cand = in && p22 == prefix22;
    const uint32_t voters = __ballot_sync(0xffffffffu, cand);
    if (in && p22 > prefix22) top += (double)x;
    if (cand) {
      const uint32_t bin = key & 1023u;
      const uint32_t peers = __match_any_sync(voters, bin);
      if (lane == (__ffs(peers) - 1)) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
    }
  }
  top = block_reduce_sum(top, red_d);
  pick_digit(hist, 1024, remaining, warp_tot, s_pick);
  if (tid == 0) {
    const uint32_t d3 = s_pick[0];
    const uint32_t need = s_pick[1];
    // keys sharing the 22-bit prefix: value is fixed by the last digit, counts are in hist
    for (uint32_t b = 1023; b > d3; --b)
      if (hist[b]) top += (double)hist[b] * (double)okey_inv((prefix22 << 10) | b);
    top += (double)need * (double)okey_inv((prefix22 << 10) | d3);
    const float lse = mx + logf((float)se);
    const float T = lse - (float)(top / (double)k);
    // request of this row: last r with tok_indptr[r] <= row
    int lo = 0, hi = n_req;
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (tok_indptr[mid] <= row) lo = mid; else hi = mid;
    }
    const int pos = hist_len[lo] + (row - tok_indptr[lo]);
    if (pos < hist_cap) conf_hist[(int64_t)lo * hist_cap + pos] = T;
    else report(status, ACTKV_E_INVALID, lo, pos);
  }
}

// -----------------------------------------------------------------------------------------------
// Single-sweep token confidence.  The k-th largest of any subset of a row is a lower bound of the
// k-th largest of the row, so: (A) take the first SW_HEAD logits into shared memory and find their
// k-th largest tau exactly; (B) stream the rest of the row ONCE from HBM with an online
// (max, sum of exp) per thread, appending the few logits >= tau to a shared candidate list;
// (C) the top k of head-candidates + list are the top k of the row.  Rows whose list overflows
// (adversarial order, e.g. ascending logits) are flagged and redone by the three-sweep kernel.
constexpr int SW_HEAD = 8192;
constexpr int SW_CAP = 4096;

struct SweepSmem {
  float head[SW_HEAD];
  float cand[SW_CAP];
  uint32_t hist[2048];
  uint32_t warp_tot[TC_NT / 32];
  uint32_t pick[3];
  uint32_t n_cand;
  float red_f[TC_NT / 32];
  double red_d[TC_NT / 32];
};

// k-th largest (k >= 1) of vals[0..n) by three radix digits; all threads call it.  Returns the key of
// that element and the number of elements equal to it that belong to the top k.
__device__ __forceinline__ void smem_kth_largest(const float* vals, int n, uint32_t k, SweepSmem* sm,
                                                 uint32_t& key_out, uint32_t& need_out) {
  const int tid = threadIdx.x;
  uint32_t prefix = 0, remaining = k;
  for (int pass = 0; pass < 3; ++pass) {
    const int nb = pass == 2 ? 1024 : 2048;
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    for (int i = tid; i < nb; i += TC_NT) sm->hist[i] = 0;
    __syncthreads();
    for (int i = tid; i < n; i += TC_NT) {
      const uint32_t key = okey(vals[i]);
      const bool in = pass == 0 || (pass == 1 ? (key >> 21) == prefix : (key >> 10) == prefix);
      if (in) atomicAdd(&sm->hist[(key >> shift) & (uint32_t)(nb - 1)], 1u);
    }
    __syncthreads();
    pick_digit(sm->hist, nb, remaining, sm->warp_tot, sm->pick);
    prefix = (pass == 0) ? sm->pick[0] : ((prefix << (pass == 1 ? 11 : 10)) | sm->pick[0]);
    remaining = sm->pick[1];
    __syncthreads();
  }
  key_out = prefix;
  need_out = remaining;
}

__global__ void __launch_bounds__(TC_NT, 1) token_conf_sweep_kernel(
    const float* __restrict__ logits, const int32_t* __restrict__ tok_indptr, int32_t vocab, int32_t n_req,
    int32_t k_top, float* __restrict__ conf_hist, const int32_t* __restrict__ hist_len, int32_t hist_cap,
    int32_t* __restrict__ redo, int32_t* status) {
  extern __shared__ __align__(16) uint8_t sweep_raw[];
  SweepSmem* sm = reinterpret_cast<SweepSmem*>(sweep_raw);
  const int row = blockIdx.x, tid = threadIdx.x;
  const float* z = logits + (int64_t)row * vocab;
  const int k = min(k_top, vocab);
  const int n_head = min(vocab, SW_HEAD);

  // ---- (A) head of the row -> shared memory, its k-th largest is the candidate threshold ----
  for (int i = tid; i < n_head; i += TC_NT) sm->head[i] = z[i];
  if (tid == 0) sm->n_cand = 0;
  __syncthreads();
  uint32_t tau_key, need;
  smem_kth_largest(sm->head, n_head, (uint32_t)k, sm, tau_key, need);
  const float tau = okey_inv(tau_key);

  // ---- (B) one sweep: online (max, sum exp2) per thread, candidates >= tau ----
  float m = -INFINITY, s = 0.f;
  auto visit = [&](float x, bool collect) {
    if (x > m) { s *= exp2f((m - x) * kLog2e); m = x; }      // m = -inf: s is 0 and stays 0
    s += exp2f((x - m) * kLog2e);
    if (collect && x >= tau) {
      const uint32_t pos = atomicAdd(&sm->n_cand, 1u);
      if (pos < SW_CAP) sm->cand[pos] = x;
    }
  };
  for (int i = tid; i < n_head; i += TC_NT) visit(sm->head[i], false);
  const bool vec = (vocab % 4 == 0) && ((reinterpret_cast<uintptr_t>(z) & 15) == 0) && (SW_HEAD % 4 == 0);
  if (vec) {
    const float4* z4 = reinterpret_cast<const float4*>(z);
    const int n4 = vocab / 4;
    int i = SW_HEAD / 4 + tid;
    for (; i + 3 * TC_NT < n4; i += 4 * TC_NT) {               // four 16-byte loads in flight per thread
      const float4 a = z4[i], b = z4[i + TC_NT], c = z4[i + 2 * TC_NT], d = z4[i + 3 * TC_NT];
      visit(a.x, true); visit(a.y, true); visit(a.z, true); visit(a.w, true);
      visit(b.x, true); visit(b.y, true); visit(b.z, true); visit(b.w, true);
      visit(c.x, true); visit(c.y, true); visit(c.z, true); visit(c.w, true);
      visit(d.x, true); visit(d.y, true); visit(d.z, true); visit(d.w, true);
    }
    for (; i < n4; i += TC_NT) {
      const float4 a = z4[i];
      visit(a.x, true); visit(a.y, true); visit(a.z, true); visit(a.w, true);
    }
  } else {
    for (int i = SW_HEAD + tid; i < vocab; i += TC_NT) visit(z[i], true);
  }
  // block (max, sum): fixed-order trees
  const float M = block_reduce_max(m, sm->red_f);
  const double S = block_reduce_sum((m > -INFINITY) ? (double)s * (double)exp2f((m - M) * kLog2e) : 0.0, sm->red_d);
  __syncthreads();
  const uint32_t n_cand = sm->n_cand;
  if (n_cand > SW_CAP) {                                     // adversarial order: leave the row to the fallback
    if (tid == 0) redo[row] = 1;
    return;
  }
  // ---- (C) top k of {head elements >= tau} U candidates ----
  // move the head's own candidates behind the streamed ones (at most k + ties of them; ties could be many,
  // so the count is checked again)
  for (int i = tid; i < n_head; i += TC_NT) {
    const float x = sm->head[i];
    if (x >= tau) {
      const uint32_t pos = atomicAdd(&sm->n_cand, 1u);
      if (pos < SW_CAP) sm->cand[pos] = x;
    }
  }
  __syncthreads();
  const uint32_t n_all = sm->n_cand;
  if (n_all > SW_CAP) {
    if (tid == 0) redo[row] = 1;
    return;
  }
  uint32_t kth_key, need_k;
  smem_kth_largest(sm->cand, (int)n_all, (uint32_t)k, sm, kth_key, need_k);
  const float kth = okey_inv(kth_key);
  double top = 0.0;
  for (int i = tid; i < (int)n_all; i += TC_NT) {
    const float x = sm->cand[i];
    if (okey(x) > kth_key) top += (double)x;
  }
  top = block_reduce_sum(top, sm->red_d);
  if (tid == 0) {
    redo[row] = 0;
    top += (double)need_k * (double)kth;
    const float lse = M + logf((float)S);
    const float T = lse - (float)(top / (double)k);
    int lo = 0, hi = n_req;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (tok_indptr[mid] <= row) lo = mid; else hi = mid;
    }
    const int pos = hist_len[lo] + (row - tok_indptr[lo]);
    if (pos < hist_cap) conf_hist[(int64_t)lo * hist_cap + pos] = T;
    else report(status, ACTKV_E_INVALID, lo, pos);
  }
}

struct BudgetParamsDev {
  int32_t w, s;
  double b_percent, scale_up;
  int32_t B_upper, clamp_lo_ppm, clamp_hi_ppm;
};

constexpr int TR_NT = 256;

__global__ void __launch_bounds__(TR_NT) trend_kernel(
    const int32_t* __restrict__ tok_indptr, const float* __restrict__ conf_hist, int32_t* hist_len,
    int32_t hist_cap, BudgetParamsDev p, const int32_t* __restrict__ seq_len,
    const int32_t* __restrict__ budget_in, int32_t* __restrict__ budget_out, double* slope_out,
    float* pooled_ws, int32_t max_m) {
  const int r = blockIdx.x, tid = threadIdx.x;
  const int n_new = tok_indptr ? tok_indptr[r + 1] - tok_indptr[r] : 0;
  const int Lh = min(hist_cap, hist_len[r] + n_new);
  const float* TL = conf_hist + (int64_t)r * hist_cap;
  float* Rp = pooled_ws + (int64_t)r * max_m;           // R' then (in place, compacted) R
  __shared__ float s_q;
  const int M = (Lh >= p.w) ? (Lh - p.w) / p.s + 1 : 0;
  for (int m = tid; m < M; m += TR_NT) {
    float v = TL[m * p.s];
    for (int i = 1; i < p.w; ++i) v = fminf(v, TL[m * p.s + i]);
    Rp[m] = v;
  }
  __syncthreads();
  double alpha = 0.0;
  if (M > 0) {
    int rank = (int)ceil(p.b_percent * (double)M / 100.0);
    if (rank < 1) rank = 1;
    if (rank > M) rank = M;
    // nearest-rank percentile: the value v with #(< v) < rank <= #(<= v)
    for (int m = tid; m < M; m += TR_NT) {
      const float v = Rp[m];
      int lt = 0, le = 0;
      for (int j = 0; j < M; ++j) { const float x = Rp[j]; lt += x < v; le += x <= v; }
      if (lt < rank && rank <= le) s_q = v;            // every writer holds the same value
    }
    __syncthreads();
    const float qv = s_q;
    // R = values <= q in time order; slope by one thread in float64 (|R| is small)
    if (tid == 0) {
      int n = 0;
      double sy = 0.0;
      for (int m = 0; m < M; ++m) if (Rp[m] <= qv) { sy += (double)Rp[m]; ++n; }
      if (n >= 2) {
        const double xm = (double)(n - 1) * 0.5;                            // mean of 0..n-1, exact
        const double ym = sy / (double)n;
        double sxy = 0.0, sxx = 0.0;
        int i = 0;
        for (int m = 0; m < M; ++m) if (Rp[m] <= qv) {
          const double dx = (double)i - xm;
          sxy += dx * ((double)Rp[m] - ym);
          sxx += dx * dx;
          ++i;
        }
        alpha = sxy / sxx;
      }
    }
  }
  if (tid == 0) {
    long long B = budget_in[r];
    if (alpha < 0.0) {
      double scaled = floor((double)B * p.scale_up);
      long long Bs = (long long)scaled;
      B = Bs < (long long)p.B_upper ? Bs : (long long)p.B_upper;
    }
    if (p.clamp_hi_ppm > 0 && seq_len != nullptr) {
      const long long L = seq_len[r];
      const long long lo = (L * p.clamp_lo_ppm + 999999LL) / 1000000LL;
      const long long hi = (L * p.clamp_hi_ppm) / 1000000LL;
      if (B < lo) B = lo;
      if (B > hi) B = hi;
    }
    budget_out[r] = (int32_t)B;
    if (slope_out) slope_out[r] = alpha;
    hist_len[r] = Lh;
  }
}

}  // namespace actkv

extern "C" {

size_t actkv_budget_workspace_bytes(int32_t n_rows, int32_t n_req, int32_t hist_cap) {
  if (n_rows < 0 || n_req < 0 || hist_cap < 0) return 0;
  // new confidences + one pooled sequence of at most hist_cap values per request
  return actkv::align_up((size_t)n_rows * 4, 256) + actkv::align_up((size_t)n_req * hist_cap * 4, 256);
}

int actkv_budget(const float* logits, const int32_t* tok_indptr, int32_t n_rows, int32_t vocab,
                 float* conf_hist, int32_t* hist_len, int32_t hist_cap,
                 const actkv_budget_params_t* params, const int32_t* seq_len,
                 const int32_t* budget_in, int32_t* budget_out, double* slope_out, int32_t n_req,
                 void* ws, size_t ws_bytes, int32_t* status, actkv_stream_t stream) {
  if (!params || n_req < 0 || n_rows < 0 || hist_cap <= 0 || hist_cap > 65536) return ACTKV_E_INVALID;
  if (params->k <= 0 || params->w <= 0 || params->s <= 0 || !(params->b_percent >= 0.0)) return ACTKV_E_INVALID;
  if (n_req == 0) return ACTKV_OK;
  if (!conf_hist || !hist_len || !budget_in || !budget_out || !ws) return ACTKV_E_INVALID;
  if (n_rows > 0 && (!logits || !tok_indptr || vocab <= 0)) return ACTKV_E_INVALID;
  if (params->clamp_hi_ppm > 0 && !seq_len) return ACTKV_E_INVALID;
  if (ws_bytes < actkv_budget_workspace_bytes(n_rows, n_req, hist_cap)) return ACTKV_E_WORKSPACE;
  cudaStream_t s = (cudaStream_t)stream;
  int32_t* redo = (int32_t*)ws;                 // per row: 1 = the single-sweep kernel gave up, redo in three sweeps
  float* pooled = (float*)((char*)ws + actkv::align_up((size_t)n_rows * 4, 256));
  if (n_rows > 0) {
    const size_t sm = sizeof(actkv::SweepSmem);
    if (cudaFuncSetAttribute(actkv::token_conf_sweep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm) !=
        cudaSuccess)
      return ACTKV_E_CUDA;
    actkv::token_conf_sweep_kernel<<<(unsigned)n_rows, actkv::TC_NT, sm, s>>>(
        logits, tok_indptr, vocab, n_req, params->k, conf_hist, hist_len, hist_cap, redo, status);
    ACTKV_CHECK_LAUNCH();
    actkv::token_conf_kernel<<<(unsigned)n_rows, actkv::TC_NT, 0, s>>>(
        logits, tok_indptr, vocab, n_req, params->k, conf_hist, hist_len, hist_cap, redo, status);
    ACTKV_CHECK_LAUNCH();
  }
  actkv::BudgetParamsDev p{params->w, params->s, params->b_percent, params->scale_up,
                           params->B_upper, params->clamp_lo_ppm, params->clamp_hi_ppm};
  const int32_t max_m = hist_cap;
  actkv::trend_kernel<<<(unsigned)n_req, actkv::TR_NT, 0, s>>>(
      n_rows > 0 ? tok_indptr : nullptr, conf_hist, hist_len, hist_cap, p, seq_len, budget_in,
      budget_out, slope_out, pooled, max_m);
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

}  // extern "C"
