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
  // each thread owns `per` (at most 4) adjacent bins, descending from nbins - 1 - per * tid
  const int per = (nbins + (int)blockDim.x - 1) / (int)blockDim.x;
  const int b0 = nbins - 1 - per * tid;
  uint32_t v[4], mine = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int b = b0 - j;
    v[j] = (j < per && b >= 0) ? hist[b] : 0u;
    mine += v[j];
  }
  uint32_t incl = mine;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    uint32_t t = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += t;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  uint32_t acc = incl - mine;                    // #(digit > b0)
  for (int w = 0; w < warp; ++w) acc += warp_tot[w];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int b = b0 - j;
    if (j < per && b >= 0 && acc < remaining && acc + v[j] >= remaining) {
      s_out[0] = (uint32_t)b; s_out[1] = remaining - acc; s_out[2] = v[j];
    }
    acc += v[j];
  }
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
// Single-sweep token confidence.  A lower bound tau of the row's k-th largest logit lets one sweep keep
// only the few logits >= tau while it sums the exponentials:
//  (A) the first SW_HEAD logits are split into 64 chunks; the k-th largest of the 64 chunk maxima is tau
//      (k of the row's logits are at least that large; k <= 64), the largest of them the reference M of
//      the exponentials;
//  (B) the row is streamed ONCE from HBM: sum of exp(x - M) per thread, logits >= tau appended to a shared
//      candidate list (about half a percent of the row);
//  (C) the top k of the list are the top k of the row: exact radix select in shared memory.
// Rows whose list overflows (adversarial order, e.g. ascending logits), whose sum overflows (M is not the
// row's maximum) or with k > 64 are flagged and redone by the three-sweep kernel.
// Two CTAs of 512 threads per SM: one streams while the other is in its serial phases.
constexpr int SW_HEAD = 4096;
constexpr int SW_CAP = 4096;
constexpr int SW_NT = 512;
constexpr int SW_PER = SW_HEAD / SW_NT;     // head logits per thread (8: a chunk is 8 lanes x 8 = 64 logits)

struct SweepSmem {
  float cand[SW_CAP];
  uint32_t hist[2048];
  float chunk_max[64];
  uint32_t warp_tot[SW_NT / 32];
  uint32_t pick[3];
  uint32_t n_cand;
  float tau, ref;
  float red_f[SW_NT / 32];
  double red_d[SW_NT / 32];
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
    for (int i = tid; i < nb; i += SW_NT) sm->hist[i] = 0;
    __syncthreads();
    for (int i = tid; i < n; i += SW_NT) {
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

__global__ void __launch_bounds__(SW_NT, 2) token_conf_sweep_kernel(
    const float* __restrict__ logits, const int32_t* __restrict__ tok_indptr, int32_t vocab, int32_t n_req,
    int32_t k_top, float* __restrict__ conf_hist, const int32_t* __restrict__ hist_len, int32_t hist_cap,
    int32_t* __restrict__ redo, int32_t* status) {
  extern __shared__ __align__(16) uint8_t sweep_raw[];
  SweepSmem* sm = reinterpret_cast<SweepSmem*>(sweep_raw);
  const int row = blockIdx.x, tid = threadIdx.x;
  const float* z = logits + (int64_t)row * vocab;
  const int k = min(k_top, vocab);
  const int n_head = min(vocab, SW_HEAD);

  // ---- (A) threshold and reference from the chunk maxima of the head ----
  const bool vec = (vocab % 4 == 0) && ((reinterpret_cast<uintptr_t>(z) & 15) == 0);
  float hv[SW_PER];
  float hm = -INFINITY;
#pragma unroll
  for (int j = 0; j < SW_PER; ++j) {
    const int i = tid * SW_PER + j;
    hv[j] = (i < n_head) ? z[i] : -INFINITY;
    hm = fmaxf(hm, hv[j]);
  }
#pragma unroll
  for (int o = 4; o >= 1; o >>= 1) hm = fmaxf(hm, __shfl_xor_sync(0xffffffffu, hm, o));     // over 8 lanes
  if ((tid & 7) == 0) sm->chunk_max[tid >> 3] = hm;
  if (tid == 0) sm->n_cand = 0;
  __syncthreads();
  if (tid < 64) {
    const float v = sm->chunk_max[tid];
    int rank = 0;                                            // chunk maxima that come before this one, descending
    float top = -INFINITY;
    for (int u = 0; u < 64; ++u) {
      const float w = sm->chunk_max[u];
      rank += (w > v || (w == v && u < tid)) ? 1 : 0;
      top = fmaxf(top, w);
    }
    if (rank == k - 1) sm->tau = v;
    if (tid == 0) sm->ref = top;
  }
  __syncthreads();
  const float tau = sm->tau, M = sm->ref;
  if (k > 64 || !(M > -INFINITY)) {                          // (uniform) no bound from 64 maxima: the fallback's row
    if (tid == 0) redo[row] = 1;
    return;
  }

  // ---- (B) one sweep: sum of exp(x - M) per thread, candidates >= tau.  M is the maximum of the head, not
  //      of the row: later logits may exceed it (the sum may grow up to the float range; a row whose sum
  //      overflows is left to the fallback) ----
  const float nmc = -M * kLog2e;
  float s = 0.f;
  auto visit = [&](float x) {
    s += exp2f(fmaf(x, kLog2e, nmc));
    if (x >= tau) {
      const uint32_t pos = atomicAdd(&sm->n_cand, 1u);
      if (pos < SW_CAP) sm->cand[pos] = x;
    }
  };
#pragma unroll
  for (int j = 0; j < SW_PER; ++j)
    if (tid * SW_PER + j < n_head) visit(hv[j]);
  if (vec) {
    const float4* z4 = reinterpret_cast<const float4*>(z);
    const int n4 = vocab / 4;
    int i = SW_HEAD / 4 + tid;
    for (; i + 7 * SW_NT < n4; i += 8 * SW_NT) {               // eight 16-byte loads in flight per thread
      float4 v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = z4[i + j * SW_NT];
#pragma unroll
      for (int j = 0; j < 8; ++j) { visit(v[j].x); visit(v[j].y); visit(v[j].z); visit(v[j].w); }
    }
    for (; i < n4; i += SW_NT) {
      const float4 a = z4[i];
      visit(a.x); visit(a.y); visit(a.z); visit(a.w);
    }
  } else {
    for (int i = SW_HEAD + tid; i < vocab; i += SW_NT) visit(z[i]);
  }
  const double S = block_reduce_sum((double)s, sm->red_d);   // fixed-order tree
  __syncthreads();
  const uint32_t n_cand = sm->n_cand;
  if (n_cand > SW_CAP || !(S < 3.0e38)) {                    // adversarial order or overflow: the fallback's row
    if (tid == 0) redo[row] = 1;
    return;
  }
  // ---- (C) the top k of the candidates are the top k of the row ----
  const uint32_t n_all = n_cand;
  uint32_t kth_key, need_k;
  smem_kth_largest(sm->cand, (int)n_all, (uint32_t)k, sm, kth_key, need_k);
  const float kth = okey_inv(kth_key);
  double top = 0.0;
  for (int i = tid; i < (int)n_all; i += SW_NT) {
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
    // nearest-rank percentile: the rank-th smallest value, i.e. the v with #(< v) < rank <= #(<= v), by a radix
    // select over the order-preserving integer image of the values (four 8-bit digits, most significant first):
    // 4 M steps for any history length (counting the values below each candidate would take M^2)
    __shared__ uint32_t s_hist[256];
    __shared__ uint32_t s_prefix, s_remaining;
    if (tid == 0) { s_prefix = 0u; s_remaining = (uint32_t)rank; }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      const uint32_t himask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
      s_hist[tid] = 0u;                                  // TR_NT == 256 bins
      __syncthreads();
      const uint32_t prefix = s_prefix;
      for (int m = tid; m < M; m += TR_NT) {
        const uint32_t k = okey(Rp[m]);
        if ((k & himask) == prefix) atomicAdd(&s_hist[(k >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (tid == 0) {
        uint32_t acc = 0, rem = s_remaining;
        for (int d = 0; d < 256; ++d) {                  // ascending: the digit that holds the rem-th smallest
          if (acc + s_hist[d] >= rem) { s_prefix = prefix | ((uint32_t)d << shift); s_remaining = rem - acc; break; }
          acc += s_hist[d];
        }
      }
      __syncthreads();
    }
    if (tid == 0) s_q = okey_inv(s_prefix);
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
    if (actkv::ensure_dyn_smem(actkv::token_conf_sweep_kernel, sm) != cudaSuccess) return ACTKV_E_CUDA;
    actkv::token_conf_sweep_kernel<<<(unsigned)n_rows, actkv::SW_NT, sm, s>>>(
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
