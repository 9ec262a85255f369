// actkv_select: TopK(score, k = B) per (layer x KV head, request) unit — Algorithm 1, step 5,
// applied to the pooled action-region score.  One CTA per unit: a 4 x 8-bit most-significant-
// digit radix select over the order-preserving integer image of the float32 scores finds the
// n-th largest value exactly; one ordered sweep with a block scan then emits the kept token
// indices in ascending order, entries equal to the threshold being kept lowest index first.
// Scores are 4 bytes per token and unit-local, so the five sweeps after the first read hit L2.
#include "common.cuh"

namespace actkv {

constexpr int SEL_NT = 1024;
constexpr int SEL_ITEMS = 4;

__device__ __forceinline__ uint32_t order_key(float x) {
  uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);     // larger float -> larger key
}

__global__ void __launch_bounds__(SEL_NT) select_kernel(
    const float* __restrict__ score, const int32_t* __restrict__ tok_indptr, int32_t sum_tok,
    const int32_t* __restrict__ budget, int32_t n_req, const int32_t* __restrict__ keep_indptr,
    int32_t* __restrict__ sel_idx, int64_t sel_stride, uint32_t* __restrict__ keep_mask,
    actkv_tie_t* __restrict__ tie, int32_t* status) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t warp_tot[SEL_NT / 32];
  __shared__ uint32_t s_bin, s_remaining, s_eq_total;
  __shared__ unsigned long long s_carry;

  const int u = blockIdx.x;
  const int r = u % n_req, o = u / n_req;
  const int base = tok_indptr[r];
  const int L = tok_indptr[r + 1] - base;
  int B = budget[r];
  if (B < 0) B = 0;
  const int n = min(B, L);
  const float* sc = score + (int64_t)o * sum_tok + base;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (n == 0) {
    if (tie != nullptr && tid == 0) tie[u] = actkv_tie_t{0.f, 0, 0, 0};
    return;
  }

  // ---- radix select: n-th largest key -----------------------------------------------------
  uint32_t prefix = 0, mask = 0, remaining = (uint32_t)n;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int i0 = 0; i0 < L; i0 += SEL_NT) {               // warp-uniform trip count
      const int i = i0 + tid;
      const uint32_t k = (i < L) ? order_key(sc[i]) : 0u;
      const bool in = (i < L) && (k & mask) == prefix;
      const uint32_t voters = __ballot_sync(0xffffffffu, in);
      if (in) {
        const uint32_t bin = (k >> shift) & 255u;
        // warp-aggregated increment: lanes with the same bin elect one to add their count
        const uint32_t peers = __match_any_sync(voters, bin);
        if (lane == (__ffs(peers) - 1)) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
      }
    }
    __syncthreads();
    // suffix sums over the 256 bins: cum(b) = #keys with digit >= b
    uint32_t v = 0, incl = 0;
    if (tid < 256) {
      v = hist[255 - tid];                               // reversed so a prefix scan is a suffix sum
      incl = v;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        uint32_t t = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += t;
      }
      if (lane == 31) warp_tot[warp] = incl;
    }
    __syncthreads();
    if (tid < 256) {
      uint32_t add = 0;
      for (int w = 0; w < warp; ++w) add += warp_tot[w];
      incl += add;                                       // keys with digit >= 255 - tid
      uint32_t excl = incl - v;                          // keys with digit >  255 - tid
      if (incl >= remaining && excl < remaining) {
        s_bin = 255u - (uint32_t)tid;
        s_remaining = remaining - excl;
        s_eq_total = v;
      }
    }
    __syncthreads();
    prefix |= s_bin << shift;
    mask |= 255u << shift;
    remaining = s_remaining;
    __syncthreads();
  }
  const uint32_t thr = prefix;                           // key of the n-th largest score
  const uint32_t need_eq = remaining;                    // entries equal to it that are kept
  const uint32_t eq_total = s_eq_total;

  // ---- ordered sweep: emit kept indices ascending ---------------------------------------------
  if (tid == 0) s_carry = 0ull;
  __syncthreads();
  int32_t* out = sel_idx + (int64_t)o * sel_stride + keep_indptr[r];
  uint32_t* mask_row = keep_mask ? keep_mask + (int64_t)o * ((sum_tok + 31) / 32) : nullptr;
  for (int c0 = 0; c0 < L; c0 += SEL_NT * SEL_ITEMS) {
    const int i0 = c0 + tid * SEL_ITEMS;
    uint32_t gt[SEL_ITEMS], eq[SEL_ITEMS];
    unsigned long long mine = 0ull;                      // high 32: #greater, low 32: #equal
#pragma unroll
    for (int k = 0; k < SEL_ITEMS; ++k) {
      const int i = i0 + k;
      uint32_t key = (i < L) ? order_key(sc[i]) : 0u;
      gt[k] = (i < L) && key > thr;
      eq[k] = (i < L) && key == thr;
      mine += ((unsigned long long)gt[k] << 32) + eq[k];
    }
    unsigned long long incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      unsigned long long t = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += t;
    }
    __shared__ unsigned long long wsum[SEL_NT / 32];
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    unsigned long long before = s_carry;
    for (int w = 0; w < warp; ++w) before += wsum[w];
    before += incl - mine;
    uint32_t gt_before = (uint32_t)(before >> 32), eq_before = (uint32_t)before;
#pragma unroll
    for (int k = 0; k < SEL_ITEMS; ++k) {
      const int i = i0 + k;
      const bool keep = gt[k] || (eq[k] && eq_before < need_eq);
      if (keep) {
        const uint32_t pos = gt_before + min(eq_before, need_eq);
        out[pos] = i;
        if (mask_row) atomicOr(&mask_row[(base + i) >> 5], 1u << ((base + i) & 31));
      }
      gt_before += gt[k];
      eq_before += eq[k];
    }
    __syncthreads();
    if (tid == SEL_NT - 1) s_carry = before + mine;
    __syncthreads();
  }
  if (tie != nullptr && tid == 0) {
    uint32_t b = (thr & 0x80000000u) ? (thr & 0x7fffffffu) : ~thr;
    tie[u] = actkv_tie_t{__uint_as_float(b), (int32_t)need_eq, (int32_t)eq_total, n};
  }
  (void)status;
}

__global__ void keep_indptr_kernel(const int32_t* seq_len, const int32_t* budget, int32_t n_req,
                                   int32_t* keep_indptr) {
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    int32_t acc = 0;
    keep_indptr[0] = 0;
    for (int r = 0; r < n_req; ++r) {
      int32_t b = budget[r] < 0 ? 0 : budget[r];
      acc += min(b, seq_len[r]);
      keep_indptr[r + 1] = acc;
    }
  }
}

}  // namespace actkv

extern "C" {

size_t actkv_select_workspace_bytes(int32_t, int32_t, int32_t) { return 0; }

int actkv_select(const float* score, const int32_t* tok_indptr, int32_t sum_tok,
                 const int32_t* budget, int32_t n_outer, int32_t n_req,
                 const int32_t* keep_indptr, int32_t* sel_idx, int64_t sel_stride,
                 uint32_t* keep_mask, actkv_tie_t* tie_report, void* ws, size_t ws_bytes,
                 int32_t* status, actkv_stream_t stream) {
  (void)ws; (void)ws_bytes;
  if (n_outer < 0 || n_req < 0 || sum_tok < 0 || sel_stride < 0) return ACTKV_E_INVALID;
  if (n_outer == 0 || n_req == 0) return ACTKV_OK;
  if (!score || !tok_indptr || !budget || !keep_indptr || !sel_idx) return ACTKV_E_INVALID;
  const int64_t units = (int64_t)n_outer * n_req;
  if (units > 0x7fffffffLL) return ACTKV_E_INVALID;
  actkv::select_kernel<<<(unsigned)units, actkv::SEL_NT, 0, (cudaStream_t)stream>>>(
      score, tok_indptr, sum_tok, budget, n_req, keep_indptr, sel_idx, sel_stride, keep_mask,
      tie_report, status);
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

int actkv_keep_indptr(const int32_t* seq_len, const int32_t* budget, int32_t n_req,
                      int32_t* keep_indptr, actkv_stream_t stream) {
  if (n_req < 0 || !keep_indptr || (n_req > 0 && (!seq_len || !budget))) return ACTKV_E_INVALID;
  actkv::keep_indptr_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(seq_len, budget, n_req, keep_indptr);
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

}  // extern "C"
