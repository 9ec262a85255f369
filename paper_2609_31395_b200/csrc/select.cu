// actkv_select: TopK(score, k = B) per (layer x KV head, request) unit — Algorithm 1, step 5,
// applied to the pooled action-region score.  One CTA per unit.  The unit's scores are read once and
// kept in shared memory as order-preserving 32-bit keys (up to 53 K tokens; longer units re-read them
// from L2); a most-significant-digit radix select with digits of 12, 12 and 8 bits (shared-memory
// histograms, plain atomics: a warp's keys spread over many bins once the digit reaches into the
// mantissa, and over the few dozen bins of the populated binades before) finds the n-th largest key
// exactly; one ordered sweep with a block scan then emits the kept token indices in ascending order,
// entries equal to the threshold being kept lowest index first.
#include "select_core.cuh"

namespace actkv {

constexpr size_t SEL_SMEM = 232448 - 1024;                            // (nearly) all of an SM's shared memory: one CTA per SM
constexpr int SEL_CAP = (int)((SEL_SMEM - SEL_BINS * 4) / 4);          // keys that fit beside the histogram

__device__ __forceinline__ uint32_t order_key(float x) {
  uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);     // larger float -> larger key
}

__global__ void __launch_bounds__(SEL_NT, 1) select_kernel(
    const float* __restrict__ score, const int32_t* __restrict__ tok_indptr, int32_t sum_tok,
    const int32_t* __restrict__ budget, int32_t n_req, const int32_t* __restrict__ keep_indptr,
    int32_t* __restrict__ sel_idx, int64_t sel_stride, uint32_t* __restrict__ keep_mask,
    actkv_tie_t* __restrict__ tie, int32_t* status) {
  extern __shared__ __align__(16) uint32_t sel_smem[];
  uint32_t* hist = sel_smem;                             // [SEL_BINS]
  uint32_t* skeys = sel_smem + SEL_BINS;                 // [SEL_CAP]
  const int u = blockIdx.x;
  const int r = u % n_req, o = u / n_req;
  const int base = tok_indptr[r];
  const int L = tok_indptr[r + 1] - base;
  int B = budget[r];
  if (B < 0) B = 0;
  const int n = min(B, L);
  const float* sc = score + (int64_t)o * sum_tok + base;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // An earlier stage of the step failed (a score kernel that gave up, a bad table): its scores are not
  // consumed.  A budget the host did not size the index buffer for (the budgets are device data, e.g.
  // straight from actkv_budget) is reported before anything is stored.
  if (status_set(status)) return;
  if ((int64_t)keep_indptr[r] + n > sel_stride) {
    if (tid == 0) report(status, ACTKV_E_INVALID, r, n);
    return;
  }
  if (n == 0) {
    if (tie != nullptr && tid == 0) tie[u] = actkv_tie_t{0.f, 0, 0, 0};
    return;
  }
  const bool resident = L <= SEL_CAP;                    // uniform over the CTA
  auto key_at = [&](int i) -> uint32_t { return resident ? skeys[i] : order_key(sc[i]); };
  // The one read of the scores (16-byte vectors between an unaligned head and tail) also fills the
  // histogram of the first digit.
  for (int i = tid; i < SEL_BINS; i += SEL_NT) hist[i] = 0;
  __syncthreads();
  {
    auto take = [&](int i, float x) {
      const uint32_t k = order_key(x);
      if (resident) skeys[i] = k;
      atomicAdd(&hist[k >> 20], 1u);
    };
    const int head = min(L, (int)((16u - ((uint32_t)(uintptr_t)sc & 15u)) & 15u) >> 2);
    const int n_vec = (L - head) >> 2;
    if (tid < head) take(tid, sc[tid]);
    const float4* sc4 = reinterpret_cast<const float4*>(sc + head);
    // (four loads in flight per thread: the read is bound by latency, not by bandwidth)
    for (int v0 = tid; v0 < n_vec; v0 += 4 * SEL_NT) {
      float4 x[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int v = v0 + j * SEL_NT;
        x[j] = v < n_vec ? __ldg(sc4 + v) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int v = v0 + j * SEL_NT;
        if (v < n_vec) {
          const int i = head + 4 * v;
          take(i, x[j].x); take(i + 1, x[j].y); take(i + 2, x[j].z); take(i + 3, x[j].w);
        }
      }
    }
    const int tail0 = head + 4 * n_vec;
    if (tail0 + tid < L) take(tail0 + tid, sc[tail0 + tid]);
  }

  select_threshold_and_emit(key_at, hist, L, n, sel_idx + (int64_t)o * sel_stride + keep_indptr[r],
                            keep_mask ? keep_mask + (int64_t)o * ((sum_tok + 31) / 32) : nullptr, base, tie, u);
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
  if (actkv::ensure_dyn_smem(actkv::select_kernel, actkv::SEL_SMEM) != cudaSuccess)
    return ACTKV_E_CUDA;
  actkv::select_kernel<<<(unsigned)units, actkv::SEL_NT, actkv::SEL_SMEM, (cudaStream_t)stream>>>(
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
