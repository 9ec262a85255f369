// actkv_select: TopK(score, k = B) per (layer x KV head, request) unit — Algorithm 1, step 5,
// applied to the pooled action-region score.  One CTA per unit.  The unit's scores are read once and
// kept in shared memory as order-preserving 32-bit keys (up to 53 K tokens; longer units re-read them
// from L2); a most-significant-digit radix select with digits of 12, 12 and 8 bits (shared-memory
// histograms, plain atomics: a warp's keys spread over many bins once the digit reaches into the
// mantissa, and over the few dozen bins of the populated binades before) finds the n-th largest key
// exactly; one ordered sweep with a block scan then emits the kept token indices in ascending order,
// entries equal to the threshold being kept lowest index first.
#include "common.cuh"

namespace actkv {

constexpr int SEL_NT = 1024;
constexpr int SEL_ITEMS = 4;
constexpr int SEL_BINS = 4096;
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
  __shared__ uint32_t warp_tot[SEL_NT / 32];
  __shared__ uint32_t s_bin, s_remaining, s_eq_total;
  __shared__ unsigned long long s_carry;
  __shared__ unsigned long long wsum[SEL_NT / 32];

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

  // ---- radix select: n-th largest key -----------------------------------------------------
  uint32_t prefix = 0, mask = 0, remaining = (uint32_t)n;
#pragma unroll 1
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 20 : pass == 1 ? 8 : 0;
    const uint32_t dmask = pass == 2 ? 255u : 4095u;
    const int n_bins = (int)dmask + 1;
    if (pass > 0) {
      for (int i = tid; i < n_bins; i += SEL_NT) hist[i] = 0;
      __syncthreads();
      for (int i = tid; i < L; i += SEL_NT) {
        const uint32_t k = key_at(i);
        if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & dmask], 1u);
      }
    }
    __syncthreads();
    // suffix sums over the bins, descending: thread t owns bins n_bins-1-4t .. n_bins-4-4t
    const int per = n_bins / SEL_NT;                     // 4, or 0 for the 256-bin pass (then one bin for tid < 256)
    uint32_t h[4] = {0, 0, 0, 0}, mine = 0;
    if (per == 4) {
#pragma unroll
      for (int j = 0; j < 4; ++j) { h[j] = hist[n_bins - 1 - 4 * tid - j]; mine += h[j]; }
    } else if (tid < n_bins) {
      h[0] = hist[n_bins - 1 - tid];
      mine = h[0];
    }
    uint32_t incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {                                     // exclusive prefix over the 32 warp totals
      const uint32_t t = warp_tot[lane];
      uint32_t in2 = t;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, in2, d);
        if (lane >= d) in2 += y;
      }
      warp_tot[lane] = in2 - t;
    }
    __syncthreads();
    uint32_t acc = incl - mine + warp_tot[warp];         // keys with a digit above this thread's first bin
    const int first_bin = per == 4 ? n_bins - 1 - 4 * tid : n_bins - 1 - tid;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (acc < remaining && acc + h[j] >= remaining) {  // exactly one bin over all threads crosses
        s_bin = (uint32_t)(first_bin - j);
        s_remaining = remaining - acc;
        s_eq_total = h[j];
      }
      acc += h[j];
    }
    __syncthreads();
    prefix |= s_bin << shift;
    mask |= dmask << shift;
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
      uint32_t key = (i < L) ? key_at(i) : 0u;
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
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    if (warp == 0) {                                     // exclusive prefix over the 32 warp totals
      const unsigned long long t = wsum[lane];
      unsigned long long in2 = t;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned long long y = __shfl_up_sync(0xffffffffu, in2, d);
        if (lane >= d) in2 += y;
      }
      wsum[lane] = in2 - t;
    }
    __syncthreads();
    unsigned long long before = s_carry + wsum[warp] + (incl - mine);
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
  if (cudaFuncSetAttribute(actkv::select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)actkv::SEL_SMEM) != cudaSuccess)
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
