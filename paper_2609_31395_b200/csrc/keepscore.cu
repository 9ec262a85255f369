// actkv_keepscore: attention-aware LRFU keep-score (Section 5.1 equation; Algorithm 1 steps 2-4) and
// actkv_gather_f32 (the keep-scores of the survivors move with them, Algorithm 1 step 5 returns KS').
//
// Per (layer x KV head, request) unit, one CTA:
//   1. mass m_i = floor(clip(score_i, 0, 256) * 2^32) as 64-bit integers; total = sum m_i (exact,
//      read off the first histogram);
//   2. mark = ceil(p_q * total / 10000); a radix search (digits of 12, 12 and 8 bits) over the
//      order-preserving image of the scores, kept in shared memory, with 64-bit integer mass histograms
//      finds the threshold score T with mass(score > T) < mark <= mass(score >= T) — exact, independent of
//      summation order;
//   3. entries above T are hits; of the entries equal to T the first ceil((mark - mass_above)/m_T)
//      by index are hits (ordered sweep with a block scan, as in select);
//   4. KS = lambda*KS + score*[hit], one float32 rounding per operation; the score buffer is
//      overwritten with the ranking key: KS, or +inf for the protected prefix.
#include "select_core.cuh"

namespace actkv {

constexpr int KS_NT = 1024;
constexpr int KS_ITEMS = 4;

__device__ __forceinline__ uint32_t ks_order_key(float x) {
  uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ unsigned long long ks_mass(float x) {
  const float c = fminf(fmaxf(x, 0.f), 256.f);
  return __float2ull_rz(c * 4294967296.f);               // exact: a power-of-two scaling, then truncation
}

// IEEE single-precision product and sum, one rounding each, subnormals kept whatever the build's
// flush-to-zero setting is (the recurrence decays towards them).
__device__ __forceinline__ float mul_ieee(float a, float b) {
  float d;
  asm("mul.rn.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}
__device__ __forceinline__ float add_ieee(float a, float b) {
  float d;
  asm("add.rn.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}

__device__ __forceinline__ float ks_key_to_float(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

constexpr int KS_BINS = 4096;
constexpr size_t KS_SMEM = 232448 - 1024;                              // (nearly) all of an SM's shared memory
constexpr int KS_CAP = (int)((KS_SMEM - KS_BINS * 12) / 4);            // keys that fit beside the histogram
// (chunk sums stay below 2^32 for units of up to 2^17 entries; the total mass needs 2^16 or fewer, see below)

// What the fused form needs of actkv_select's arguments.
struct FusedSelectArgs {
  const int32_t* budget;
  const int32_t* keep_indptr;
  int32_t* sel_idx;
  int64_t sel_stride;
  uint32_t* keep_mask;
  actkv_tie_t* tie;
  int32_t* status;
};

// FUSED: the ranking keys go straight into TopK (the second half of select_kernel, on the keys in shared memory)
// instead of back to the score array: one read of the scores, one launch.  Every unit must fit in shared memory.
template <bool FUSED>
__global__ void __launch_bounds__(KS_NT, 1) keepscore_kernel(
    float* __restrict__ score, const int32_t* __restrict__ tok_indptr, int32_t sum_tok, int32_t n_req,
    int32_t p_q, float lambda, const int32_t* __restrict__ n_protect, float* __restrict__ keep_score,
    uint32_t* __restrict__ hit_mask, FusedSelectArgs fs) {
  static_assert(KS_NT == SEL_NT && KS_BINS == SEL_BINS, "the fused form runs select's second half in this CTA");
  // A mass is below 2^41; its three 14-bit chunks are summed in three 32-bit histograms (native shared
  // atomics; a 64-bit shared atomic is a compare-and-swap loop) and put together when the bins are scanned.
  extern __shared__ __align__(16) uint32_t ks_smem[];
  uint32_t* hist = ks_smem;                                            // [3][KS_BINS] mass chunks per digit
  uint32_t* skeys = ks_smem + 3 * KS_BINS;                             // [KS_CAP] order keys of the unit
  auto hist_add = [&](uint32_t bin, unsigned long long m) {
    atomicAdd(&hist[bin], (uint32_t)(m & 0x3fffull));
    atomicAdd(&hist[KS_BINS + bin], (uint32_t)((m >> 14) & 0x3fffull));
    atomicAdd(&hist[2 * KS_BINS + bin], (uint32_t)(m >> 28));
  };
  auto hist_get = [&](int bin) -> unsigned long long {
    return (unsigned long long)hist[bin] + ((unsigned long long)hist[KS_BINS + bin] << 14) +
           ((unsigned long long)hist[2 * KS_BINS + bin] << 28);
  };
  __shared__ unsigned long long warp_tot[KS_NT / 32];
  __shared__ unsigned long long s_above, s_carry;
  __shared__ uint32_t s_bin;

  const int u = blockIdx.x;
  const int r = u % n_req, o = u / n_req;
  const int base = tok_indptr[r];
  const int L = tok_indptr[r + 1] - base;
  int n_keep = 0;
  if (FUSED) {
    n_keep = min(max(fs.budget[r], 0), L);
    // as actkv_select: nothing after an earlier error of the step, and no store past the index buffer
    if (status_set(fs.status)) return;
    if ((int64_t)fs.keep_indptr[r] + n_keep > fs.sel_stride) {
      if (threadIdx.x == 0) report(fs.status, ACTKV_E_INVALID, r, n_keep);
      return;
    }
    if (n_keep == 0 && fs.tie != nullptr && threadIdx.x == 0) fs.tie[u] = actkv_tie_t{0.f, 0, 0, 0};
  }
  if (L <= 0) return;
  float* sc = score + (int64_t)o * sum_tok + base;
  float* ks = keep_score + (int64_t)o * sum_tok + base;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool resident = L <= KS_CAP;                     // uniform over the CTA
  auto key_at = [&](int i) -> uint32_t { return resident ? skeys[i] : ks_order_key(sc[i]); };

  // ---- radix search: largest key T with mass(key >= T) >= mark; digits of 12, 12 and 8 bits ----
  // The scores are read once (kept in shared memory as order keys; longer units re-read them from L2) and
  // that read also fills the histogram of the first digit, whose bins add up to the total mass, from
  // which  mark = ceil(p_q * total / 10000)  (total < 2^57 for up to 2^16 entries, p_q <= 10000 < 2^14: the
  // product is taken in two halves to stay inside 64 bits).
  for (int i = tid; i < 3 * KS_BINS; i += KS_NT) hist[i] = 0u;
  __syncthreads();
  for (int i = tid; i < L; i += KS_NT) {
    const float x = sc[i];
    const uint32_t k = ks_order_key(x);
    if (resident) skeys[i] = k;
    const unsigned long long m = ks_mass(x);
    if (m != 0ull) hist_add(k >> 20, m);
  }
  uint32_t prefix = 0, mask = 0;
  unsigned long long above = 0;        // mass of keys strictly above the current prefix range
  unsigned long long mark = 0;
#pragma unroll 1
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 20 : pass == 1 ? 8 : 0;
    const uint32_t dmask = pass == 2 ? 255u : 4095u;
    const int n_bins = (int)dmask + 1;
    if (pass > 0) {
      for (int i = tid; i < 3 * KS_BINS; i += KS_NT) hist[i] = 0u;
      __syncthreads();
      for (int i = tid; i < L; i += KS_NT) {
        const uint32_t k = key_at(i);
        if ((k & mask) == prefix) {
          const unsigned long long m = ks_mass(ks_key_to_float(k));
          if (m != 0ull) hist_add((k >> shift) & dmask, m);
        }
      }
    }
    __syncthreads();
    // suffix sums over the bins, descending: thread t owns bins n_bins-1-4t .. n_bins-4-4t
    const int per = n_bins / KS_NT;                      // 4, or 0 for the 256-bin pass (then one bin for tid < 256)
    unsigned long long h[4] = {0ull, 0ull, 0ull, 0ull}, mine = 0ull;
    if (per == 4) {
#pragma unroll
      for (int j = 0; j < 4; ++j) { h[j] = hist_get(n_bins - 1 - 4 * tid - j); mine += h[j]; }
    } else if (tid < n_bins) {
      h[0] = hist_get(n_bins - 1 - tid);
      mine = h[0];
    }
    unsigned long long incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    unsigned long long acc = above + incl - mine;        // mass above this thread's first bin
    unsigned long long total = 0ull;
    for (int w = 0; w < KS_NT / 32; ++w) {
      const unsigned long long t = warp_tot[w];
      if (w < warp) acc += t;
      total += t;
    }
    if (pass == 0) {
      const unsigned long long q = total / 10000ull, rem = total % 10000ull;
      mark = q * (unsigned long long)p_q + (rem * (unsigned long long)p_q + 9999ull) / 10000ull;
    }
    if (mark == 0ull) break;                             // nothing to cover: no hits (uniform over the CTA)
    const int first_bin = per == 4 ? n_bins - 1 - 4 * tid : n_bins - 1 - tid;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (acc < mark && acc + h[j] >= mark) {            // exactly one bin over all threads crosses the mark
        s_bin = (uint32_t)(first_bin - j);
        s_above = acc;
      }
      acc += h[j];
    }
    __syncthreads();
    prefix |= s_bin << shift;
    mask |= dmask << shift;
    above = s_above;
    __syncthreads();
  }
  uint32_t thr = 0;                    // key of the last hit
  uint32_t ties_hit = 0;               // how many of the entries equal to thr are hits (lowest indices)
  if (mark > 0) {
    thr = prefix;
    // all entries with key == thr share one score, hence one mass (> 0: the bin crossed the mark)
    const float tv = __uint_as_float((thr & 0x80000000u) ? (thr & 0x7fffffffu) : ~thr);
    const unsigned long long thr_mass = ks_mass(tv);
    const unsigned long long need_at_thr = mark - above;   // > 0 by construction
    ties_hit = thr_mass > 0 ? (uint32_t)((need_at_thr + thr_mass - 1) / thr_mass) : 0u;
  }

  // ---- ordered sweep: hits, keep-score update, ranking keys ----
  if (FUSED) {                                           // the mass histograms are done with: first-digit counts of the ranking keys
    __syncthreads();
    for (int i = tid; i < KS_BINS; i += KS_NT) hist[i] = 0u;
  }
  if (tid == 0) s_carry = 0ull;
  __syncthreads();
  const int np = n_protect ? n_protect[r] : 0;
  uint32_t* mrow = hit_mask ? hit_mask + (int64_t)o * ((sum_tok + 31) / 32) : nullptr;
  for (int c0 = 0; c0 < L; c0 += KS_NT * KS_ITEMS) {
    const int i0 = c0 + tid * KS_ITEMS;
    float x[KS_ITEMS];
    uint32_t eq[KS_ITEMS], gt[KS_ITEMS];
    uint32_t n_eq = 0;
#pragma unroll
    for (int k = 0; k < KS_ITEMS; ++k) {
      const int i = i0 + k;
      x[k] = (i < L) ? sc[i] : 0.f;
      const uint32_t key = ks_order_key(x[k]);
      gt[k] = (i < L) && mark > 0 && key > thr;
      eq[k] = (i < L) && mark > 0 && key == thr;
      n_eq += eq[k];
    }
    // exclusive scan of the tie counts in index order
    uint32_t incl = n_eq;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += t;
    }
    __shared__ uint32_t wsum[KS_NT / 32];
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    uint32_t before = (uint32_t)s_carry;
    for (int w = 0; w < warp; ++w) before += wsum[w];
    before += incl - n_eq;
#pragma unroll
    for (int k = 0; k < KS_ITEMS; ++k) {
      const int i = i0 + k;
      if (i < L) {
        const bool hit = gt[k] || (eq[k] && before < ties_hit);
        const float decayed = mul_ieee(lambda, ks[i]);
        const float nk = hit ? add_ieee(decayed, x[k]) : decayed;
        ks[i] = nk;
        const float rank = (i < np) ? INFINITY : nk;          // what TopK ranks
        if (FUSED) {
          const uint32_t rk = ks_order_key(rank);
          skeys[i] = rk;
          atomicAdd(&hist[rk >> 20], 1u);
        } else {
          sc[i] = rank;
        }
        if (hit && mrow) atomicOr(&mrow[(base + i) >> 5], 1u << ((base + i) & 31));
      }
      before += eq[k];
    }
    __syncthreads();
    if (tid == KS_NT - 1) s_carry = before;
    __syncthreads();
  }
  if (FUSED && n_keep > 0) {                             // uniform over the CTA
    auto rank_key_at = [&](int i) -> uint32_t { return skeys[i]; };
    select_threshold_and_emit(rank_key_at, hist, L, n_keep, fs.sel_idx + (int64_t)o * fs.sel_stride + fs.keep_indptr[r],
                              fs.keep_mask ? fs.keep_mask + (int64_t)o * ((sum_tok + 31) / 32) : nullptr, base, fs.tie, u);
  }
}

__global__ void gather_f32_kernel(const float* __restrict__ src, int64_t src_stride, const int32_t* __restrict__ tok_indptr,
                                  const int32_t* __restrict__ sel_idx, int64_t sel_stride,
                                  const int32_t* __restrict__ keep_indptr, int32_t n_req, float* __restrict__ dst,
                                  int64_t dst_stride) {
  const int o = blockIdx.y;
  const int total = keep_indptr[n_req];
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    int lo = 0, hi = n_req;                                    // request of survivor slot i
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (keep_indptr[mid] <= i) lo = mid; else hi = mid;
    }
    const int tok = sel_idx[(int64_t)o * sel_stride + i];
    dst[(int64_t)o * dst_stride + i] = src[(int64_t)o * src_stride + tok_indptr[lo] + tok];
  }
}

}  // namespace actkv

extern "C" {

int actkv_keepscore(float* score, const int32_t* tok_indptr, int32_t sum_tok, int32_t n_outer, int32_t n_req,
                    float top_p, float lambda, const int32_t* n_protect, float* keep_score, uint32_t* hit_mask,
                    int32_t* status, actkv_stream_t stream) {
  (void)status;
  if (n_outer < 0 || n_req < 0 || sum_tok < 0) return ACTKV_E_INVALID;
  if (!(top_p >= 0.f && top_p <= 1.f) || !(lambda >= 0.f && lambda <= 1.f)) return ACTKV_E_INVALID;
  if (n_outer == 0 || n_req == 0 || sum_tok == 0) return ACTKV_OK;
  if (!score || !tok_indptr || !keep_score) return ACTKV_E_INVALID;
  const int64_t units = (int64_t)n_outer * n_req;
  if (units > 0x7fffffffLL) return ACTKV_E_INVALID;
  const int32_t p_q = (int32_t)lrintf(top_p * 10000.f);
  if (actkv::ensure_dyn_smem(actkv::keepscore_kernel<false>, actkv::KS_SMEM) != cudaSuccess)
    return ACTKV_E_CUDA;
  actkv::keepscore_kernel<false><<<(unsigned)units, actkv::KS_NT, actkv::KS_SMEM, (cudaStream_t)stream>>>(
      score, tok_indptr, sum_tok, n_req, p_q, lambda, n_protect, keep_score, hit_mask, actkv::FusedSelectArgs{});
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

int actkv_keepscore_select(float* score, const int32_t* tok_indptr, int32_t sum_tok, int32_t max_tok, int32_t n_outer,
                           int32_t n_req, float top_p, float lambda, const int32_t* n_protect, float* keep_score,
                           uint32_t* hit_mask, const int32_t* budget, const int32_t* keep_indptr, int32_t* sel_idx,
                           int64_t sel_stride, uint32_t* keep_mask, actkv_tie_t* tie_report, int32_t* status,
                           actkv_stream_t stream) {
  if (n_outer < 0 || n_req < 0 || sum_tok < 0 || max_tok < 0 || sel_stride < 0) return ACTKV_E_INVALID;
  if (!(top_p >= 0.f && top_p <= 1.f) || !(lambda >= 0.f && lambda <= 1.f)) return ACTKV_E_INVALID;
  if (n_outer == 0 || n_req == 0 || sum_tok == 0) return ACTKV_OK;
  if (!score || !tok_indptr || !keep_score || !budget || !keep_indptr || !sel_idx) return ACTKV_E_INVALID;
  if (max_tok > actkv::KS_CAP) {
    // a unit that does not fit in shared memory: the two stages as two kernels (the ranking keys go through `score`)
    int rc = actkv_keepscore(score, tok_indptr, sum_tok, n_outer, n_req, top_p, lambda, n_protect, keep_score, hit_mask,
                             status, stream);
    if (rc != ACTKV_OK) return rc;
    return actkv_select(score, tok_indptr, sum_tok, budget, n_outer, n_req, keep_indptr, sel_idx, sel_stride, keep_mask,
                        tie_report, nullptr, 0, status, stream);
  }
  const int64_t units = (int64_t)n_outer * n_req;
  if (units > 0x7fffffffLL) return ACTKV_E_INVALID;
  const int32_t p_q = (int32_t)lrintf(top_p * 10000.f);
  if (actkv::ensure_dyn_smem(actkv::keepscore_kernel<true>, actkv::KS_SMEM) != cudaSuccess)
    return ACTKV_E_CUDA;
  actkv::FusedSelectArgs fs{budget, keep_indptr, sel_idx, sel_stride, keep_mask, tie_report, status};
  actkv::keepscore_kernel<true><<<(unsigned)units, actkv::KS_NT, actkv::KS_SMEM, (cudaStream_t)stream>>>(
      score, tok_indptr, sum_tok, n_req, p_q, lambda, n_protect, keep_score, hit_mask, fs);
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

int actkv_gather_f32(const float* src, int64_t src_stride, const int32_t* tok_indptr, const int32_t* sel_idx,
                     int64_t sel_stride, const int32_t* keep_indptr, int32_t n_outer, int32_t n_req,
                     int32_t max_total_keep, float* dst, int64_t dst_stride, actkv_stream_t stream) {
  if (n_outer < 0 || n_req < 0 || max_total_keep < 0) return ACTKV_E_INVALID;
  if (n_outer == 0 || n_req == 0 || max_total_keep == 0) return ACTKV_OK;
  if (!src || !tok_indptr || !sel_idx || !keep_indptr || !dst || n_outer > 65535) return ACTKV_E_INVALID;
  dim3 grid((unsigned)((max_total_keep + 255) / 256), (unsigned)n_outer);
  if (grid.x > 1024) grid.x = 1024;
  actkv::gather_f32_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(src, src_stride, tok_indptr, sel_idx, sel_stride,
                                                                   keep_indptr, n_req, dst, dst_stride);
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

}  // extern "C"
