// actkv_keepscore: attention-aware LRFU keep-score (Section 5.1 equation; Algorithm 1 steps 2-4) and
// actkv_gather_f32 (the keep-scores of the survivors move with them, Algorithm 1 step 5 returns KS').
//
// Per (layer x KV head, request) unit, one CTA:
//   1. mass m_i = floor(clip(score_i, 0, 256) * 2^32) as 64-bit integers; total = sum m_i (exact,
//      read off the first histogram);
//   2. mark = ceil(p_q * total / 10000); a 4 x 8-bit radix search over the order-preserving image of
//      the scores with 64-bit integer mass histograms (warp-aggregated adds) finds the threshold
//      score T with mass(score > T) < mark <= mass(score >= T) — exact, independent of summation order;
//   3. entries above T are hits; of the entries equal to T the first ceil((mark - mass_above)/m_T)
//      by index are hits (ordered sweep with a block scan, as in select);
//   4. KS = lambda*KS + score*[hit], one float32 rounding per operation; the score buffer is
//      overwritten with the ranking key: KS, or +inf for the protected prefix.
#include "common.cuh"

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

__global__ void __launch_bounds__(KS_NT) keepscore_kernel(
    float* __restrict__ score, const int32_t* __restrict__ tok_indptr, int32_t sum_tok, int32_t n_req,
    int32_t p_q, float lambda, const int32_t* __restrict__ n_protect, float* __restrict__ keep_score,
    uint32_t* __restrict__ hit_mask) {
  __shared__ unsigned long long hist[256];
  __shared__ unsigned long long s_above, s_carry, s_mark;
  __shared__ uint32_t s_bin;

  const int u = blockIdx.x;
  const int r = u % n_req, o = u / n_req;
  const int base = tok_indptr[r];
  const int L = tok_indptr[r + 1] - base;
  if (L <= 0) return;
  float* sc = score + (int64_t)o * sum_tok + base;
  float* ks = keep_score + (int64_t)o * sum_tok + base;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // ---- radix search: largest key T with mass(key >= T) >= mark ----
  // The first pass histograms every entry, so its bins also add up to the total mass, from which
  // mark = ceil(p_q * total / 10000)  (total < 2^57 for up to 2^16 entries, p_q <= 10000 < 2^14:
  // the product is taken in two halves to stay inside 64 bits).
  uint32_t prefix = 0, mask = 0;
  unsigned long long above = 0;        // mass of keys strictly above the current prefix range
  unsigned long long mark = 0;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int i0 = 0; i0 < L; i0 += KS_NT) {                // warp-uniform trip count
      const int i = i0 + tid;
      const float x = (i < L) ? sc[i] : 0.f;
      const uint32_t k = ks_order_key(x);
      const unsigned long long m = ks_mass(x);
      const bool in = (i < L) && (k & mask) == prefix && m != 0ull;
      const uint32_t voters = __ballot_sync(0xffffffffu, in);
      if (in) {
        // warp-aggregated add: lanes with the same bin sum their masses (<= 2^40 each, as two
        // chunks that cannot overflow 32 bits over 32 lanes) and elect one lane to add the sum
        const uint32_t bin = (k >> shift) & 255u;
        const uint32_t peers = __match_any_sync(voters, bin);
        const uint32_t lo = __reduce_add_sync(peers, (uint32_t)(m & 0x1fffffull));
        const uint32_t hi = __reduce_add_sync(peers, (uint32_t)(m >> 21));
        if (lane == (__ffs(peers) - 1)) atomicAdd(&hist[bin], ((unsigned long long)hi << 21) + lo);
      }
    }
    __syncthreads();
    // warp 0: suffix sums over the 256 bins, lane l owns bins 255-8l .. 248-8l (descending)
    if (warp == 0) {
      unsigned long long h[8], mine = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        h[j] = hist[255 - 8 * lane - j];
        mine += h[j];
      }
      unsigned long long incl = mine;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += t;
      }
      if (shift == 24) {
        const unsigned long long total = __shfl_sync(0xffffffffu, incl, 31);
        const unsigned long long q = total / 10000ull, rem = total % 10000ull;
        mark = q * (unsigned long long)p_q + (rem * (unsigned long long)p_q + 9999ull) / 10000ull;
        if (lane == 0) s_mark = mark;
      }
      if (mark > 0) {
        unsigned long long acc = above + incl - mine;      // mass above this lane's first bin
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (acc < mark && acc + h[j] >= mark) {          // exactly one bin over all lanes crosses the mark
            s_bin = 255u - 8u * lane - j;
            s_above = acc;
          }
          acc += h[j];
        }
      }
    }
    __syncthreads();
    mark = s_mark;
    if (mark == 0) break;                                  // nothing to cover: no hits (uniform over the CTA)
    prefix |= s_bin << shift;
    mask |= 255u << shift;
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
        sc[i] = (i < np) ? INFINITY : nk;                     // what TopK ranks
        if (hit && mrow) atomicOr(&mrow[(base + i) >> 5], 1u << ((base + i) & 31));
      }
      before += eq[k];
    }
    __syncthreads();
    if (tid == KS_NT - 1) s_carry = before;
    __syncthreads();
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
  actkv::keepscore_kernel<<<(unsigned)units, actkv::KS_NT, 0, (cudaStream_t)stream>>>(
      score, tok_indptr, sum_tok, n_req, p_q, lambda, n_protect, keep_score, hit_mask);
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
