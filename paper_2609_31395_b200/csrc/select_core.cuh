// The second half of TopK(score, k = B) for one unit held by one CTA of SEL_NT threads (Algorithm 1 step 5):
// given the unit's order-preserving 32-bit keys (key_at(i), i < L) and the histogram of their first 12-bit digit
// in hist[0 .. SEL_BINS), a most-significant-digit radix select (digits of 12, 12 and 8 bits) finds the n-th
// largest key exactly, and one ordered sweep with a block scan emits the kept token indices in ascending order,
// entries equal to the threshold being kept lowest index first.  Shared by actkv_select and the fused
// keep-score + select kernel.
#pragma once

#include "common.cuh"

namespace actkv {

constexpr int SEL_NT = 1024;
constexpr int SEL_ITEMS = 4;
constexpr int SEL_BINS = 4096;

template <class KeyAt>
__device__ __forceinline__ void select_threshold_and_emit(KeyAt key_at, uint32_t* hist, int L, int n, int32_t* out,
                                                          uint32_t* mask_row, int base, actkv_tie_t* tie, int u) {
  __shared__ uint32_t warp_tot[SEL_NT / 32];
  __shared__ uint32_t s_bin, s_remaining, s_eq_total;
  __shared__ unsigned long long s_carry;
  __shared__ unsigned long long wsum[SEL_NT / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
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

}  // namespace actkv
