// FMA path of actkv_score: any head_dim (multiple of 8, <= 256), any page size and strides,
// any window.  It is the path for small windows (window x group rows < 64, where a tensor-core
// tile would be mostly padding) and for pool layouts the tensor-core path does not take.
//
// Section 7.1 / Algorithm 3: s = q.k, A = exp(s - LSE), max over the GQA group, mean over the
// action tokens.  Logits are kept in log2 units (t = s * sm_scale * log2 e) so that exp2 maps to
// one MUFU op.
#pragma once

#include "common.cuh"

namespace actkv {

constexpr int FMA_TK = 64;        // keys per tile
constexpr int FMA_RQ = 32;        // window x group rows per chunk (at most)
constexpr int FMA_NT = 256;       // threads per CTA
constexpr int LSE_CHUNK = 512;    // fewest keys per partial (m, sum) of the LSE pass (both paths)
constexpr int LSE_CHUNK_LONG = 4096;  // fewest keys per partial while the launch still has LSE_ITEMS_MIN work items
constexpr int LSE_ITEMS = 20 * 148;  // work items an LSE launch aims for: 20 per SM
constexpr int LSE_ITEMS_MIN = 4 * 148;

struct ScoreArgs {
  PoolView pool;
  TablesView tab;
  const __nv_bfloat16* q;        // [NLs, sum_win, Hq, D]
  const int32_t* win_indptr;
  const int32_t* tok_indptr;
  const float* lse;              // [NLs, sum_win, Hq] natural log (pass 2 input)
  float2* partials;              // [units, n_chunks, rows_max] (pass 1 output), log2 units
  float* score_out;              // [NLs, Hkv, sum_tok]
  int32_t* status;
  int32_t layer_begin, n_layers_sub, n_q_heads, group;
  int32_t sum_win, sum_tok, rows_max, n_chunks, n_tiles;
  int32_t lse_chunk;             // keys per LSE partial of this launch (multiple of 128, >= LSE_CHUNK)
  float scale_log2;              // sm_scale * log2(e)
  int32_t causal;
  int32_t win_left;              // sliding-window layer: a query at position p sees keys p - win_left < j <= p (0: all)
  const int32_t* acc_steps;      // accumulate mode (streaming, Algorithm 3 step 5): [R] action queries already
                                 // folded into score_out; nullptr: score_out is overwritten with this call's mean
};

// What is stored for one key: the mean over this call's W action tokens (`mean_w`), or in accumulate
// mode the running mean over the n earlier action tokens of the region and this call's W
// (n = 0: the old value is not read, the state restarts).
__device__ __forceinline__ void store_pooled(const ScoreArgs& a, int r, float* slot, float sum_w, float mean_w, int W) {
  if (a.acc_steps != nullptr) {
    const int n = a.acc_steps[r];
    if (n > 0) mean_w = fmaf(*slot, (float)n, sum_w) / (float)(n + W);
  }
  *slot = mean_w;
}

__device__ __forceinline__ float2 bf16x2_to_float2(uint32_t v) {
  return make_float2(__uint_as_float(v << 16), __uint_as_float(v & 0xffff0000u));
}

// Copies `n_rows` rows of D bf16 (row r at src + r*src_stride... given by a functor) into padded
// shared rows of (D/2 + 1) 32-bit words.
template <class RowPtr>
__device__ __forceinline__ void load_rows_padded(uint32_t* dst, int n_rows, int D, RowPtr row_ptr) {
  const int vec_per_row = D / 8;
  const int wstride = D / 2 + 1;
  for (int i = threadIdx.x; i < n_rows * vec_per_row; i += blockDim.x) {
    int r = i / vec_per_row, v = i - r * vec_per_row;
    const __nv_bfloat16* src = row_ptr(r);
    uint4 x = make_uint4(0, 0, 0, 0);
    if (src != nullptr) x = __ldg(reinterpret_cast<const uint4*>(src) + v);
    uint32_t* d = dst + r * wstride + v * 4;
    d[0] = x.x; d[1] = x.y; d[2] = x.z; d[3] = x.w;
  }
}

// One kernel for both passes.  PASS 1: partial (max, sum) of exp2 over a chunk of lse_chunk keys
// for every window row.  PASS 2: pooled score of a tile of FMA_TK keys.
template <int PASS>
__global__ void __launch_bounds__(FMA_NT) score_fma_kernel(const ScoreArgs a) {
  extern __shared__ __align__(16) uint32_t smem[];
  const int D = a.pool.head_dim;
  const int wstride = D / 2 + 1;
  const int R = a.tab.n_req, Hkv = a.pool.n_kv_heads, G = a.group;
  const int per_unit = (PASS == 1) ? a.n_chunks : a.n_tiles;
  const int u = blockIdx.x / per_unit;                 // (slab * Hkv + h) * R + r
  const int part = blockIdx.x - u * per_unit;
  const int r = u % R, h = (u / R) % Hkv, slab = u / (R * Hkv);
  const int L = a.tab.seq_len[r];
  const int w0 = a.win_indptr[r], W = a.win_indptr[r + 1] - w0;
  const int key_begin = part * ((PASS == 1) ? a.lse_chunk : FMA_TK);
  if (key_begin >= L) return;
  if (W <= 0 && a.acc_steps != nullptr) return;      // accumulate mode: a request outside its action region
  if (W <= 0 || (a.causal && W > L)) {               // no window, or a window longer than the cache
    if (threadIdx.x == 0 && part == 0) report(a.status, ACTKV_E_INVALID, r, W);
    return;
  }
  const int key_end = min(L, key_begin + ((PASS == 1) ? a.lse_chunk : FMA_TK));
  const int rows = W * G;
  const int wpc = FMA_RQ / G;                          // window rows per chunk
  const int n_rc = (W + wpc - 1) / wpc;

  uint32_t* Ks = smem;                                 // [FMA_TK][wstride]
  uint32_t* Qs = Ks + FMA_TK * wstride;                // [FMA_RQ][wstride]
  float* Ps = reinterpret_cast<float*>(Qs + FMA_RQ * wstride);   // PASS 2: [FMA_RQ][FMA_TK+1]
  float* m_s = Ps;                                     // PASS 1: [rows] running max
  float* s_s = Ps + rows;                              // PASS 1: [rows] running sum

  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int layer = a.layer_begin + slab;
  const __nv_bfloat16* kbase = a.pool.base + (int64_t)layer * a.pool.stride_layer + (int64_t)h * a.pool.stride_head;
  const __nv_bfloat16* qbase = a.q + ((int64_t)slab * a.sum_win + w0) * a.n_q_heads * D + (int64_t)h * G * D;
  const float* lse_base = (PASS == 2) ? a.lse + ((int64_t)slab * a.sum_win + w0) * a.n_q_heads + h * G : nullptr;

  if (PASS == 1) {
    for (int i = threadIdx.x; i < rows; i += blockDim.x) { m_s[i] = -INFINITY; s_s[i] = 0.f; }
  }
  float pooled = 0.f;                                  // PASS 2: thread `key` accumulates sum_w max_g

  for (int t0 = key_begin; t0 < key_end; t0 += FMA_TK) {
    __syncthreads();
    const int P = a.pool.page_size;
    load_rows_padded(Ks, FMA_TK, D, [&](int k) -> const __nv_bfloat16* {
      int j = t0 + k;
      if (j >= L) return nullptr;
      int page = checked_page(a.tab, a.pool.n_pages, r, j / P, a.status);
      return kbase + (int64_t)page * a.pool.stride_page + (int64_t)(j % P) * a.pool.stride_slot;
    });
    for (int rc = 0; rc < n_rc; ++rc) {
      const int wc0 = rc * wpc;
      const int n_w = min(wpc, W - wc0);
      const int n_rows = n_w * G;
      __syncthreads();                                 // Ks ready / previous chunk's Qs and Ps consumed
      load_rows_padded(Qs, FMA_RQ, D, [&](int rl) -> const __nv_bfloat16* {
        if (rl >= n_rows) return nullptr;
        int w = wc0 + rl / G, g = rl % G;
        return qbase + ((int64_t)w * a.n_q_heads + g) * D;
      });
      __syncthreads();
      float acc[2][4];
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int k = 0; k < 4; ++k) acc[i][k] = 0.f;
      const uint32_t* q0 = Qs + ty * wstride;
      const uint32_t* q1 = Qs + (ty + 16) * wstride;
      const uint32_t* k0 = Ks + tx * wstride;
      for (int d2 = 0; d2 < D / 2; ++d2) {
        float2 qa = bf16x2_to_float2(q0[d2]), qb = bf16x2_to_float2(q1[d2]);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          float2 kk = bf16x2_to_float2(k0[k * 16 * wstride + d2]);
          acc[0][k] = fmaf(qa.x, kk.x, fmaf(qa.y, kk.y, acc[0][k]));
          acc[1][k] = fmaf(qb.x, kk.x, fmaf(qb.y, kk.y, acc[1][k]));
        }
      }
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int rl = ty + 16 * i;
        const bool row_ok = rl < n_rows;
        const int w = wc0 + rl / G;
        const int row = w * G + rl % G;
        const int last_visible = a.causal ? (L - W + w) : (L - 1);
        float t[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          int j = t0 + tx + 16 * k;
          bool vis = row_ok && j < L && j <= last_visible && (a.win_left <= 0 || j > last_visible - a.win_left);
          t[k] = vis ? acc[i][k] * a.scale_log2 : -INFINITY;
        }
        if (PASS == 1) {
          float mx = fmaxf(fmaxf(t[0], t[1]), fmaxf(t[2], t[3]));
#pragma unroll
          for (int o = 8; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
          float m_old = row_ok ? m_s[row] : -INFINITY;
          float m_new = fmaxf(m_old, mx);
          float sum = 0.f;
          if (m_new > -INFINITY) {
#pragma unroll
            for (int k = 0; k < 4; ++k) sum += exp2f(t[k] - m_new);
          }
#pragma unroll
          for (int o = 8; o >= 1; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
          if (row_ok && tx == 0 && m_new > -INFINITY) {
            s_s[row] = s_s[row] * exp2f(m_old - m_new) + sum;
            m_s[row] = m_new;
          }
        } else {
          const float l2 = row_ok ? lse_base[(int64_t)w * a.n_q_heads + rl % G] * kLog2e : 0.f;
#pragma unroll
          for (int k = 0; k < 4; ++k)
            Ps[rl * (FMA_TK + 1) + tx + 16 * k] = (t[k] > -INFINITY) ? exp2f(t[k] - l2) : 0.f;
        }
      }
      if (PASS == 2) {
        __syncthreads();
        if (threadIdx.x < FMA_TK) {
          for (int wl = 0; wl < n_w; ++wl) {
            float mx = 0.f;
            for (int g = 0; g < G; ++g) mx = fmaxf(mx, Ps[(wl * G + g) * (FMA_TK + 1) + threadIdx.x]);
            pooled += mx;
          }
        }
      }
    }
  }
  if (PASS == 1) {
    __syncthreads();
    float2* out = a.partials + ((int64_t)u * a.n_chunks + part) * a.rows_max;
    for (int i = threadIdx.x; i < rows; i += blockDim.x) out[i] = make_float2(m_s[i], s_s[i]);
  } else {
    const int j = key_begin + threadIdx.x;
    if (threadIdx.x < FMA_TK && j < L) {
      store_pooled(a, r, a.score_out + ((int64_t)slab * Hkv + h) * a.sum_tok + a.tok_indptr[r] + j, pooled,
                   pooled / (float)W, W);
    }
  }
}

inline size_t score_fma_smem_bytes(int D, int rows_max, int pass) {
  size_t w = (size_t)(FMA_TK + FMA_RQ) * (D / 2 + 1) * 4;
  size_t tail = pass == 1 ? (size_t)rows_max * 8 : (size_t)FMA_RQ * (FMA_TK + 1) * 4;
  return w + tail;
}

// Merges the per-chunk (max, sum) partials of one window row into its LSE (natural log units).
__global__ void lse_combine_kernel(const ScoreArgs a, float* lse_out, float* lse_out2) {
  const int R = a.tab.n_req, Hkv = a.pool.n_kv_heads, G = a.group;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // over units * rows_max
  const int64_t total = (int64_t)a.n_layers_sub * Hkv * R * a.rows_max;
  if (idx >= total) return;
  const int row = (int)(idx % a.rows_max);
  const int u = (int)(idx / a.rows_max);
  const int r = u % R, h = (u / R) % Hkv, slab = u / (R * Hkv);
  const int L = a.tab.seq_len[r];
  const int w0 = a.win_indptr[r], W = a.win_indptr[r + 1] - w0;
  if (row >= W * G || L <= 0) return;
  const int n_chunks = (L + a.lse_chunk - 1) / a.lse_chunk;
  const float2* p = a.partials + (int64_t)u * a.n_chunks * a.rows_max + row;
  float M = -INFINITY;
  for (int c = 0; c < n_chunks; ++c) M = fmaxf(M, p[(int64_t)c * a.rows_max].x);
  float S = 0.f;
  for (int c = 0; c < n_chunks; ++c) {
    float2 v = p[(int64_t)c * a.rows_max];
    if (v.x > -INFINITY) S += v.y * exp2f(v.x - M);
  }
  const float lse = (M + log2f(S)) * kLn2;
  const int w = row / G, g = row % G;
  const int64_t o = ((int64_t)slab * a.sum_win + w0 + w) * a.n_q_heads + h * G + g;
  lse_out[o] = lse;
  if (lse_out2 != nullptr) lse_out2[o] = lse;
}

}  // namespace actkv
