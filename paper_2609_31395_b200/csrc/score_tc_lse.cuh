// LSE pass of the tensor-core score path (Section 7.1, LSE equation):
//   lse[row] = log sum_{key visible} exp(sm_scale * q_row . k_key),   row = (window token w, group head g).
//
// D[row, key] = Q K^T with the rows on the TMEM lanes, so every epilogue thread owns one row and keeps
// its running (max, sum of exp2) in registers: no shuffles.  A CTA covers 256 rows (two 128-row
// blocks) x one chunk of LSE_CHUNK keys.
//
// Operand placement.  With both operands in shared memory the operand fetch (A 4 KB + B 4 KB per
// 128x128x16 MMA) caps the tensor pipe near half rate.  The Q block is the same for every key tile
// of the CTA, so it is written once into tensor memory (tcgen05.st, two bf16 per 32-bit column) and
// used as the A operand from there; only the K tile (B) streams through shared memory.
// TMEM columns: [0,128) the two Q blocks, [128,512) a ring of three 128-column accumulators; a job
// is one (key tile, row block) product.
//
// Exp rate.  One exp2 per (row, key) is more than the 16 MUFU results per clock of an SM can follow,
// so POLY of every 8 column pairs are evaluated on the FMA / ALU pipes instead: 2^x = 2^j p(f),
// j = round(x), f = x - j in [-0.5, 0.5], p a cubic fitted to 2^f (max relative error 7.5e-5, far
// inside the 2e-3 score tolerance), 2^j applied by adding j to the exponent field; two columns at a
// time with the packed fp32x2 instructions.
#pragma once

#include "tc_common.cuh"

namespace actkv {
namespace tc {

constexpr int LSE_POLY_PAIRS_DEFAULT = 2;        // measured best on B200 (0: 9.0 ms, 1: 8.6, 2: 8.4, 3: 8.9 at the bench shape)

__device__ __forceinline__ void exp2_poly2(float& e0, float& e1, float x0, float x1) {
  constexpr float MAGIC = 12582912.f;            // 1.5 * 2^23: x + MAGIC rounds x to the nearest integer
  x0 = fmaxf(x0, -126.f);
  x1 = fmaxf(x1, -126.f);
  float t0 = x0, t1 = x1;
  fadd2(t0, t1, MAGIC, MAGIC);                   // integer part in the low mantissa bits
  float j0 = t0, j1 = t1;
  fadd2(j0, j1, -MAGIC, -MAGIC);
  float f0 = x0, f1 = x1;
  fadd2(f0, f1, -j0, -j1);                       // f = x - round(x)
  float p0, p1;                                  // Horner, both lanes per instruction
  ffma2(p0, p1, f0, f1, 0.0551716648042202f, 0.2426111251115799f, 0.2426111251115799f);
  ffma2v(p0, p1, p0, p1, f0, f1, 0.6932609677314758f, 0.6932609677314758f);
  ffma2v(p0, p1, p0, p1, f0, f1, 0.9999280571937561f, 0.9999280571937561f);
  e0 = __int_as_float(__float_as_int(p0) + (__float_as_int(t0) << 23));
  e1 = __int_as_float(__float_as_int(p1) + (__float_as_int(t1) << 23));
}

// One full group of 32 logits of a row: online max, then sum += sum_i exp2((v_i - m) * c).
template <int POLY>
__device__ __forceinline__ void lse_group(const float* v, float c, float& m, float& sum) {
  float t[11];                                   // max tree: 32 -> 11 -> 4 -> 1
#pragma unroll
  for (int i = 0; i < 10; ++i) t[i] = fmax3(v[3 * i], v[3 * i + 1], v[3 * i + 2]);
  t[10] = fmaxf(v[30], v[31]);
  const float u0 = fmax3(t[0], t[1], t[2]), u1 = fmax3(t[3], t[4], t[5]), u2 = fmax3(t[6], t[7], t[8]);
  const float gm = fmaxf(fmax3(u0, u1, u2), fmaxf(t[9], t[10]));
  if (gm > m) { sum *= exp2f((m - gm) * c); m = gm; }     // m = -inf: sum is 0 and stays 0
  const float nmc = -m * c;
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
  for (int p = 0; p < 16; ++p) {
    float x0, x1, e0, e1;
    ffma2(x0, x1, v[2 * p], v[2 * p + 1], c, nmc, nmc);
    if ((p & 7) < POLY) {
      exp2_poly2(e0, e1, x0, x1);
    } else {
      e0 = exp2f(x0);
      e1 = exp2f(x1);
    }
    if (p & 1) fadd2(s2, s3, e0, e1); else fadd2(s0, s1, e0, e1);
  }
  sum += (s0 + s1) + (s2 + s3);
}

constexpr int LSE_EPI_WARPS = 16;                // (row block, TMEM lane quarter, column half)
constexpr int LSE_THREADS = (2 + LSE_EPI_WARPS) * 32;
constexpr int LSE_SLOTS = 3;                     // accumulator ring
constexpr int LSE_A_COLS = 128;                  // TMEM columns holding the two Q blocks

struct LseBarriers {
  uint64_t k_full[8];
  uint64_t k_empty[8];
  uint64_t q_ready;
  uint64_t tmem_full[LSE_SLOTS];
  uint64_t tmem_empty[LSE_SLOTS];
  uint64_t drained;
  uint32_t tmem_base;
  int abort_flag;
  float2 exch[256];            // (max, sum) of the upper column half, handed to the lower half's thread
};

template <int POLY>
__global__ void __launch_bounds__(LSE_THREADS, 1)
score_tc_lse_kernel(const __grid_constant__ CUtensorMap kmap, const TcArgs ta) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const ScoreArgs& a = ta.a;
  const int R = a.tab.n_req, Hkv = a.pool.n_kv_heads, G = a.group;
  int idx = blockIdx.x;
  const int chunk = idx % a.n_chunks; idx /= a.n_chunks;
  const int rg = idx % ta.n_rg;
  const int u = idx / ta.n_rg;
  const int r = u % R, h = (u / R) % Hkv, slab = u / (R * Hkv);
  const int L = a.tab.seq_len[r];
  const int w0 = a.win_indptr[r], W = a.win_indptr[r + 1] - w0;
  const int rows = W * G;
  const int key_begin = chunk * a.lse_chunk;
  if (key_begin >= L || rg * 256 >= rows) return;
  if (W <= 0 || (a.causal && W > L)) {
    if (threadIdx.x == 0 && chunk == 0 && rg == 0) report(a.status, ACTKV_E_INVALID, r, W);
    return;
  }
  const int n_mb = min(2, (rows - rg * 256 + 127) / 128);
  const int t_begin = key_begin / TK;
  const int t_end = min((L + TK - 1) / TK, t_begin + a.lse_chunk / TK);
  const int n_tiles = t_end - t_begin;
  const int n_jobs = n_tiles * n_mb;
  const int S = ta.n_stages;

  const uint32_t smem_base = smem_u32(smem);
  const uint32_t k_smem = smem_base;                               // S x 32 KB
  LseBarriers* bars = reinterpret_cast<LseBarriers*>(smem + (size_t)S * KTILE_BYTES);
  volatile int* abort_flag = &bars->abort_flag;
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;   // warp-uniform

  if ((smem_base & 1023u) != 0) {                                  // swizzled tiles need 1024-byte alignment
    if (threadIdx.x == 0) report(a.status, ACTKV_E_CUDA, -2, (int32_t)smem_base);
    return;
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(smem_u32(&bars->k_full[s]), 1); mbar_init(smem_u32(&bars->k_empty[s]), 1); }
    mbar_init(smem_u32(&bars->q_ready), 8);
    for (int b = 0; b < LSE_SLOTS; ++b) {
      mbar_init(smem_u32(&bars->tmem_full[b]), 1);
      mbar_init(smem_u32(&bars->tmem_empty[b]), LSE_EPI_WARPS / 2);
    }
    mbar_init(smem_u32(&bars->drained), 1);
    bars->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars->tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  // epilogue identity (also used after the role split)
  const int ew = warp - 2;                       // 0..15 for epilogue warps
  const int quarter = warp & 3;                  // TMEM lanes this warp may touch
  const int mb = (ew >> 2) & 1;                  // row block
  const int ch = ew >> 3;                        // column half of a 128-key tile
  const int row_in_blk = quarter * 32 + lane;
  const int n = rg * 256 + mb * 128 + row_in_blk;                 // row within the unit
  const bool row_ok = warp >= 2 && (mb < n_mb) && n < rows;
  float m = -INFINITY, sum = 0.f;
  bool epi_ok = true;

  if (warp == 0) {
    // ---------------- TMA producer: K tiles through the block table ----------------
    const int n_lp = (L + a.pool.page_size - 1) / a.pool.page_size;
    const int layer = a.layer_begin + slab;
    // page ids of four tiles at a time, one per lane (lane / 8 = tile within the group, lane % 8 = page);
    // the next group's ids are loaded while the current four tiles are being issued
    int32_t pid = page_for_tile(a.tab, a.pool.n_pages, r, t_begin * 8 + lane, n_lp, a.status);
    int32_t pid_next = 0;
    for (int it = 0; it < n_tiles; ++it) {
      const int s = it % S;
      const uint32_t ph = (uint32_t)(it / S) & 1u;
      if ((it & 3) == 0 && it + 4 < n_tiles)
        pid_next = page_for_tile(a.tab, a.pool.n_pages, r, (t_begin + it + 4) * 8 + lane, n_lp, a.status);
      int ok = 1;
      if (lane == 0) {
        ok = mbar_wait(smem_u32(&bars->k_empty[s]), ph ^ 1u, abort_flag) ? 1 : 0;
        if (ok) mbar_expect_tx(smem_u32(&bars->k_full[s]), KTILE_BYTES);
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if ((lane >> 3) == (it & 3)) {
        const uint32_t dst = k_smem + s * KTILE_BYTES + (lane & 7) * 2048;
        tma_load_4d(dst, &kmap, smem_u32(&bars->k_full[s]), 0, h, pid * 16, layer);
        tma_load_4d(dst + HALF_BYTES, &kmap, smem_u32(&bars->k_full[s]), 64, h, pid * 16, layer);
      }
      if ((it & 3) == 3) pid = pid_next;
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: A = Q block in TMEM, B = K tile in shared memory ----------------
    // The whole warp runs the loop (waits and descriptor arithmetic stay warp-uniform, so they can
    // live in uniform registers); one elected lane issues the tcgen05 instructions.
    // The tensor pipe's queue is shallow: whatever the issuing warp spends between two jobs (a successful
    // barrier wait costs 100-200 cycles) is idle time of the pipe.  So the barriers of job j+1 are polled
    // (mbarrier.test_wait, non-blocking) BEFORE the MMAs of job j are issued and the answers are only read
    // afterwards; the blocking wait is the fallback when they were not ready yet.
    const uint32_t idesc = idesc_bf16(128, 128);
    const uint64_t desc0 = smem_desc_sw128(k_smem);
    bool ok = mbar_wait(smem_u32(&bars->q_ready), 0, abort_flag);
    tc_fence_after();
    if (ok) ok = mbar_wait(smem_u32(&bars->k_full[0]), 0, abort_flag);               // job 0: stage 0, slot 0
    // All indices are carried incrementally (no divisions in the loop): any cycle the issuer spends
    // between two MMAs beyond the queue's depth is a bubble in the tensor pipe.
    int s = 0, b = 0, slot = 0;
    uint32_t kpar = 0, epar = 7u;                  // bit i: parity to wait for on tmem_empty[i] (fresh barriers pass with 1)
    const bool leader = elect_one();
    for (int job = 0; ok && job < n_jobs; ++job) {
      int bn = b + 1, sn = s;
      uint32_t kparn = kpar;
      if (bn == n_mb) { bn = 0; sn = s + 1; if (sn == S) { sn = 0; kparn ^= 1u; } }
      const int slotn = slot == LSE_SLOTS - 1 ? 0 : slot + 1;
      const bool has_next = job + 1 < n_jobs;
      const uint32_t kfull_n = smem_u32(&bars->k_full[sn]);
      const uint32_t empty_n = smem_u32(&bars->tmem_empty[slotn]);
      const uint32_t epar_n = (epar >> slotn) & 1u;
      bool kready = true, eready = true;
      if (has_next) {
        kready = (sn == s) || mbar_test_wait(kfull_n, kparn);
        eready = mbar_test_wait(empty_n, epar_n);
      }
      tc_fence_after();
      if (leader) {
        const uint64_t desc_s = desc0 + (uint64_t)((s * KTILE_BYTES) >> 4);
        const uint32_t d = tmem_base + LSE_A_COLS + slot * 128, at = tmem_base + b * 64;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          umma_bf16_ts(d, at + kk * 8, desc_s + (uint64_t)(((kk >> 2) * HALF_BYTES + (kk & 3) * 32) >> 4), idesc,
                       kk > 0 ? 1u : 0u);
        umma_commit(smem_u32(&bars->tmem_full[slot]));
        if (bn == 0) umma_commit(smem_u32(&bars->k_empty[s]));
      }
      epar ^= 1u << slot;
      if (has_next) {
        if (!kready) ok = mbar_wait(kfull_n, kparn, abort_flag);
        if (ok && !eready) ok = mbar_wait(empty_n, epar_n, abort_flag);
      }
      b = bn; s = sn; kpar = kparn; slot = slotn;
    }
    // drain: every MMA issued above has completed before TMEM is freed
    __syncwarp();
    if (leader) umma_commit(smem_u32(&bars->drained));
    __syncwarp();
    mbar_wait(smem_u32(&bars->drained), 0, abort_flag, ok ? WAIT_LIMIT_NS : DRAIN_LIMIT_NS);
    __syncwarp();
  } else {
    // ---------------- epilogue warps ----------------
    if (ch == 0) {
      // Q row of this thread -> its TMEM lane, 64 packed columns of block mb (zeros for padding rows)
      const int w = n / G, g = n - w * G;
      const uint4* src = reinterpret_cast<const uint4*>(
          a.q + (((int64_t)slab * a.sum_win + w0 + w) * a.n_q_heads + h * G + g) * HD);
      const uint32_t dst = tmem_base + ((uint32_t)(quarter * 32) << 16) + mb * 64;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        uint4 x[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) x[k] = row_ok ? __ldg(src + i * 4 + k) : make_uint4(0, 0, 0, 0);
        tmem_st16(dst + i * 16, reinterpret_cast<const uint32_t*>(x));
      }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->q_ready));
    }
    const int w = n / G;
    const int jmax = a.causal ? (L - W + w) : (L - 1);            // last key this row sees
    const float c = a.scale_log2;
    for (int job = mb; mb < n_mb && job < n_jobs; job += n_mb) {
      const int it = job / n_mb;
      const int slot = job % LSE_SLOTS;
      epi_ok = mbar_wait(smem_u32(&bars->tmem_full[slot]), (uint32_t)(job / LSE_SLOTS) & 1u, abort_flag);
      if (!epi_ok) break;
      tc_fence_after();
      const int col0 = (t_begin + it) * TK + ch * 64;              // first key of this thread's columns
      int n_valid = min(jmax, L - 1) - col0 + 1;
      n_valid = row_ok ? max(0, min(64, n_valid)) : 0;
#ifdef ACTKV_EXP_NO_EPI
      if (false) {
#else
      if (__any_sync(0xffffffffu, n_valid > 0)) {
#endif
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + LSE_A_COLS + slot * 128 + ch * 64;
        float v[2][32];
        tmem_ld32(taddr, v[0]);
        tmem_ld32(taddr + 32, v[1]);
        tmem_ld_wait();
#pragma unroll
        for (int cg = 0; cg < 2; ++cg) {
          const float* x = v[cg];
          const int nv = n_valid - cg * 32;       // valid columns of this group for this row
          if (nv >= 32) {
            lse_group<POLY>(x, c, m, sum);
          } else if (nv > 0) {
            float gm = -INFINITY;
#pragma unroll
            for (int i = 0; i < 32; ++i) gm = fmaxf(gm, i < nv ? x[i] : -INFINITY);
            if (gm > m) { sum = (m == -INFINITY) ? 0.f : sum * exp2f((m - gm) * c); m = gm; }
            const float mc = m * c;
#pragma unroll
            for (int i = 0; i < 32; ++i) sum += (i < nv) ? exp2f(fmaf(x[i], c, -mc)) : 0.f;
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->tmem_empty[slot]));
    }
    if (ch == 1) bars->exch[mb * 128 + row_in_blk] = make_float2(m, sum);
  }
  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (warp >= 2 && ch == 0 && row_ok && epi_ok && !*abort_flag) {
    // merge the two column halves of the row, store (max in log2 units, sum); (-inf, 0) when the row saw
    // no key of this chunk
    const float2 o = bars->exch[mb * 128 + row_in_blk];
    const float mm = fmaxf(m, o.x);
    float ss = 0.f;
    if (mm > -INFINITY) {
      const float c = a.scale_log2;
      ss = (m > -INFINITY ? sum * exp2f((m - mm) * c) : 0.f) + (o.x > -INFINITY ? o.y * exp2f((o.x - mm) * c) : 0.f);
    }
    a.partials[((int64_t)u * a.n_chunks + chunk) * a.rows_max + n] =
        make_float2(mm == -INFINITY ? mm : mm * a.scale_log2, ss);
  }
  if (warp == 0 && lane == 0 && *abort_flag) {
    report(a.status, ACTKV_E_TIMEOUT, u, chunk);
    // loads still in flight land in this CTA's shared memory: give them a moment before exiting
    for (int s = 0; s < S; ++s) mbar_wait(smem_u32(&bars->k_full[s]), 0, abort_flag, DRAIN_LIMIT_NS / 8);
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace tc
}  // namespace actkv
