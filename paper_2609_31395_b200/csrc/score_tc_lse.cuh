// LSE pass of the tensor-core score path (Section 7.1, LSE equation):
//   lse[row] = log sum_{key visible} exp(sm_scale * q_row . k_key),   row = (window token w, group head g).
//
// D[row, key] = Q K^T with the rows on the TMEM lanes, so every epilogue thread owns one row per
// 128-row block and folds its share of the row's logits into a running (reference, sum of exp2): no
// shuffles.  A CTA covers ALL row blocks of a unit (up to four, 512 rows) x one chunk of keys, so a
// K tile is fetched once per unit.
//
// Operand placement.  An A operand in shared memory is re-read for every MMA and that read is not
// overlapped with the MMA (measured 105 cycles per 128x128x16 MMA against 74 with A in tensor memory,
// 64 nominal).  The Q blocks are the same for every key tile of the CTA, so they are written once into
// tensor memory (tcgen05.st, two bf16 per 32-bit column) and used as the A operand from there; only
// the K tile (B) streams through shared memory.
// TMEM columns: [0,256) the four Q blocks, [256,512) two 128-column accumulators; a job is one
// (key tile, row block) product.  Even jobs go to accumulator 0, odd jobs to accumulator 1; each
// accumulator has its own MMA-issuing warp and its own group of eight epilogue warps (64 columns per
// thread), which hand the accumulator back as soon as their columns are in registers.  While one group
// waits for tensor memory the other keeps the special function unit busy.
//
// What bounds the kernel (measured on B200 with micro-benchmarks and per-job timestamps):
//  * Issuing is not free: a tcgen05.mma costs the issuing thread about 50 cycles and a tcgen05.commit
//    about 80, some 470 cycles for a job the tensor pipe executes in 512, and the commit reaches the
//    waiting warps about 240 cycles after the last MMA retires.  One issuer doing its barrier
//    handshakes in between left the pipe idle 40 % of the time; hence two issuers.
//  * An SM sub-partition dispatches about one fp32 operation per clock (the packed fp32x2 forms take
//    two, so they save nothing) and its special function unit delivers one warp-wide exp2 per 8 clocks.
//    One exp2 per (row, key) on that unit alone costs 8 clocks per warp and logit against 4.6 for the
//    contraction: the pass is bound by the exp rate.  Of each 8 columns, NPOLY take a polynomial on the
//    FMA pipe instead (ten dispatch slots each, against three slots and eight clocks of the unit); the
//    two kinds overlap only partly, and NPOLY = 1 measured best (0: 9.06 ms, 1: 8.63, 2: 8.90, 3: 9.32 at
//    the bench shape).
//  * To keep the slot count low there is no running maximum: the reference m of a row is the maximum of
//    the first logits the thread saw, later logits may exceed it (2^x is evaluated for x up to 126), and
//    only if a partial sum grows past 2^40 is the reference moved (a rare, slower path that also serves
//    tiles cut by the end of the request or by the causal diagonal).
// Polynomial: y = sat(x/252 + 1/2) clamps x to [-126, 126] inside the multiply-add that forms it;
// j = round(x) by the magic-number addition, f = x - j in [-0.5, 0.5], 2^x = 2^j p(f) with p a cubic
// fitted to 2^f (max relative error 7.5e-5, far inside the 2e-3 score tolerance), 2^j applied by adding
// j to the exponent field.
#pragma once

#include "tc_common.cuh"

namespace actkv {
namespace tc {

constexpr int LSE_NPOLY = 1;                     // columns of every 8 whose exp2 is the polynomial

__device__ __forceinline__ float ffma_sat(float a, float b, float c) {
  float d;
  asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// 2^x for x = 252 y - 126, y in [0, 1]
__device__ __forceinline__ float exp2_poly_y(float y) {
  constexpr float MAGIC = 12582912.f;            // 1.5 * 2^23: adding it rounds to the nearest integer
  const float t = fmaf(y, 252.f, MAGIC - 126.f); // MAGIC + j, j = round(x), in the low mantissa bits
  const float j = t - MAGIC;
  const float f = fmaf(y, 252.f, -126.f - j);    // x - j
  float p = fmaf(0.0551716648042202f, f, 0.2426111251115799f);
  p = fmaf(p, f, 0.6932609677314758f);
  p = fmaf(p, f, 0.9999280571937561f);
  return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}

// 32 logits of one row, all visible, against the row's reference m (finite): returns
// sum_i exp2((v_i - m) c).  nmc = -m c; c1 = c / 252, c0 = 1/2 - m c / 252.
template <int NPOLY>
__device__ __forceinline__ float lse_fast32(const float* v, float c, float nmc, float c1, float c0) {
  float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int g8 = 0; g8 < 4; ++g8) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float x = v[g8 * 8 + i];
      // the polynomial columns are spread over the group so that the two kinds interleave in program order
      const bool poly = (NPOLY >= 1 && i == 1) || (NPOLY >= 2 && i == 4) || (NPOLY >= 3 && i == 6) || (NPOLY >= 4 && i == 3);
      const float e = poly ? exp2_poly_y(ffma_sat(x, c1, c0)) : exp2f(fmaf(x, c, nmc));
      s[i & 3] += e;
    }
  }
  return (s[0] + s[1]) + (s[2] + s[3]);
}

// The general form: logits n_lo <= i < nv (any integers) are visible; moves the reference to the maximum seen
// so far.  Also the entry for a row's first logits (m = -inf, sum = 0).
__device__ __forceinline__ void lse_slow32(const float* v, int n_lo, int nv, float c, float& m, float& sum) {
  if (nv <= 0 || n_lo >= 32 || n_lo >= nv) return;
  float gm = -INFINITY;
#pragma unroll
  for (int i = 0; i < 32; ++i) gm = fmaxf(gm, (i >= n_lo && i < nv) ? v[i] : -INFINITY);
  if (gm > m) { sum = (m == -INFINITY) ? 0.f : sum * exp2f((m - gm) * c); m = gm; }
  const float mc = m * c;
#pragma unroll
  for (int i = 0; i < 32; ++i) sum += (i >= n_lo && i < nv) ? exp2f(fmaf(v[i], c, -mc)) : 0.f;
}

constexpr int LSE_EPI_WARPS = 16;                // (TMEM lane quarter, accumulator, column half)
// Warp 0 is the producer, warps 1 and 2 the MMA issuers, warps 3..18 the epilogue: 19 warps leave each thread 104
// registers.  The epilogue is sensitive to that: with a 20th warp (tried: a copy role for the items of a pending
// compaction, as in the pooled-score kernel) the allocation is 96 and the pass 7-9 % slower, also when the
// epilogue warpgroups take their 104 back from the control warps at run time; what the copies gained by hiding
// under this kernel was less than that.
constexpr int LSE_EPI_WARP0 = 3;
constexpr int LSE_THREADS = (LSE_EPI_WARP0 + LSE_EPI_WARPS) * 32;
constexpr int LSE_SLOTS = 2;                     // accumulators
constexpr int LSE_A_COLS = 256;                  // TMEM columns holding the four Q blocks
constexpr float LSE_BIG = 1099511627776.f;       // 2^40: a partial sum beyond it moves the reference

struct LseBarriers {
  uint64_t k_full[8];
  uint64_t k_empty[8];
  uint64_t q_ready;
  uint64_t tmem_full[LSE_SLOTS];
  uint64_t tmem_empty[LSE_SLOTS];
  uint64_t drained[2];
  uint32_t tmem_base;
  int abort_flag;
  float2 state[2][4][2][128];  // (reference, sum) per (group, row block, column half, row in block)
};

// After tcgen05.wait::ld: ties the loaded registers to the wait, so that no use of them is scheduled
// ahead of it (the loads are asynchronous; the compiler sees their outputs as defined at issue).
template <int N>
__device__ __forceinline__ void tmem_ld_fence(float* v) {
#pragma unroll
  for (int i = 0; i < N; ++i) asm volatile("" : "+f"(v[i]));
}

__device__ __forceinline__ int sel4(const int (&x)[4], int i) { return i == 0 ? x[0] : i == 1 ? x[1] : i == 2 ? x[2] : x[3]; }

// One job as one epilogue warp sees it: the warp takes 64 columns (two register buffers of 32) of the
// accumulator of its group, hands the accumulator back as soon as they are in registers, and folds them
// into the row's (reference, sum) in `st`.  The two groups work on alternate jobs, so while one waits
// for tensor memory the other keeps the special function unit busy.
//   tq      tensor-memory address of the group's accumulator, this warp's lane quarter and first column
//   nv_min  visible columns (from the warp's first column) of the most restricted row of this thread
//   nlo_max columns (from the warp's first column) below the first visible key of the most restricted row
//   jm, jl  last / first visible key of this thread's row in each row block; key0 = key of the warp's first column
// WIN: the layer has a sliding window (a first visible key per row); kept out of the common instantiation, whose
// epilogue should not carry the second bound.
template <int NPOLY, bool WIN>
__device__ __forceinline__ bool lse_job(LseBarriers* bars, volatile int* abort_flag, uint32_t tq, int grp, int job,
                                        int mb, float2* st, int nv_min, int nlo_max, const int (&jm)[4], const int (&jl)[4],
                                        int key0, float c, float c1, int lane, long long wait_cycles) {
  float v[64];
  float* va = v;
  float* vb = v + 32;
  if (!mbar_wait_warp(smem_u32(&bars->tmem_full[grp]), (uint32_t)(job >> 1) & 1u, abort_flag, wait_cycles)) return false;
  tc_fence_after();
  tmem_ld64(tq, v);
  float2 ms = *st;
  tmem_ld_wait();
  tmem_ld_fence<64>(v);
  tc_fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(smem_u32(&bars->tmem_empty[grp]));
  bool slow = __any_sync(0xffffffffu, nv_min < 64 || (WIN && nlo_max > 0) || ms.x == -INFINITY);
  if (!slow) {
    const float nmc = -ms.x * c, c0 = fmaf(nmc, 1.f / 252.f, 0.5f);
    const float ps = lse_fast32<NPOLY>(va, c, nmc, c1, c0) + lse_fast32<NPOLY>(vb, c, nmc, c1, c0);
    slow = __any_sync(0xffffffffu, !(ps < LSE_BIG));
    if (!slow) ms.y += ps;
  }
  if (slow) {
    const int nv = sel4(jm, mb) - key0 + 1, nlo = WIN ? sel4(jl, mb) - key0 : 0;
    lse_slow32(va, nlo, nv, c, ms.x, ms.y);
    lse_slow32(vb, nlo - 32, nv - 32, c, ms.x, ms.y);
  }
  *st = ms;
  return true;
}

// ROW_GROUPS: the unit's window has more than MAX_ROWS rows and the grid has a row-group dimension (kept
// out of the common instantiation, whose code should not change with it).
// NH: 64-dim halves of the head dimension (head_dim = 64 NH); a K tile is NH x [128 keys][64 bf16].
template <int NPOLY, bool ROW_GROUPS, int NH, bool WIN>
__global__ void __launch_bounds__(LSE_THREADS, 1)
score_tc_lse_kernel(const __grid_constant__ CUtensorMap kmap, const TcArgs ta) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const ScoreArgs& a = ta.a;
  const int R = a.tab.n_req, Hkv = a.pool.n_kv_heads, G = a.group;
  const int cu = blockIdx.x / a.n_chunks;
  const int chunk = blockIdx.x - cu * a.n_chunks;
  const int rg = ROW_GROUPS ? cu % ta.n_rg : 0;          // row group: rows [row0, row0 + MAX_ROWS) of the unit
  const int u = ROW_GROUPS ? cu / ta.n_rg : cu;
  const int r = u % R, h = (u / R) % Hkv, slab = u / (R * Hkv);
  const int L = a.tab.seq_len[r];
  const int w0 = a.win_indptr[r], W = a.win_indptr[r + 1] - w0;
  const int row0 = ROW_GROUPS ? rg * MAX_ROWS : 0;
  const int rows = ROW_GROUPS ? min(W * G - row0, MAX_ROWS) : W * G;     // rows of this CTA
  const int key_begin = chunk * a.lse_chunk;
  if (key_begin >= L || (rg > 0 && rows <= 0)) return;
  if (W <= 0 || (a.causal && W > L)) {
    if (threadIdx.x == 0 && chunk == 0 && rg == 0) report(a.status, ACTKV_E_INVALID, r, W);
    return;
  }
  // the host sized shared memory, tensor memory and the partials from upper bounds of the window and the length
  if (W * G > a.rows_max || L > a.n_chunks * a.lse_chunk || rows > MAX_ROWS) {
    if (threadIdx.x == 0 && chunk == 0 && rg == 0) report(a.status, ACTKV_E_INVALID, r, W * G > a.rows_max ? W : L);
    return;
  }
  const int n_mb = (rows + 127) / 128;                   // 1..4
  const int t_end = min((L + TK - 1) / TK, key_begin / TK + a.lse_chunk / TK);
  // sliding-window layer: key tiles below the first key any row of the unit sees are not fetched at all
  const int lo_all = (WIN && a.win_left > 0) ? max(0, (a.causal ? L - W : L - 1) - a.win_left + 1) : 0;
  const int t_begin = max(key_begin / TK, lo_all / TK);
  const int n_tiles = t_end - t_begin;
  if (n_tiles <= 0) {                                    // no row sees a key of this chunk
    for (int n = threadIdx.x; n < rows; n += blockDim.x)
      a.partials[((int64_t)u * a.n_chunks + chunk) * a.rows_max + row0 + n] = make_float2(-INFINITY, 0.f);
    return;
  }
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
    for (int s = 0; s < S; ++s) { mbar_init(smem_u32(&bars->k_full[s]), 1); mbar_init(smem_u32(&bars->k_empty[s]), 2); }
    mbar_init(smem_u32(&bars->q_ready), LSE_EPI_WARPS);
    for (int b = 0; b < LSE_SLOTS; ++b) {
      mbar_init(smem_u32(&bars->tmem_full[b]), 1);
      mbar_init(smem_u32(&bars->tmem_empty[b]), LSE_EPI_WARPS / 2);
    }
    mbar_init(smem_u32(&bars->drained[0]), 1);
    mbar_init(smem_u32(&bars->drained[1]), 1);
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
  const int ew = warp - LSE_EPI_WARP0;           // 0..15 for epilogue warps
  const int quarter = warp & 3;                  // TMEM lanes this warp may touch
  const int k = ew >> 2;                         // 0..3
  const int grp = k >> 1;                        // accumulator / job parity this warp serves
  const int half = k & 1;                        // its columns: [64 half, 64 half + 64)
  const int rib = quarter * 32 + lane;           // row within a 128-row block
  bool epi_ok = true;

  if (warp == 0) {
    // ---------------- TMA producer: K tiles through the block table ----------------
    const int layer = a.layer_begin + slab;
    // (one producer: this pass needs a K tile per four jobs, far below what one warp delivers)
    if (ta.k5) k_tile_producer<true, NH>(&kmap, a, bars, k_smem, S, r, h, layer, L, t_begin, n_tiles, lane, abort_flag, 0, 1, ta.wait_cycles, ta.stall_tile);
    else k_tile_producer<false, NH>(&kmap, a, bars, k_smem, S, r, h, layer, L, t_begin, n_tiles, lane, abort_flag, 0, 1, ta.wait_cycles, ta.stall_tile);
  } else if (warp < LSE_EPI_WARP0) {
    // ---------------- MMA issuers: A = Q block in TMEM, B = K tile in shared memory ----------------
    // Two warps, one per accumulator: warp 1 issues the even jobs into accumulator 0, warp 2 the odd jobs
    // into accumulator 1.  Issuing is not free for the issuing thread (measured: about 50 cycles per
    // tcgen05.mma and 80 per tcgen05.commit, i.e. some 470 cycles for a job that the tensor pipe executes
    // in 512) and the barrier handshakes come on top, so one issuer alone cannot keep the pipe busy.
    // The whole warp runs the loop (waits stay warp-uniform); one elected lane issues.
    // Every issuer waits for every K tile and releases it (tcgen05.commit after its last job of the tile,
    // or a plain arrive when it had none), so a stage is refilled only when both are done with it.
    const int mw = warp - 1;
    const uint32_t idesc = idesc_bf16(128, 128);
    const uint64_t desc0 = smem_desc_sw128(k_smem);
    const uint32_t full_bar = smem_u32(&bars->tmem_full[mw]), empty_bar = smem_u32(&bars->tmem_empty[mw]);
    const uint32_t d = tmem_base + LSE_A_COLS + mw * 128;
    bool ok = mbar_wait_warp(smem_u32(&bars->q_ready), 0, abort_flag, ta.wait_cycles);
    tc_fence_after();
    int s = 0, job = 0;
    uint32_t kpar = 0, epar = 1u;                  // parity to wait for on tmem_empty[mw] (a fresh barrier passes with 1)
    const bool leader = elect_one();
    for (int it = 0; ok && it < n_tiles; ++it) {
      ok = mbar_wait_warp(smem_u32(&bars->k_full[s]), kpar, abort_flag, ta.wait_cycles);
      if (!ok) break;
      tc_fence_after();
      const uint64_t desc_s = desc0 + (uint64_t)((s * KTILE_BYTES) >> 4);
      bool mine = false;
      for (int b = 0; b < n_mb; ++b, ++job) {
        if ((job & 1) != mw) continue;
        ok = mbar_wait_warp(empty_bar, epar, abort_flag, ta.wait_cycles);
        if (!ok) break;
        epar ^= 1u;
        tc_fence_after();
        if (leader) {
          const uint32_t at = tmem_base + b * 64;
#pragma unroll
          for (int kk = 0; kk < 4 * NH; ++kk)
            umma_bf16_ts(d, at + kk * 8, desc_s + (uint64_t)(((kk >> 2) * HALF_BYTES + (kk & 3) * 32) >> 4), idesc,
                         kk > 0 ? 1u : 0u);
          umma_commit(full_bar);
        }
        mine = true;
      }
      if (!ok) break;
      if (leader) {
        if (mine) umma_commit(smem_u32(&bars->k_empty[s]));
        else mbar_arrive(smem_u32(&bars->k_empty[s]));
      }
      if (++s == S) { s = 0; kpar ^= 1u; }
    }
    // drain: every MMA issued above has completed before TMEM is freed
    __syncwarp();
    if (leader) umma_commit(smem_u32(&bars->drained[mw]));
    __syncwarp();
    // (a tear-down wait: it does not end early because another role gave up)
    mbar_wait_warp(smem_u32(&bars->drained[mw]), 0, nullptr, ok ? ta.wait_cycles : DRAIN_LIMIT_CYCLES);
    __syncwarp();
  } else {
    // ---------------- epilogue warps ----------------
    {
      // Q row (block k, row rib) -> this thread's TMEM lane, 64 packed columns (zeros for padding rows)
      const int n = k * 128 + rib;
      const bool live = k < n_mb && n < rows;
      const int w = (row0 + n) / G, g = (row0 + n) % G;
      const uint4* src = reinterpret_cast<const uint4*>(
          a.q + (((int64_t)slab * a.sum_win + w0 + (live ? w : 0)) * a.n_q_heads + h * G + (live ? g : 0)) * (64 * NH));
      const uint32_t dst = tmem_base + ((uint32_t)(quarter * 32) << 16) + k * 64;
      if (k < n_mb) {
        // (the whole row in flight at once: under load one round trip to L2 is thousands of cycles, and the
        // MMA issuers wait for the last row)
        uint4 x[8 * NH];
#pragma unroll
        for (int j = 0; j < 8 * NH; ++j) x[j] = live ? __ldg(src + j) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int i = 0; i < 2 * NH; ++i) tmem_st16(dst + i * 16, reinterpret_cast<const uint32_t*>(x + 4 * i));
        tmem_st_wait();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->q_ready));
    }
    // last key each of this thread's rows sees (padding rows: every key, their sums are dropped)
    // ... and the first one (0 unless the layer has a sliding window)
    int jm[4], jl[4];
#pragma unroll
    for (int mb = 0; mb < 4; ++mb) {
      const int n = mb * 128 + rib;
      jm[mb] = (a.causal && n < rows) ? (L - W + (row0 + n) / G) : (L - 1);
      jl[mb] = (WIN && a.win_left > 0 && n < rows) ? max(0, jm[mb] - a.win_left + 1) : 0;
      bars->state[grp][mb][half][rib] = make_float2(-INFINITY, 0.f);
    }
    const int jfast = min(min(jm[0], jm[1]), min(jm[2], jm[3]));
    const int jlmax = max(max(jl[0], jl[1]), max(jl[2], jl[3]));
    const float c = a.scale_log2, c1 = c * (1.f / 252.f);
    const uint32_t tq = tmem_base + ((uint32_t)(quarter * 32) << 16) + LSE_A_COLS + grp * 128 + half * 64;
    // (key tile, row block) of this group's jobs, carried along without divisions: job = tile * n_mb + mb
    int mb = grp % n_mb, key0 = (t_begin + grp / n_mb) * TK + half * 64;
    const int mb_step = 2 % n_mb, tile_step = 2 / n_mb;
    for (int job = grp; job < n_jobs; job += 2) {
      epi_ok = lse_job<NPOLY, WIN>(bars, abort_flag, tq, grp, job, mb, &bars->state[grp][mb][half][rib], jfast - key0 + 1,
                              jlmax - key0, jm, jl, key0, c, c1, lane, ta.wait_cycles);
      if (!epi_ok) break;
      mb += mb_step;
      key0 += tile_step * TK;
      if (mb >= n_mb) { mb -= n_mb; key0 += TK; }
    }
  }
  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (warp >= LSE_EPI_WARP0 && k == 0 && !*abort_flag) {
    // merge the four shares (group, column half) of each row, store (reference in log2 units, sum); (-inf, 0) when the
    // row saw no key of this chunk
    const float c = a.scale_log2;
#pragma unroll
    for (int mb = 0; mb < 4; ++mb) {
      const int n = mb * 128 + rib;
      if (mb < n_mb && n < rows) {
        float2 o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) o[i] = bars->state[i >> 1][mb][i & 1][rib];
        const float mm = fmaxf(fmaxf(o[0].x, o[1].x), fmaxf(o[2].x, o[3].x));
        float ss = 0.f;
        if (mm > -INFINITY) {
#pragma unroll
          for (int i = 0; i < 4; ++i) ss += o[i].x > -INFINITY ? o[i].y * exp2f((o[i].x - mm) * c) : 0.f;
        }
        a.partials[((int64_t)u * a.n_chunks + chunk) * a.rows_max + row0 + n] =
            make_float2(mm == -INFINITY ? mm : mm * a.scale_log2, ss);
      }
    }
  }
  if (warp == 0 && lane == 0 && *abort_flag) {
    report(a.status, ACTKV_E_TIMEOUT, u, chunk);
    // loads still in flight land in this CTA's shared memory: give them a moment before exiting
    for (int s = 0; s < S; ++s) mbar_wait(smem_u32(&bars->k_full[s]), 0, nullptr, DRAIN_LIMIT_CYCLES / 64);
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace tc
}  // namespace actkv
