// Pooled-score pass of the tensor-core score path (Section 7.1 recovery identity A = exp(s - LSE);
// Algorithm 3 steps 3-5: max over the GQA group, mean over the action tokens).
//
// D[key, row] = K Q^T: the 128 keys of a tile sit on the TMEM lanes, row = w*G + g on the columns,
// 256 columns per accumulator, two accumulators in the 512 TMEM columns.  A "job" is one (key tile,
// 256-row chunk) accumulator; even jobs use accumulator 0, odd jobs accumulator 1, each with its own
// MMA-issuing warp.  The two epilogue warpgroups take alternate jobs whole, one key per thread; with two
// row chunks per key tile warpgroup 1 hands its sum of a tile to warpgroup 0 through shared memory.
#pragma once

#include "tc_common.cuh"

namespace actkv {
namespace tc {

// Warps: 0 producer, 1-2 MMA issuers, 3 second producer (the control warpgroup); 4-11 epilogue (two
// warpgroups); 12-15 copy role (items of a pending compaction, when the launch carries one).
// Registers: the kernel starts with 128 per thread (512 threads); the control warpgroup drops to 64 and the copy
// warpgroup to 112, the two epilogue warpgroups rise to 168: 128 x (64 + 2 x 168 + 112) = 65536.
constexpr int POOL_EPI_WARPS = 8;
constexpr int POOL_EPI_WARP0 = 4;                           // first epilogue warp
constexpr int POOL_COPY_WARP0 = POOL_EPI_WARP0 + POOL_EPI_WARPS;
constexpr int POOL_THREADS = (POOL_COPY_WARP0 + 4) * 32;
constexpr int POOL_PRODUCER2 = 3;                           // warp index of the second producer
constexpr uint32_t POOL_REGS_CTRL = 64, POOL_REGS_EPI = 168, POOL_REGS_COPY = 112;
constexpr int POOL_REGS_ENTRY = 128;                        // what the launch must have allocated per thread
static_assert(128 * (POOL_REGS_CTRL + 2 * POOL_REGS_EPI + POOL_REGS_COPY) <= POOL_THREADS * POOL_REGS_ENTRY, "register budget");

struct PoolBarriers {
  uint64_t k_full[8];
  uint64_t k_empty[8];
  uint64_t q_full;
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t part_full;         // warpgroup 1 -> warpgroup 0: partial sums of a tile are in `exch`
  uint64_t part_empty;        // warpgroup 0 -> warpgroup 1: `exch` has been read
  uint64_t drained[2];
  uint32_t tmem_base;
  int abort_flag;
  int prod_done;              // the first producer has issued its last key tile: the copy role takes no more items
  float exch[TK];
};

// 64 columns of one accumulator lane: x = s for rows n .. n + 63 of this key, nlse = -lse*log2(e) of those rows
// (-inf for padding rows).  Adds sum_w exp2(max_g(s*c + nlse)) over the action tokens w_first .. that lie
// in [w_min, w_end) to `acc`.  Action tokens outside [w_min, w_end) do not count: below w_min the key is
// not visible yet (causal rule), from w_end on the columns are padding (with a narrow MMA they were never
// written and may hold anything).
template <int G>
__device__ __forceinline__ void pool_fold64(float* x, const float* nlse, int w_first, int w_min, int w_end, float c,
                                            float& acc) {
  const float4* l4 = reinterpret_cast<const float4*>(nlse);
#pragma unroll
  for (int q4 = 0; q4 < 16; ++q4) {
    const float4 l = l4[q4];
    ffma2(x[q4 * 4 + 0], x[q4 * 4 + 1], x[q4 * 4 + 0], x[q4 * 4 + 1], c, l.x, l.y);
    ffma2(x[q4 * 4 + 2], x[q4 * 4 + 3], x[q4 * 4 + 2], x[q4 * 4 + 3], c, l.z, l.w);
  }
  constexpr int WPG = 64 / G;                 // action tokens per 64-column group (G <= 32)
#pragma unroll
  for (int i = 0; i < WPG; ++i) {
    const float mx = max_of<G>(x + i * G);
    const int w = w_first + i;
    acc += (w >= w_min && w < w_end) ? exp2f(mx) : 0.f;
  }
}

template <int G>
__device__ __forceinline__ void pool_job(uint32_t taddr, const float* nlse, int n_cg, int w_first, int w_min, int w_end,
                                         float c, float& acc, uint32_t empty_bar, int lane) {
  // At most 128 columns (n_cg <= 4 groups of 32): both 64-column loads are issued at once and the
  // accumulator is handed back to the MMA warp as soon as they are in registers, before anything is folded.
  const int n_c2 = (n_cg + 1) >> 1;
  float v[2][64];
  tmem_ld64(taddr, v[0]);
  if (n_c2 > 1) tmem_ld64(taddr + 64, v[1]);
  tmem_ld_wait();
  tc_fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(empty_bar);
  pool_fold64<G>(v[0], nlse, w_first, w_min, w_end, c, acc);
  if (n_c2 > 1) pool_fold64<G>(v[1], nlse + 64, w_first + 64 / G, w_min, w_end, c, acc);
}

// G: the group size rounded up to a power of two.  A group of a.group < G query heads is padded with
// rows that drop out of the max (-lse = -inf); their queries are whatever the TMA box picks up behind
// the group (the next group's heads, or zeros past the last head).
// NH: 64-dim halves of the head dimension (head_dim = 64 NH).
template <int G, int NH>
__global__ void __launch_bounds__(POOL_THREADS, 1)
score_tc_pool_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap qmap, const TcArgs ta) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const ScoreArgs& a = ta.a;
  const int R = a.tab.n_req, Hkv = a.pool.n_kv_heads;
  const int u = blockIdx.x / ta.n_kchunks;
  const int kchunk = blockIdx.x - u * ta.n_kchunks;
  const int r = u % R, h = (u / R) % Hkv, slab = u / (R * Hkv);
  const int L = a.tab.seq_len[r];
  const int w0 = a.win_indptr[r], W = a.win_indptr[r + 1] - w0;
  // rows of this launch: [row_begin, row_begin + rows) of the unit's W*G; a window of more than MAX_ROWS
  // rows is taken MAX_ROWS (a whole number of action tokens) per launch, later launches add to the score
  const int row_begin = ta.row_begin, w_begin = row_begin / G;
  const int rows = min(W * G - row_begin, MAX_ROWS);
  const int t_first = kchunk * ta.tiles_per_cta;           // first key tile of this CTA's range
  if (t_first * TK >= L) return;
  if (row_begin > 0 && rows <= 0) return;                   // this request's window ends before this row group
  if (W <= 0 && a.acc_steps != nullptr) return;            // accumulate mode: a request outside its action region
  if (W <= 0 || (a.causal && W > L)) {
    if (threadIdx.x == 0 && kchunk == 0) report(a.status, ACTKV_E_INVALID, r, W);
    return;
  }
  // the host sized shared memory and the launch from upper bounds of the window and the length
  if (W * a.group > a.rows_max || L > ta.n_kchunks * ta.tiles_per_cta * TK) {
    if (threadIdx.x == 0 && kchunk == 0) report(a.status, ACTKV_E_INVALID, r, W * a.group > a.rows_max ? W : L);
    return;
  }
  const int t_end = min((L + TK - 1) / TK, t_first + ta.tiles_per_cta);
  // Sliding-window layer: a key below the first key any row of the unit sees scores 0; whole key tiles of
  // them are written here and neither fetched nor multiplied.
  const int lw = L - W;
  const int win = a.win_left;
  int t_vis = t_first;
  if (win > 0) {
    const int lo_all = max(0, (a.causal ? lw : L - 1) - win + 1);
    t_vis = min(t_end, max(t_first, lo_all / TK));
    float* out0 = a.score_out + ((int64_t)slab * Hkv + h) * a.sum_tok + a.tok_indptr[r];
    if (row_begin == 0)
      for (int key = t_first * TK + threadIdx.x; key < min(L, t_vis * TK); key += blockDim.x)
        store_pooled(a, r, out0 + key, 0.f, 0.f, W);
    if (t_vis >= t_end) return;
  }
  const int t_begin = t_vis;                               // first key tile that is fetched and multiplied
  const int n_tiles = t_end - t_begin;
  const int rows_pad = (rows + 127) & ~127;               // <= MAX_ROWS (checked by the host)
  const bool whole = rows > 128;                          // a job has up to 256 columns: two register loads (see the epilogue)
  const int n_rc = (rows_pad + 255) / 256;                // 256-row chunks per key tile: 1 or 2
  const int n_qblk = rows_pad / 128;
  const int n_jobs = n_tiles * n_rc;
  const int S = ta.n_stages;

  const uint32_t smem_base = smem_u32(smem);
  const uint32_t q_bytes = (uint32_t)n_rc * 2 * QBLK_BYTES;     // per chunk: [2 halves][256 rows x 128 B]
  const uint32_t q_smem = smem_base;
  const uint32_t k_smem = smem_base + q_bytes;
  float* nlse = reinterpret_cast<float*>(smem + q_bytes + (size_t)S * KTILE_BYTES);       // [rows_pad]
  PoolBarriers* bars = reinterpret_cast<PoolBarriers*>(reinterpret_cast<uint8_t*>(nlse) + MAX_ROWS * 4);
  volatile int* abort_flag = &bars->abort_flag;
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;   // warp-uniform

  if ((smem_base & 1023u) != 0) {
    if (threadIdx.x == 0) report(a.status, ACTKV_E_CUDA, -2, (int32_t)smem_base);
    return;
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(smem_u32(&bars->k_full[s]), 1); mbar_init(smem_u32(&bars->k_empty[s]), 2); }
    mbar_init(smem_u32(&bars->q_full), 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars->tmem_full[b]), 1);
      mbar_init(smem_u32(&bars->tmem_empty[b]), POOL_EPI_WARPS / 2);
    }
    mbar_init(smem_u32(&bars->part_full), POOL_EPI_WARPS / 2);
    mbar_init(smem_u32(&bars->part_empty), POOL_EPI_WARPS / 2);
    mbar_init(smem_u32(&bars->drained[0]), 1);
    mbar_init(smem_u32(&bars->drained[1]), 1);
    bars->abort_flag = 0;
    bars->prod_done = 0;
    fence_barrier_init();
  }
  {
    // -lse of every row in log2 units; padding rows get -inf so that s*c + nlse drops out of the max
    const int g_real = a.group;
    const float* lse_base = a.lse + ((int64_t)slab * a.sum_win + w0 + w_begin) * a.n_q_heads + h * g_real;
    for (int n = threadIdx.x; n < rows_pad; n += blockDim.x)
      nlse[n] = (n < rows && (n % G) < g_real) ? -lse_base[(int64_t)(n / G) * a.n_q_heads + (n % G)] * kLog2e : -INFINITY;
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars->tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  if (warp >= POOL_COPY_WARP0) {
    // ---------------- copy role: items of the pending compaction of another layer group ----------------
    // Order-free copies between pages this kernel neither reads nor writes (Section 7.2); they use the HBM
    // bandwidth the contraction leaves idle.  Items are taken until the producer has issued the CTA's last
    // key tile: the last item then ends about when the last tiles have been scored, and the CTA retires with
    // its main work.
    reg_dec<POOL_REGS_COPY>();
    volatile int* done = &bars->prod_done;
    cj_copy_role<NH + 2, 16>(ta.copy_ws, lane, [&]() {
      int go = 0;
      if (lane == 0) go = (!*done && !*abort_flag) ? 1 : 0;
      return __shfl_sync(0xffffffffu, go, 0) != 0;
    });
  } else if (warp < POOL_EPI_WARP0) {
    reg_dec<POOL_REGS_CTRL>();
  if (warp == 0) {
    // ---------------- TMA producer ----------------
    const int layer = a.layer_begin + slab;
    if (lane == 0) {
      mbar_expect_tx(smem_u32(&bars->q_full), (uint32_t)n_qblk * NH * HALF_BYTES);
      const int wrow = slab * a.sum_win + w0 + w_begin;
      for (int qb = 0; qb < n_qblk; ++qb)
        for (int hf = 0; hf < NH; ++hf)
          tma_load_3d(q_smem + (qb >> 1) * 2 * QBLK_BYTES + hf * QBLK_BYTES + (qb & 1) * HALF_BYTES, &qmap,
                      smem_u32(&bars->q_full), hf * 64, h * a.group, wrow + qb * (128 / G));
    }
    if (ta.k5) k_tile_producer<true, NH>(&kmap, a, bars, k_smem, S, r, h, layer, L, t_begin, n_tiles, lane, abort_flag, 0, 2, ta.wait_cycles, ta.stall_tile);
    else k_tile_producer<false, NH>(&kmap, a, bars, k_smem, S, r, h, layer, L, t_begin, n_tiles, lane, abort_flag, 0, 2, ta.wait_cycles, ta.stall_tile);
    if (lane == 0) bars->prod_done = 1;
  } else if (warp == POOL_PRODUCER2) {
    const int layer = a.layer_begin + slab;
    if (ta.k5) k_tile_producer<true, NH>(&kmap, a, bars, k_smem, S, r, h, layer, L, t_begin, n_tiles, lane, abort_flag, 1, 2, ta.wait_cycles, ta.stall_tile);
    else k_tile_producer<false, NH>(&kmap, a, bars, k_smem, S, r, h, layer, L, t_begin, n_tiles, lane, abort_flag, 1, 2, ta.wait_cycles, ta.stall_tile);
  } else {
    // ---------------- MMA issuers: D[key, row] = K Q^T ----------------
    // Two warps, one per accumulator: warp 1 issues the even jobs, warp 2 the odd ones.  Issuing costs the
    // issuing thread about 50 cycles per tcgen05.mma and 80 per tcgen05.commit, and the barrier
    // handshakes come on top; with one issuer that time showed up as idle time of the tensor pipe.
    // The whole warp runs the loop (waits stay warp-uniform); one elected lane issues.  Every issuer
    // waits for every K tile and releases it (tcgen05.commit after its last job of the tile, or a plain
    // arrive when it had none), so a stage is refilled only when both are done with it.
    const int mw = warp - 1;
    const uint64_t kdesc0 = smem_desc_sw128(k_smem);
    const uint64_t qdesc0 = smem_desc_sw128(q_smem);
    // MMA width of each row chunk: its live rows rounded up to 16 (a decode-step update has only G)
    const int n0 = rows <= 256 ? max(16, (rows + 15) & ~15) : 256;
    const int n1 = max(16, (rows - 256 + 15) & ~15);
    const uint32_t idesc_c[2] = {idesc_bf16(128, n0), idesc_bf16(128, n1)};
    const uint32_t full_bar = smem_u32(&bars->tmem_full[mw]), empty_bar = smem_u32(&bars->tmem_empty[mw]);
    bool ok = mbar_wait_warp(smem_u32(&bars->q_full), 0, abort_flag, ta.wait_cycles);
    int s = 0, job = 0;
    uint32_t kpar = 0, epar = 1u;                  // parity to wait for on tmem_empty[mw] (a fresh barrier passes with 1)
    const bool leader = elect_one();
    for (int it = 0; ok && it < n_tiles; ++it) {
      ok = mbar_wait_warp(smem_u32(&bars->k_full[s]), kpar, abort_flag, ta.wait_cycles);
      if (!ok) break;
      tc_fence_after();
      const uint64_t adesc_s = kdesc0 + (uint64_t)((s * KTILE_BYTES) >> 4);
      bool mine = false;
      for (int rc = 0; rc < n_rc; ++rc, ++job) {
        if ((job & 1) != mw) continue;
        ok = mbar_wait_warp(empty_bar, epar, abort_flag, ta.wait_cycles);
        if (!ok) break;
        epar ^= 1u;
        tc_fence_after();
        if (leader) {
          const uint64_t bdesc_c = qdesc0 + (uint64_t)((rc * 2 * QBLK_BYTES) >> 4);
#pragma unroll
          for (int kk = 0; kk < 4 * NH; ++kk)
            umma_bf16(tmem_base + mw * 256, adesc_s + (uint64_t)(((kk >> 2) * HALF_BYTES + (kk & 3) * 32) >> 4),
                      bdesc_c + (uint64_t)(((kk >> 2) * QBLK_BYTES + (kk & 3) * 32) >> 4), idesc_c[rc], kk > 0 ? 1u : 0u);
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
    __syncwarp();
    if (leader) umma_commit(smem_u32(&bars->drained[mw]));
    __syncwarp();
    // (a tear-down wait: it does not end early because another role gave up)
    mbar_wait_warp(smem_u32(&bars->drained[mw]), 0, nullptr, ok ? ta.wait_cycles : DRAIN_LIMIT_CYCLES);
    __syncwarp();
  }
  } else {
    // ---------------- epilogue: one key per thread ----------------
    reg_inc<POOL_REGS_EPI>();
    // The two warpgroups take alternate jobs whole, so they are one job apart and one folds while the other
    // waits for tensor memory (with both on every job, half the columns each, they ran in lockstep and the
    // sub-partitions idled through every wait: 5.25 against 5.0 ms at the bench shape, 0.57 against 0.50
    // at 32K x 1).  A job of more than 128 live rows is taken in two steps of 128 columns, the registers a
    // thread has for it, and the accumulator goes back to its MMA warp when the second step is in
    // registers.  With two row chunks per key tile a warpgroup always gets the same chunk; warpgroup 1
    // hands its sum of a tile to warpgroup 0 through shared memory, which picks it up one job later, so
    // neither waits for the other.
    const int wg = (warp - POOL_EPI_WARP0) >> 2;
    const int quarter = warp & 3;                 // TMEM lane quarter this warp may read
    const float c = a.scale_log2;
    // divisor of the mean: this call's W action tokens, plus, in the streaming form, the n already folded in (the
    // first row group of a window forms (n Out + S) / (n + W) in store_pooled, later row groups add their S / (n + W))
    const float inv_w = 1.0f / (float)(W + (a.acc_steps != nullptr ? a.acc_steps[r] : 0));
    float* out = a.score_out + ((int64_t)slab * Hkv + h) * a.sum_tok + a.tok_indptr[r];
    const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    float acc = 0.f;
    if (whole) {
      bool pending = false;
      float acc_prev = 0.f;
      int key_prev = 0;
      uint32_t par_prev = 0;
      bool ok = true;
      // what does not change from job to job: a warpgroup always has the same accumulator and row chunk
      const int b = wg;
      const int rc = (n_rc == 2) ? wg : 0;
      const uint32_t tq = taddr + b * 256;
      const int n_cg_job = (min(rows, rc * 256 + 256) - rc * 256 + 31) / 32;       // 32-column groups with live rows: 1..8
      const float* nl = nlse + rc * 256;
      const int wf = w_begin + (rc * 256) / G;
      const uint32_t full_bar = smem_u32(&bars->tmem_full[b]), empty_bar = smem_u32(&bars->tmem_empty[b]);
      int it = (n_rc == 2) ? 0 : wg;
      const int it_step = (n_rc == 2) ? 1 : 2;
      int key = (t_begin + it) * TK + quarter * 32 + lane;
      uint32_t fpar = 0;
      for (int job = wg; job < n_jobs; job += 2, it += it_step, key += it_step * TK, fpar ^= 1u) {
        const int w_min = a.causal ? max(0, key - lw) : 0;
        const int w_end = win > 0 ? (a.causal ? min(W, key - lw + win) : (key >= L - win ? W : 0)) : W;
        if (!mbar_wait_warp(full_bar, fpar, abort_flag, ta.wait_cycles)) { ok = false; break; }
        tc_fence_after();
        {
          float v[2][64];
          // columns [0, 128)
          tmem_ld64(tq, v[0]);
          if (n_cg_job > 2) tmem_ld64(tq + 64, v[1]);
          tmem_ld_wait();
          if (n_cg_job <= 4) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar);
          }
          pool_fold64<G>(v[0], nl, wf, w_min, w_end, c, acc);
          if (n_cg_job > 2) pool_fold64<G>(v[1], nl + 64, wf + 64 / G, w_min, w_end, c, acc);
          if (n_cg_job > 4) {
            // columns [128, 256)
            tmem_ld64(tq + 128, v[0]);
            if (n_cg_job > 6) tmem_ld64(tq + 192, v[1]);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar);
            pool_fold64<G>(v[0], nl + 128, wf + 128 / G, w_min, w_end, c, acc);
            if (n_cg_job > 6) pool_fold64<G>(v[1], nl + 192, wf + 192 / G, w_min, w_end, c, acc);
          }
        }
        if (n_rc == 1) {
          if (key < L) { if (row_begin > 0) out[key] += acc * inv_w; else store_pooled(a, r, out + key, acc, acc * inv_w, W); }
          acc = 0.f;
          continue;
        }
        if (wg == 1) {
          if (!mbar_wait_warp(smem_u32(&bars->part_empty), ((uint32_t)it & 1u) ^ 1u, abort_flag, ta.wait_cycles)) { ok = false; break; }
          bars->exch[quarter * 32 + lane] = acc;
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&bars->part_full));
        } else {
          if (pending) {
            if (!mbar_wait_warp(smem_u32(&bars->part_full), par_prev, abort_flag, ta.wait_cycles)) { ok = false; break; }
            acc_prev += bars->exch[quarter * 32 + lane];
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars->part_empty));
            if (key_prev < L) {
              if (row_begin > 0) out[key_prev] += acc_prev * inv_w;
              else store_pooled(a, r, out + key_prev, acc_prev, acc_prev * inv_w, W);
            }
          }
          pending = true;
          acc_prev = acc;
          key_prev = key;
          par_prev = (uint32_t)it & 1u;
        }
        acc = 0.f;
      }
      if (ok && pending && mbar_wait_warp(smem_u32(&bars->part_full), par_prev, abort_flag, ta.wait_cycles)) {
        acc_prev += bars->exch[quarter * 32 + lane];
        if (key_prev < L) {
          if (row_begin > 0) out[key_prev] += acc_prev * inv_w;
          else store_pooled(a, r, out + key_prev, acc_prev, acc_prev * inv_w, W);
        }
      }
    } else {
      // at most 128 live rows: one row chunk per key tile, a job is a tile
      for (int job = wg; job < n_jobs; job += 2) {
        const int b = job & 1;
        const int key = (t_begin + job) * TK + quarter * 32 + lane;
        const int w_min = a.causal ? max(0, key - lw) : 0;
        const int w_end = win > 0 ? (a.causal ? min(W, key - lw + win) : (key >= L - win ? W : 0)) : W;
        if (!mbar_wait_warp(smem_u32(&bars->tmem_full[b]), (uint32_t)(job >> 1) & 1u, abort_flag, ta.wait_cycles)) break;
        tc_fence_after();
        const int n_cg = (rows + 31) / 32;
        pool_job<G>(taddr + b * 256, nlse, n_cg, w_begin, w_min, w_end, c, acc, smem_u32(&bars->tmem_empty[b]), lane);
        if (key < L) { if (row_begin > 0) out[key] += acc * inv_w; else store_pooled(a, r, out + key, acc, acc * inv_w, W); }
        acc = 0.f;
      }
    }
  }
  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (warp == 0 && lane == 0 && *abort_flag) {
    report(a.status, ACTKV_E_TIMEOUT, u, kchunk);
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
