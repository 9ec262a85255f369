// LSE pass of the tensor-core score path (Section 7.1, LSE equation).
#pragma once

#include "tc_common.cuh"

namespace actkv {
namespace tc {

// ---------------------------------------------------------------------------------------------
// LSE pass

constexpr int LSE_EPI_WARPS = 8;
constexpr int LSE_THREADS = (2 + LSE_EPI_WARPS) * 32;

__global__ void __launch_bounds__(LSE_THREADS, 1)
score_tc_lse_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap qmap, const TcArgs ta) {
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
  const int key_begin = chunk * LSE_CHUNK;
  if (key_begin >= L || rg * 256 >= rows) return;
  if (W <= 0 || (a.causal && W > L)) {
    if (threadIdx.x == 0 && chunk == 0 && rg == 0) report(a.status, ACTKV_E_INVALID, r, W);
    return;
  }
  const int n_mb = min(2, (rows - rg * 256 + 127) / 128);
  const int t_begin = key_begin / TK;
  const int t_end = min((L + TK - 1) / TK, t_begin + LSE_CHUNK / TK);
  const int n_tiles = t_end - t_begin;
  const int S = ta.n_stages;

  const uint32_t smem_base = smem_u32(smem);
  const uint32_t q_smem = smem_base;                               // 2 x 32 KB
  const uint32_t k_smem = smem_base + 2 * QBLK_BYTES;              // S x 32 KB
  Barriers* bars = reinterpret_cast<Barriers*>(smem + 2 * QBLK_BYTES + (size_t)S * KTILE_BYTES);
  volatile int* abort_flag = &bars->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if ((smem_base & 1023u) != 0) {                                  // swizzled tiles need 1024-byte alignment
    if (threadIdx.x == 0) report(a.status, ACTKV_E_CUDA, -2, (int32_t)smem_base);
    return;
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(smem_u32(&bars->k_full[s]), 1); mbar_init(smem_u32(&bars->k_empty[s]), 1); }
    mbar_init(smem_u32(&bars->q_full), 1);
    for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&bars->tmem_full[b]), 1); mbar_init(smem_u32(&bars->tmem_empty[b]), LSE_EPI_WARPS); }
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

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    const int n_lp = (L + a.pool.page_size - 1) / a.pool.page_size;
    const int layer = a.layer_begin + slab;
    if (lane == 0) {
      mbar_expect_tx(smem_u32(&bars->q_full), (uint32_t)n_mb * QBLK_BYTES);
      const int wrow = slab * a.sum_win + w0 + (rg * 256) / G;
      for (int mb = 0; mb < n_mb; ++mb)
        for (int hf = 0; hf < 2; ++hf)
          tma_load_3d(q_smem + mb * QBLK_BYTES + hf * HALF_BYTES, &qmap, smem_u32(&bars->q_full), hf * 64, h * G,
                      wrow + mb * (128 / G));
    }
    int32_t pid = (lane < 8) ? page_for_tile(a.tab, a.pool.n_pages, r, t_begin * 8 + lane, n_lp, a.status) : 0;
    for (int it = 0; it < n_tiles; ++it) {
      const int s = it % S;
      const uint32_t ph = (uint32_t)(it / S) & 1u;
      int32_t pid_next = 0;
      if (lane < 8 && it + 1 < n_tiles)
        pid_next = page_for_tile(a.tab, a.pool.n_pages, r, (t_begin + it + 1) * 8 + lane, n_lp, a.status);
      int ok = 1;
      if (lane == 0) {
        ok = mbar_wait(smem_u32(&bars->k_empty[s]), ph ^ 1u, abort_flag) ? 1 : 0;
        if (ok) mbar_expect_tx(smem_u32(&bars->k_full[s]), KTILE_BYTES);
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane < 8) {
        const uint32_t dst = k_smem + s * KTILE_BYTES + lane * 2048;
        tma_load_4d(dst, &kmap, smem_u32(&bars->k_full[s]), 0, h, pid * 16, layer);
        tma_load_4d(dst + HALF_BYTES, &kmap, smem_u32(&bars->k_full[s]), 64, h, pid * 16, layer);
      }
      pid = pid_next;
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16(128, 128);
      bool ok = mbar_wait(smem_u32(&bars->q_full), 0, abort_flag);
      for (int it = 0; ok && it < n_tiles; ++it) {
        const int s = it % S, b = it & 1;
        ok = mbar_wait(smem_u32(&bars->k_full[s]), (uint32_t)(it / S) & 1u, abort_flag);
        if (!ok) break;
        ok = mbar_wait(smem_u32(&bars->tmem_empty[b]), ((uint32_t)(it >> 1) & 1u) ^ 1u, abort_flag);
        if (!ok) break;
        tc_fence_after();
        for (int mb = 0; mb < n_mb; ++mb) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (kk >> 2) * HALF_BYTES + (kk & 3) * 32;
            umma_bf16(tmem_base + b * 256 + mb * 128, smem_desc_sw128(q_smem + mb * QBLK_BYTES + off),
                      smem_desc_sw128(k_smem + s * KTILE_BYTES + off), idesc, kk > 0 ? 1u : 0u);
          }
        }
        umma_commit(smem_u32(&bars->k_empty[s]));
        umma_commit(smem_u32(&bars->tmem_full[b]));
      }
      // drain: every MMA issued above has completed before TMEM is freed
      umma_commit(smem_u32(&bars->drained));
      mbar_wait(smem_u32(&bars->drained), 0, abort_flag, ok ? WAIT_LIMIT_NS : DRAIN_LIMIT_NS);
    }
    __syncwarp();                                  // lanes 1..31 wait here for the issuing lane
  } else {
    // ---------------- epilogue: one row per thread ----------------
    const int ew = warp - 2;                       // 0..7
    const int mb = ew >> 2;                        // warps 2..5 -> block 0, 6..9 -> block 1
    const int quarter = warp & 3;                  // TMEM lanes this warp may read
    const int n = rg * 256 + mb * 128 + quarter * 32 + lane;      // row within the unit
    const bool row_ok = (mb < n_mb) && n < rows;
    const int w = n / G;
    const int jmax = a.causal ? (L - W + w) : (L - 1);            // last key this row sees
    const float c = a.scale_log2;
    float m = -INFINITY, sum = 0.f;
    bool ok = true;
    for (int it = 0; it < n_tiles; ++it) {
      const int b = it & 1;
      ok = mbar_wait(smem_u32(&bars->tmem_full[b]), (uint32_t)(it >> 1) & 1u, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const int tile_start = (t_begin + it) * TK;
      int n_valid = min(jmax, L - 1) - tile_start + 1;
      n_valid = row_ok ? max(0, min(TK, n_valid)) : 0;
      const bool warp_has_work = __any_sync(0xffffffffu, n_valid > 0) && (mb < n_mb);
      if (warp_has_work) {
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * 256 + mb * 128;
#pragma unroll 1
        for (int cg = 0; cg < TK / 32; ++cg) {
          float v[32];
          tmem_ld32(taddr + cg * 32, v);
          tmem_ld_wait();
          const int nv = n_valid - cg * 32;       // valid columns of this group for this row
          if (nv >= 32) {
            float gm = v[0];
#pragma unroll
            for (int i = 1; i < 32; ++i) gm = fmaxf(gm, v[i]);
            if (gm > m) { sum *= exp2f((m - gm) * c); m = gm; }     // m = -inf: sum is 0, 0 * 0 stays 0
            const float mc = m * c;
#pragma unroll
            for (int i = 0; i < 32; ++i) sum += exp2f(fmaf(v[i], c, -mc));
          } else if (nv > 0) {
            float gm = -INFINITY;
#pragma unroll
            for (int i = 0; i < 32; ++i) gm = fmaxf(gm, i < nv ? v[i] : -INFINITY);
            if (gm > m) { sum = (m == -INFINITY) ? 0.f : sum * exp2f((m - gm) * c); m = gm; }
            const float mc = m * c;
#pragma unroll
            for (int i = 0; i < 32; ++i) sum += (i < nv) ? exp2f(fmaf(v[i], c, -mc)) : 0.f;
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->tmem_empty[b]));
    }
    if (ok && row_ok) {
      // (-inf, 0) when the row saw no key of this chunk
      a.partials[((int64_t)u * a.n_chunks + chunk) * a.rows_max + n] = make_float2(m == -INFINITY ? m : m * c, sum);
    }
  }
  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
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
