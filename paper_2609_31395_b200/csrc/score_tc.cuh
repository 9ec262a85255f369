// Tensor-core path of actkv_score for sm_100a: tcgen05.mma with TMEM accumulators, operands
// staged by TMA (cp.async.bulk.tensor, 128-byte swizzle) straight from the paged pool through the
// block table, one TMA box per (page, half of the head dimension).
//
// Two kernels, both warp-specialised (warp 0: TMA producer, warp 1: MMA issuer + TMEM owner,
// the other warps: epilogue reading TMEM with tcgen05.ld):
//
//  * LSE pass (Section 7.1, LSE equation).  D[row, key] = Q K^T with the window x group rows on
//    the TMEM lanes, so every epilogue thread owns one row and keeps its running (max, sum of
//    exp2) in registers: no shuffles.  A CTA covers 256 rows x one chunk of LSE_CHUNK keys, two
//    128x128 accumulators double-buffered in the 512 TMEM columns.
//  * Pooled-score pass (Section 7.1 recovery identity, Algorithm 3 steps 3-5).  The transposed
//    product D[key, row] = K Q^T with the keys on the lanes and row = w*G + g on the columns, so
//    the max over the GQA group and the sum over the action tokens run inside one thread.  Because
//    exp is monotone the max over the group is taken on (s - lse) BEFORE the exp: W exps per key
//    instead of W*G.
//
// Every wait on an mbarrier is bounded (wall-clock limit); on give-up the kernel records
// ACTKV_E_TIMEOUT in the status word, every role leaves its loop, outstanding MMAs are drained,
// TMEM is freed and the CTA returns.
#pragma once

#include <cuda.h>
#include <cstdlib>

#include "score_fma.cuh"

namespace actkv {
namespace tc {

constexpr int TK = 128;                      // keys per tile
constexpr int HD = 128;                      // head dim
constexpr uint32_t KTILE_BYTES = TK * HD * 2;        // 32 KB: [2 halves][128 keys][64 bf16]
constexpr uint32_t HALF_BYTES = TK * 64 * 2;         // 16 KB
constexpr uint32_t QBLK_BYTES = 128 * HD * 2;        // 32 KB per 128 rows
constexpr int MAX_ROWS = 512;                // window x group rows (padded to 128) held in smem
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;    // bounded waits give up after 2 s
constexpr uint64_t DRAIN_LIMIT_NS = 50000000ull;     // waits while tearing down after a give-up

// ---------------------------------------------------------------------------------------------
// PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when another role already gave up or the limit passed (then the
// abort flag is raised so that every role stops).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          uint64_t limit_ns = WAIT_LIMIT_NS) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (globaltimer_ns() - t0 > limit_ns) {
      *abort_flag = 1;
      return false;
    }
  }
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]^T, bf16 x bf16 -> fp32
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptor: K-major tile, 128-byte swizzle, rows of 64 bf16 (128 B), eight-row
// groups 1024 B apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFF) >> 4);            // start address
  d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset: 8 rows x 128 B
  d |= (uint64_t)1 << 46;                            // descriptor version (sm_100)
  d |= (uint64_t)2 << 61;                            // SWIZZLE_128B
  return d;
}
__host__ __device__ constexpr uint32_t idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

struct TcArgs {
  ScoreArgs a;
  int32_t tiles_per_cta;     // pooled-score pass: key tiles per CTA
  int32_t n_kchunks;         // pooled-score pass: CTAs per unit
  int32_t n_rg;              // LSE pass: 256-row groups per unit (1 or 2)
  int32_t n_stages;          // K stages in shared memory
};

// Barrier block at the tail of dynamic shared memory.
struct Barriers {
  uint64_t k_full[8];
  uint64_t k_empty[8];
  uint64_t q_full;
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t drained;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ int32_t page_for_tile(const TablesView& tab, int32_t n_pages, int r, int lp, int n_lp,
                                                 int32_t* status) {
  // logical pages past the end of the request re-read its last page (their keys are masked later)
  lp = min(lp, n_lp - 1);
  return checked_page(tab, n_pages, r, lp, status);
}

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

// ---------------------------------------------------------------------------------------------
// Pooled-score pass

constexpr int POOL_EPI_WARPS = 4;
constexpr int POOL_THREADS = (2 + POOL_EPI_WARPS) * 32;

template <int G>
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
  const int rows = W * G;
  const int t_begin = kchunk * ta.tiles_per_cta;
  if (t_begin * TK >= L) return;
  if (W <= 0 || (a.causal && W > L)) {
    if (threadIdx.x == 0 && kchunk == 0) report(a.status, ACTKV_E_INVALID, r, W);
    return;
  }
  const int t_end = min((L + TK - 1) / TK, t_begin + ta.tiles_per_cta);
  const int n_tiles = t_end - t_begin;
  const int rows_pad = (rows + 127) & ~127;               // <= MAX_ROWS (checked by the host)
  const int n_rc = (rows_pad + 255) / 256;                // 256-row column chunks per key tile
  const int n_qblk = rows_pad / 128;
  const int S = ta.n_stages;

  const uint32_t smem_base = smem_u32(smem);
  const uint32_t q_bytes = (uint32_t)n_rc * 2 * QBLK_BYTES;     // per chunk: [2 halves][256 rows x 128 B]
  const uint32_t q_smem = smem_base;
  const uint32_t k_smem = smem_base + q_bytes;
  float* lse2 = reinterpret_cast<float*>(smem + q_bytes + (size_t)S * KTILE_BYTES);       // [rows_pad] log2 units
  Barriers* bars = reinterpret_cast<Barriers*>(reinterpret_cast<uint8_t*>(lse2) + MAX_ROWS * 4);
  volatile int* abort_flag = &bars->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if ((smem_base & 1023u) != 0) {
    if (threadIdx.x == 0) report(a.status, ACTKV_E_CUDA, -2, (int32_t)smem_base);
    return;
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(smem_u32(&bars->k_full[s]), 1); mbar_init(smem_u32(&bars->k_empty[s]), 1); }
    mbar_init(smem_u32(&bars->q_full), 1);
    for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&bars->tmem_full[b]), 1); mbar_init(smem_u32(&bars->tmem_empty[b]), POOL_EPI_WARPS); }
    mbar_init(smem_u32(&bars->drained), 1);
    bars->abort_flag = 0;
    fence_barrier_init();
  }
  {
    // LSE of every row in log2 units; padded rows get +inf so that s*c - lse = -inf drops out of the max
    const float* lse_base = a.lse + ((int64_t)slab * a.sum_win + w0) * a.n_q_heads + h * G;
    for (int n = threadIdx.x; n < rows_pad; n += blockDim.x)
      lse2[n] = (n < rows) ? lse_base[(int64_t)(n / G) * a.n_q_heads + (n % G)] * kLog2e : INFINITY;
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
      mbar_expect_tx(smem_u32(&bars->q_full), (uint32_t)n_qblk * QBLK_BYTES);
      const int wrow = slab * a.sum_win + w0;
      for (int qb = 0; qb < n_qblk; ++qb)
        for (int hf = 0; hf < 2; ++hf)
          tma_load_3d(q_smem + (qb >> 1) * 2 * QBLK_BYTES + hf * QBLK_BYTES + (qb & 1) * HALF_BYTES, &qmap,
                      smem_u32(&bars->q_full), hf * 64, h * G, wrow + qb * (128 / G));
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
    // ---------------- MMA issuer: D[key, row] = K Q^T ----------------
    if (lane == 0) {
      bool ok = mbar_wait(smem_u32(&bars->q_full), 0, abort_flag);
      int job = 0;
      for (int it = 0; ok && it < n_tiles; ++it) {
        const int s = it % S;
        ok = mbar_wait(smem_u32(&bars->k_full[s]), (uint32_t)(it / S) & 1u, abort_flag);
        for (int rc = 0; ok && rc < n_rc; ++rc, ++job) {
          const int b = job & 1;
          ok = mbar_wait(smem_u32(&bars->tmem_empty[b]), ((uint32_t)(job >> 1) & 1u) ^ 1u, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const int ncols = min(256, rows_pad - rc * 256);
          const uint32_t idesc = idesc_bf16(128, ncols);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint64_t adesc = smem_desc_sw128(k_smem + s * KTILE_BYTES + (kk >> 2) * HALF_BYTES + (kk & 3) * 32);
            const uint64_t bdesc = smem_desc_sw128(q_smem + rc * 2 * QBLK_BYTES + (kk >> 2) * QBLK_BYTES + (kk & 3) * 32);
            umma_bf16(tmem_base + b * 256, adesc, bdesc, idesc, kk > 0 ? 1u : 0u);
          }
          umma_commit(smem_u32(&bars->tmem_full[b]));
        }
        if (ok) umma_commit(smem_u32(&bars->k_empty[s]));
      }
      umma_commit(smem_u32(&bars->drained));
      mbar_wait(smem_u32(&bars->drained), 0, abort_flag, ok ? WAIT_LIMIT_NS : DRAIN_LIMIT_NS);
    }
    __syncwarp();                                  // lanes 1..31 wait here for the issuing lane
  } else {
    // ---------------- epilogue: one key per thread ----------------
    const int quarter = warp & 3;
    const float c = a.scale_log2;
    const float inv_w = 1.0f / (float)W;
    float* out = a.score_out + ((int64_t)slab * Hkv + h) * a.sum_tok + a.tok_indptr[r];
    bool ok = true;
    int job = 0;
    for (int it = 0; ok && it < n_tiles; ++it) {
      const int key = (t_begin + it) * TK + quarter * 32 + lane;
      // causal: row w sees key j iff j <= L - W + w  <=>  w >= j - (L - W)
      const int w_min = a.causal ? max(0, key - (L - W)) : 0;
      float acc = 0.f;
      for (int rc = 0; rc < n_rc; ++rc, ++job) {
        const int b = job & 1;
        ok = mbar_wait(smem_u32(&bars->tmem_full[b]), (uint32_t)(job >> 1) & 1u, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * 256;
        const int n_cg = (min(rows, rc * 256 + 256) - rc * 256 + 31) / 32;    // 32-column groups with live rows
#pragma unroll 1
        for (int cg = 0; cg < n_cg; ++cg) {
          float v[32];
          tmem_ld32(taddr + cg * 32, v);
          tmem_ld_wait();
          const int n0 = rc * 256 + cg * 32;
          const float4* l4 = reinterpret_cast<const float4*>(lse2 + n0);
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4) {
            const float4 l = l4[q4];
            v[q4 * 4 + 0] = fmaf(v[q4 * 4 + 0], c, -l.x);
            v[q4 * 4 + 1] = fmaf(v[q4 * 4 + 1], c, -l.y);
            v[q4 * 4 + 2] = fmaf(v[q4 * 4 + 2], c, -l.z);
            v[q4 * 4 + 3] = fmaf(v[q4 * 4 + 3], c, -l.w);
          }
          constexpr int WPG = 32 / G;                 // window rows per 32-column group
#pragma unroll
          for (int i = 0; i < WPG; ++i) {
            float mx = v[i * G];
#pragma unroll
            for (int g = 1; g < G; ++g) mx = fmaxf(mx, v[i * G + g]);
            const int w = n0 / G + i;
            acc += (w < W && w >= w_min) ? exp2f(mx) : 0.f;
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->tmem_empty[b]));
      }
      if (ok && key < L) out[key] = acc * inv_w;
    }
  }
  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (warp == 0 && lane == 0 && *abort_flag) {
    report(a.status, ACTKV_E_TIMEOUT, u, kchunk);
    for (int s = 0; s < S; ++s) mbar_wait(smem_u32(&bars->k_full[s]), 0, abort_flag, DRAIN_LIMIT_NS / 8);
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------------------------
// host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return (EncodeTiledFn)p;
  }();
  return fn;
}

inline bool make_maps(const actkv_pool_t* pool, const void* q, int nls, int sum_win, int n_q_heads, int G,
                      CUtensorMap* kmap, CUtensorMap* qmap) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  {
    // K half of the pool: [layer][slot (page*16 + s)][head][128]
    cuuint64_t dims[4] = {(cuuint64_t)HD, (cuuint64_t)pool->n_kv_heads, (cuuint64_t)pool->n_pages * pool->page_size,
                          (cuuint64_t)pool->n_layers};
    cuuint64_t strides[3] = {(cuuint64_t)pool->stride_head * 2, (cuuint64_t)pool->stride_slot * 2,
                             (cuuint64_t)pool->stride_layer * 2};
    cuuint32_t box[4] = {64, 1, 16, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    if (enc(kmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, pool->base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  {
    // q: [slab*sum_win + w][q head][128]; a box is (64 dims, the G heads of one group, 128/G window rows)
    cuuint64_t dims[3] = {(cuuint64_t)HD, (cuuint64_t)n_q_heads, (cuuint64_t)nls * sum_win};
    cuuint64_t strides[2] = {(cuuint64_t)HD * 2, (cuuint64_t)n_q_heads * HD * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)(128 / G)};
    cuuint32_t es[3] = {1, 1, 1};
    if (enc(qmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  return true;
}

}  // namespace tc

// The tensor-core path takes: page 16, head_dim 128, packed [slot][head][dim] pages, 128-byte aligned
// base, power-of-two group size <= 32, 64 <= window x group rows <= 512, positive softmax scale.
inline bool score_tc_supported(const actkv_pool_t* p, int G, int max_win, float sm_scale, const void* q) {
  if (p->page_size != 16 || p->head_dim != 128) return false;
  if (p->stride_head != 128 || p->stride_slot != (int64_t)p->n_kv_heads * 128 || p->stride_page != 16 * p->stride_slot)
    return false;
  if (((uintptr_t)p->base & 127) || ((uintptr_t)q & 127) || (p->stride_layer % 8) != 0) return false;
  if (G < 1 || G > 32 || (G & (G - 1)) != 0) return false;
  const int rows = max_win * G;
  if (rows < 64 || rows > tc::MAX_ROWS) return false;
  if (!(sm_scale > 0.f)) return false;
  if (getenv("ACTKV_FORCE_FMA") != nullptr) return false;
  return tc::encode_fn() != nullptr;
}

inline int score_tc_launch_lse(ScoreArgs& a, const actkv_pool_t* pool, int max_tok, int max_win, cudaStream_t s) {
  (void)max_tok;
  CUtensorMap kmap, qmap;
  if (!tc::make_maps(pool, a.q, a.n_layers_sub, a.sum_win, a.n_q_heads, a.group, &kmap, &qmap)) return ACTKV_E_CUDA;
  tc::TcArgs ta;
  ta.a = a;
  const int rows_pad = (max_win * a.group + 127) & ~127;
  ta.n_rg = (rows_pad + 255) / 256;
  ta.n_stages = 4;
  ta.tiles_per_cta = 0;
  ta.n_kchunks = 0;
  const int64_t units = (int64_t)a.n_layers_sub * a.pool.n_kv_heads * a.tab.n_req;
  const int64_t grid = units * ta.n_rg * a.n_chunks;
  if (grid > 0x7fffffffLL) return ACTKV_E_INVALID;
  const size_t smem = 2 * tc::QBLK_BYTES + (size_t)ta.n_stages * tc::KTILE_BYTES + sizeof(tc::Barriers);
  if (cudaFuncSetAttribute(tc::score_tc_lse_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return ACTKV_E_CUDA;
  tc::score_tc_lse_kernel<<<(unsigned)grid, tc::LSE_THREADS, smem, s>>>(kmap, qmap, ta);
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

template <int G>
inline int score_tc_launch_pool_g(const CUtensorMap& kmap, const CUtensorMap& qmap, const tc::TcArgs& ta, unsigned grid,
                                  size_t smem, cudaStream_t s) {
  if (cudaFuncSetAttribute(tc::score_tc_pool_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return ACTKV_E_CUDA;
  tc::score_tc_pool_kernel<G><<<grid, tc::POOL_THREADS, smem, s>>>(kmap, qmap, ta);
  ACTKV_CHECK_LAUNCH();
  return ACTKV_OK;
}

inline int score_tc_launch_score(ScoreArgs& a, const actkv_pool_t* pool, int max_tok, int max_win, cudaStream_t s) {
  CUtensorMap kmap, qmap;
  if (!tc::make_maps(pool, a.q, a.n_layers_sub, a.sum_win, a.n_q_heads, a.group, &kmap, &qmap)) return ACTKV_E_CUDA;
  tc::TcArgs ta;
  ta.a = a;
  const int rows_pad = (max_win * a.group + 127) & ~127;
  const int n_rc = (rows_pad + 255) / 256;
  const size_t q_bytes = (size_t)n_rc * 2 * tc::QBLK_BYTES;
  const size_t fixed = q_bytes + tc::MAX_ROWS * 4 + sizeof(tc::Barriers);
  int stages = (int)((232448 - fixed) / tc::KTILE_BYTES);
  if (stages > 6) stages = 6;
  if (stages < 2) return ACTKV_E_INVALID;
  ta.n_stages = stages;
  ta.n_rg = 0;
  const int64_t units = (int64_t)a.n_layers_sub * a.pool.n_kv_heads * a.tab.n_req;
  const int max_tiles = (max_tok + tc::TK - 1) / tc::TK;
  // enough CTAs to fill the 148 SMs a few times over, few enough that the Q load is amortised
  int64_t tpc = (units * max_tiles) / (148 * 8);
  if (tpc < 4) tpc = 4;
  if (tpc > 64) tpc = 64;
  ta.tiles_per_cta = (int)tpc;
  ta.n_kchunks = (max_tiles + ta.tiles_per_cta - 1) / ta.tiles_per_cta;
  const int64_t grid = units * ta.n_kchunks;
  if (grid > 0x7fffffffLL) return ACTKV_E_INVALID;
  const size_t smem = fixed + (size_t)stages * tc::KTILE_BYTES;
  switch (a.group) {
    case 1: return score_tc_launch_pool_g<1>(kmap, qmap, ta, (unsigned)grid, smem, s);
    case 2: return score_tc_launch_pool_g<2>(kmap, qmap, ta, (unsigned)grid, smem, s);
    case 4: return score_tc_launch_pool_g<4>(kmap, qmap, ta, (unsigned)grid, smem, s);
    case 8: return score_tc_launch_pool_g<8>(kmap, qmap, ta, (unsigned)grid, smem, s);
    case 16: return score_tc_launch_pool_g<16>(kmap, qmap, ta, (unsigned)grid, smem, s);
    case 32: return score_tc_launch_pool_g<32>(kmap, qmap, ta, (unsigned)grid, smem, s);
    default: return ACTKV_E_INVALID;
  }
}

}  // namespace actkv
