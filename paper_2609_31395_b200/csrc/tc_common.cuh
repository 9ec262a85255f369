// PTX wrappers, descriptors and shared structures of the tcgen05 / TMEM / TMA score kernels (sm_100a).
#pragma once

#include <cuda.h>

#include "compact_job.cuh"
#include "score_fma.cuh"

namespace actkv {
namespace tc {

constexpr int TK = 128;                      // keys per tile
constexpr int HD = 128;                      // head dim
constexpr uint32_t KTILE_BYTES = TK * HD * 2;        // 32 KB: [2 halves][128 keys][64 bf16]
constexpr uint32_t HALF_BYTES = TK * 64 * 2;         // 16 KB
constexpr uint32_t QBLK_BYTES = 128 * HD * 2;        // 32 KB per 128 rows
constexpr int MAX_ROWS = 512;                // window x group rows (padded to 128) one CTA handles
constexpr int MAX_ROWS_TOTAL = 4096;         // ... per unit: more than MAX_ROWS are taken in groups of MAX_ROWS
// Bounded waits are counted on the SM cycle counter (cheap to read, unlike the global nanosecond timer).  The
// counter runs at 2.1 GHz at most, so a limit of n cycles lasts at least n / 2.1 ns.
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;      // default limit of a wait: about two seconds
constexpr long long DRAIN_LIMIT_CYCLES = 100000000ll;      // waits while tearing down after a give-up: about 50 ms

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
// Non-blocking poll of a barrier phase.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait of ONE thread.  Returns false when another role already gave up or the limit passed (then the
// abort flag is raised so that every role stops).  abort_flag == nullptr: a wait of the tear-down path, which
// neither looks at the flag nor raises it and only ends on success or on its own limit.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit_cycles) {
  // try_wait parks the thread in hardware (no polling traffic on shared memory, which the MMA operand
  // fetch needs); measured the same or better than spinning on test_wait here.
#pragma unroll 1
  for (int i = 0; i < 64; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (abort_flag != nullptr && *abort_flag) return false;
    if (clock64() - t0 > limit_cycles) {
      if (abort_flag != nullptr) *abort_flag = 1;
      return false;
    }
  }
}
// The same wait called by all 32 lanes of a converged warp, with ONE answer for the warp: the callers go on
// to warp-collective instructions (tcgen05.ld, elect, __syncwarp) and must not split on a wait that some
// lanes saw complete and others gave up on.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit_cycles) {
  const bool ok = mbar_wait(bar, parity, abort_flag, limit_cycles);
  return __all_sync(0xffffffffu, ok);
}
// One lane of a converged warp (always the same one for a full mask).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
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
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
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
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr));
}
// N consecutive columns (a multiple of 4, at most 64) as a few power-of-two loads
template <int N>
__device__ __forceinline__ void tmem_ld_n(uint32_t taddr, float* v) {
  static_assert(N % 4 == 0 && N >= 0 && N <= 64, "column count");
  if constexpr (N >= 64) { tmem_ld64(taddr, v); }
  else if constexpr (N >= 32) { tmem_ld32(taddr, v); tmem_ld_n<N - 32>(taddr + 32, v + 32); }
  else if constexpr (N >= 16) { tmem_ld16(taddr, v); tmem_ld_n<N - 16>(taddr + 16, v + 16); }
  else if constexpr (N >= 8) { tmem_ld8(taddr, v); tmem_ld_n<N - 8>(taddr + 8, v + 8); }
  else if constexpr (N >= 4) { tmem_ld4(taddr, v); }
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 16 consecutive 32-bit columns of this thread's TMEM lane <- registers
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D[tmem] (+)= A[tmem] * B[smem desc]^T, bf16 x bf16 -> fp32, A = 128 rows x 16 bf16 packed in 8 columns
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// Register budget of a warpgroup (four consecutive warps, all of whose threads execute the instruction): the
// control and copy warpgroups hand registers back, the epilogue warpgroups take them.
template <uint32_t N>
__device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <uint32_t N>
__device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

// sm_100 arithmetic the epilogues lean on: packed two-lane fp32 FMA / add, three-input max.
__device__ __forceinline__ void ffma2(float& x0, float& x1, float a0, float a1, float b, float c0, float c1) {
  uint64_t ra, rb, rc, rd;                      // (x0, x1) = (a0, a1) * b + (c0, c1)
  asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a0), "f"(a1));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b), "f"(b));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rc) : "f"(c0), "f"(c1));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(rd) : "l"(ra), "l"(rb), "l"(rc));
  asm("mov.b64 {%0, %1}, %2;" : "=f"(x0), "=f"(x1) : "l"(rd));
}
__device__ __forceinline__ void ffma2v(float& x0, float& x1, float a0, float a1, float b0, float b1, float c0, float c1) {
  uint64_t ra, rb, rc, rd;                      // (x0, x1) = (a0, a1) * (b0, b1) + (c0, c1)
  asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a0), "f"(a1));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b0), "f"(b1));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rc) : "f"(c0), "f"(c1));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(rd) : "l"(ra), "l"(rb), "l"(rc));
  asm("mov.b64 {%0, %1}, %2;" : "=f"(x0), "=f"(x1) : "l"(rd));
}
__device__ __forceinline__ void fadd2(float& x0, float& x1, float a0, float a1) {
  uint64_t ra, rb, rd;                          // (x0, x1) += (a0, a1)
  asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(x0), "f"(x1));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(a0), "f"(a1));
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(rd) : "l"(ra), "l"(rb));
  asm("mov.b64 {%0, %1}, %2;" : "=f"(x0), "=f"(x1) : "l"(rd));
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
template <int N>
__device__ __forceinline__ float max_of(const float* v) {       // max of v[0..N), N a power of two
  if constexpr (N == 1) return v[0];
  else if constexpr (N == 2) return fmaxf(v[0], v[1]);
  else if constexpr (N == 4) return fmaxf(fmax3(v[0], v[1], v[2]), v[3]);
  else if constexpr (N == 8) return fmaxf(fmax3(fmax3(v[0], v[1], v[2]), fmax3(v[3], v[4], v[5]), v[6]), v[7]);
  else return fmaxf(max_of<N / 2>(v), max_of<N / 2>(v + N / 2));
}

// max of v[0..N) for any N >= 1, as a tree of three-input max
template <int N>
__device__ __forceinline__ float max_n(const float* v) {
  if constexpr (N == 1) return v[0];
  else if constexpr (N == 2) return fmaxf(v[0], v[1]);
  else if constexpr (N == 3) return fmax3(v[0], v[1], v[2]);
  else {
    constexpr int A = (N + 2) / 3, B = (N - A + 1) / 2, C = N - A - B;
    return fmax3(max_n<A>(v), max_n<B>(v + A), max_n<C>(v + A + B));
  }
}

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
  int32_t n_rg;              // LSE pass: groups of MAX_ROWS rows per unit (a grid dimension)
  int32_t row_begin;         // pooled-score pass: first row of this launch's row group (multiple of MAX_ROWS)
  int32_t n_stages;          // K stages in shared memory
  int32_t k5;                // K tensor map has five dimensions (pages that are not slot-major), else four
  CompactWs* copy_ws;        // pending compaction of another layer group whose copies this launch's spare warps
                             // take on (nullptr: none)
  int32_t stall_tile;        // fault-injection hook: the K-tile producers issue no tile from this one on (< 0: off)
  long long wait_cycles;     // limit of every bounded wait, in SM cycles
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

// The K-tile producers of both score kernels: producer p of P takes tiles p, p + P, ... of
// [t_begin, t_begin + n_tiles) of request r, head h, layer `layer` through the block table into the ring of S
// stages, one TMA box per (page, 64-dim half), one box per lane.  Pages of 16, 32, 64 or 128 tokens: a
// tile of 128 keys is ppt = 128 / page_size pages, a box page_size rows of 128 B.
// Measured on B200 (boxes of 16 rows x 128 B from random pages): one warp issuing a tile's 16 boxes from
// 8 lanes delivers a tile per 1950 cycles, from 16 lanes per 1570, two warps per 1235, four per 1180 (the
// memory system's rate).  Only the streaming update is bound by this.
// Page ids of four of the producer's tiles at a time, one per lane (lane / ppt = tile within the group,
// lane % ppt = page); the next group's ids are loaded while the current four tiles are being issued.
// K5: five-dimensional tensor map (pages that are not slot-major).
template <bool K5, int NH, class Bars>
__device__ __forceinline__ void k_tile_producer(const CUtensorMap* kmap, const ScoreArgs& a, Bars* bars, uint32_t k_smem,
                                                int S, int r, int h, int layer, int L, int t_begin, int n_tiles,
                                                int lane, volatile int* abort_flag, int p, int P, long long wait_cycles,
                                                int stall_tile) {
  const int ps = a.pool.page_size;
  const int ppt = TK / ps;                                      // pages per tile: 8, 4, 2 or 1
  const int lp_shift = 31 - __clz(ppt);                         // log2(ppt)
  const uint32_t box_bytes = (uint32_t)ps * 128u;
  const int n_lp = (L + ps - 1) / ps;
  const int n_mine = (n_tiles - p + P - 1) / P;                  // tiles p, p + P, ... below n_tiles
  const int g_tile = lane >> lp_shift, g_page = lane & (ppt - 1);            // this lane's slot in a group of four tiles
  int32_t pid = page_for_tile(a.tab, a.pool.n_pages, r, (t_begin + p + min(g_tile, 3) * P) * ppt + g_page, n_lp, a.status);
  int32_t pid_next = 0;
  for (int i = 0; i < n_mine; ++i) {
    const int it = p + i * P;
    if (stall_tile >= 0 && it >= stall_tile) break;       // injected fault: this and all later tiles never arrive
    const int s = it % S;
    const uint32_t ph = (uint32_t)(it / S) & 1u;
    if ((i & 3) == 0 && i + 4 < n_mine)
      pid_next = page_for_tile(a.tab, a.pool.n_pages, r, (t_begin + p + (i + 4 + min(g_tile, 3)) * P) * ppt + g_page, n_lp,
                               a.status);
    int ok = 1;
    if (lane == 0) {
      ok = mbar_wait(smem_u32(&bars->k_empty[s]), ph ^ 1u, abort_flag, wait_cycles) ? 1 : 0;
      if (ok) mbar_expect_tx(smem_u32(&bars->k_full[s]), NH * HALF_BYTES);
    }
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (!ok) break;
    // lane j < ppt NH: page j % ppt, half j / ppt of this tile
    const int32_t my_pid = __shfl_sync(0xffffffffu, pid, ((i & 3) << lp_shift) | (lane & (ppt - 1)));
    if (lane < ppt * NH) {
      const int half = lane >> lp_shift;
      const uint32_t dst = k_smem + s * KTILE_BYTES + half * HALF_BYTES + (lane & (ppt - 1)) * box_bytes;
      const uint32_t bar = smem_u32(&bars->k_full[s]);
      if constexpr (K5) tma_load_5d(dst, kmap, bar, half * 64, 0, h, my_pid, layer);
      else tma_load_4d(dst, kmap, bar, half * 64, h, my_pid * ps, layer);
    }
    if ((i & 3) == 3) pid = pid_next;
  }
}

}  // namespace tc
}  // namespace actkv
