// Shared device/host helpers of the ActKV CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <mutex>

#include "../../include/actkv.h"

// (a failed launch also drops the remembered launch attributes: after a device reset by the caller the kernels have
//  lost them, and the next call asks the driver again)
#define ACTKV_CHECK_LAUNCH()                                   \
  do {                                                         \
    if (cudaGetLastError() != cudaSuccess) {                   \
      ::actkv::forget_kernel_attrs();                          \
      return ACTKV_E_CUDA;                                     \
    }                                                          \
  } while (0)

namespace actkv {

// First device-detected error wins; later ones are dropped.
__device__ __forceinline__ void report(int32_t* status, int32_t code, int32_t where, int32_t what) {
  if (status == nullptr) return;
  if (atomicCAS(status, 0, code) == 0) {
    status[1] = where;
    status[2] = what;
  }
}

__device__ __forceinline__ bool status_set(const int32_t* status) {
  return status != nullptr && *((const volatile int32_t*)status) != 0;
}

// Plain-value copy of actkv_pool_t for kernel parameters.
struct PoolView {
  const __nv_bfloat16* base;
  int32_t n_layers, n_pages, page_size, n_kv_heads, head_dim;
  int64_t stride_layer, stride_kv, stride_page, stride_slot, stride_head;
};

struct TablesView {
  int32_t n_req, max_pages;
  int32_t* page_table;
  int32_t* seq_len;
  int32_t* free_list;
  int32_t* free_count;
};

inline PoolView make_view(const actkv_pool_t* p) {
  PoolView v;
  v.base = (const __nv_bfloat16*)p->base;
  v.n_layers = p->n_layers; v.n_pages = p->n_pages; v.page_size = p->page_size;
  v.n_kv_heads = p->n_kv_heads; v.head_dim = p->head_dim;
  v.stride_layer = p->stride_layer; v.stride_kv = p->stride_kv; v.stride_page = p->stride_page;
  v.stride_slot = p->stride_slot; v.stride_head = p->stride_head;
  return v;
}

inline TablesView make_view(const actkv_tables_t* t) {
  TablesView v;
  v.n_req = t->n_req; v.max_pages = t->max_pages; v.page_table = t->page_table;
  v.seq_len = t->seq_len; v.free_list = t->free_list; v.free_count = t->free_count;
  return v;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Per-kernel launch attributes are asked of the driver once per (kernel, device) and remembered: on steps of a few
// dozen microseconds the attribute calls of every launch were a tenth of the time.
struct KernelAttrCache {
  struct Entry { const void* fn; int dev; int smem; int regs; };
  static constexpr int kCap = 128;
  Entry e[kCap];
  int n = 0;
  std::mutex m;
  // entry of (fn, current device), created on first use; nullptr when the table is full or the device is unknown
  Entry* find(const void* fn) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    for (int i = 0; i < n; ++i)
      if (e[i].fn == fn && e[i].dev == dev) return &e[i];
    if (n >= kCap) return nullptr;
    e[n] = Entry{fn, dev, -1, -1};
    return &e[n++];
  }
};
inline KernelAttrCache& kernel_attr_cache() { static KernelAttrCache c; return c; }
inline void forget_kernel_attrs() {
  KernelAttrCache& c = kernel_attr_cache();
  std::lock_guard<std::mutex> lock(c.m);
  c.n = 0;
}

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) only when this kernel has not been given at least `bytes` yet.
template <class K>
inline cudaError_t ensure_dyn_smem(K kernel, size_t bytes) {
  KernelAttrCache& c = kernel_attr_cache();
  std::lock_guard<std::mutex> lock(c.m);
  KernelAttrCache::Entry* en = c.find(reinterpret_cast<const void*>(kernel));
  if (en != nullptr && en->smem >= (int)bytes) return cudaSuccess;
  const cudaError_t rc = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (rc == cudaSuccess && en != nullptr) en->smem = (int)bytes;
  return rc;
}

// Registers per thread the kernel was compiled to (cudaFuncGetAttributes, remembered); -1 on failure.
template <class K>
inline int kernel_num_regs(K kernel) {
  KernelAttrCache& c = kernel_attr_cache();
  std::lock_guard<std::mutex> lock(c.m);
  KernelAttrCache::Entry* en = c.find(reinterpret_cast<const void*>(kernel));
  if (en != nullptr && en->regs >= 0) return en->regs;
  cudaFuncAttributes fa;
  if (cudaFuncGetAttributes(&fa, kernel) != cudaSuccess) return -1;
  if (en != nullptr) en->regs = fa.numRegs;
  return fa.numRegs;
}

// Page id of logical page `lp` of request r; out-of-range ids are reported and replaced by 0.
__device__ __forceinline__ int32_t checked_page(const TablesView& t, int32_t n_pages, int32_t r,
                                                int32_t lp, int32_t* status) {
  int32_t id = t.page_table[(int64_t)r * t.max_pages + lp];
  if ((uint32_t)id >= (uint32_t)n_pages) {
    report(status, ACTKV_E_BADPAGE, r, id);
    id = 0;
  }
  return id;
}

// The same lookup for accesses that must not be redirected (the destination of a store, pages pushed on the
// free list): an out-of-range id is reported and -1 returned, the caller drops the access.
__device__ __forceinline__ int32_t page_or_neg(const TablesView& t, int32_t n_pages, int32_t r, int32_t lp,
                                               int32_t* status) {
  const int32_t id = t.page_table[(int64_t)r * t.max_pages + lp];
  if ((uint32_t)id >= (uint32_t)n_pages) {
    report(status, ACTKV_E_BADPAGE, r, id);
    return -1;
  }
  return id;
}

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

}  // namespace actkv
