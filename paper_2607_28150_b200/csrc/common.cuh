// Shared host/device helpers of the smartgen kernels (argument checks, status word, small PTX wrappers).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "smartgen.h"

namespace sg {

constexpr int kNumSMs = 148;           // B200: 2 dies x 74 SMs; grids are sized in multiples of this
constexpr int kMaxBatchSmem = 1024;    // largest batch whose prefix arrays sg_score caches in shared memory

// last failed CUDA call on this host thread (sg_last_cuda_error)
extern thread_local int g_last_cuda_error;

inline sg_status cuda_fail(int err) {
  g_last_cuda_error = err;
  return SG_ERR_CUDA;
}

#define SG_CUDA_TRY(expr)                                        \
  do {                                                           \
    cudaError_t _e = (expr);                                     \
    if (_e != cudaSuccess) return ::sg::cuda_fail((int)_e);      \
  } while (0)

// Opt a kernel in to `bytes` of dynamic shared memory, once per device and call site (the setting is
// sticky per device, so later calls -- including calls made during stream capture -- skip the driver).
#define SG_ENSURE_SMEM(func, bytes)                                                                   \
  do {                                                                                                \
    static std::atomic<int> _sg_set[64];                                                              \
    int _sg_dev = 0;                                                                                  \
    SG_CUDA_TRY(cudaGetDevice(&_sg_dev));                                                             \
    if (_sg_dev < 0 || _sg_dev >= 64 || _sg_set[_sg_dev].load(std::memory_order_relaxed) < (bytes)) { \
      SG_CUDA_TRY(cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, (bytes)));  \
      if (_sg_dev >= 0 && _sg_dev < 64) _sg_set[_sg_dev].store((bytes), std::memory_order_relaxed);   \
    }                                                                                                 \
  } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Checks common to every call.  `need_window` also validates shape->window.
inline sg_status check_shape(const sg_shape* s, bool need_window) {
  if (!s || !s->cu_seqlens) return SG_ERR_INVALID;
  if (s->num_layers < 1 || s->batch < 1 || s->num_q_heads < 1 || s->num_kv_heads < 1) return SG_ERR_INVALID;
  if (s->total_tokens < 0 || s->max_seqlen < 0 || s->max_seqlen > s->total_tokens) return SG_ERR_INVALID;
  if (need_window && s->window < 1) return SG_ERR_INVALID;
  if (s->head_dim != 64 && s->head_dim != 128) return SG_ERR_UNSUPPORTED;
  if (s->num_q_heads % s->num_kv_heads != 0) return SG_ERR_UNSUPPORTED;
  if (s->num_q_heads / s->num_kv_heads > 16) return SG_ERR_UNSUPPORTED;
  if (s->cache_token_stride < s->head_dim || s->cache_head_stride < 0) return SG_ERR_INVALID;
  if ((s->cache_token_stride & 7) || (s->cache_head_stride & 7) || (s->cache_layer_stride & 7)) return SG_ERR_INVALID;
  if (!aligned16(s->cu_seqlens)) return SG_ERR_INVALID;
  return SG_OK;
}

__device__ __forceinline__ void raise(int32_t* dev_status, int code) {
  if (dev_status) atomicOr(dev_status, 1 << code);
}

// Largest b in [0, B) with prefix[b] <= x, for an ascending prefix array with prefix[0] = 0.
__device__ __forceinline__ int upper_segment(const int32_t* __restrict__ prefix, int B, int64_t x, int64_t mult = 1) {
  int lo = 0, hi = B;   // invariant: prefix[lo]*mult <= x, answer in [lo, hi)
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if ((int64_t)prefix[mid] * mult <= x) lo = mid; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

}  // namespace sg
