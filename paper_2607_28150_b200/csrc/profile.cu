// Profile-based proactive selection on the device: selection counts S(e), block importance (Eq. 1), the
// transfer budget (Eq. 2, host arithmetic) and the KV mask left by the proactive transfer.  The global
// top-K_r over the L*M block importances is sg_select_topk on the flattened matrix.  Integer work plus one
// double division per block; every result is bit-exact against a scalar fp64 CPU restatement of the equations.
#include <math.h>

#include "common.cuh"

namespace sg {
namespace {

constexpr int kProfThreads = 256;

__global__ void __launch_bounds__(kProfThreads) profile_accumulate_kernel(const int32_t* __restrict__ kv_index,
                                                                           const int32_t* __restrict__ cu,
                                                                           const int32_t* __restrict__ cu_k, int32_t* counts,
                                                                           int32_t* dev_status, int B, int Hkv, int K_tot,
                                                                           int64_t T) {
  const int64_t i = (int64_t)blockIdx.x * kProfThreads + threadIdx.x;
  if (i >= (int64_t)Hkv * K_tot) return;
  const int g = (int)(i / K_tot), j = (int)(i - (int64_t)g * K_tot);
  const int b = upper_segment(cu_k, B, j);
  const int t = kv_index[i];
  if (t < 0 || t >= cu[b + 1] - cu[b]) { raise(dev_status, SG_ERR_INDEX); return; }
  atomicAdd(counts + (int64_t)g * T + cu[b] + t, 1);
}

// One warp per (layer, block): sums the counts of the block's tokens over all heads and sequences.
__global__ void __launch_bounds__(kProfThreads) block_importance_kernel(const int32_t* __restrict__ counts,
                                                                         const int32_t* __restrict__ cu, float* importance,
                                                                         int L, int B, int Hkv, int M, int64_t T) {
  const int lane = threadIdx.x & 31;
  const int64_t w = (int64_t)blockIdx.x * (kProfThreads / 32) + (threadIdx.x >> 5);
  if (w >= (int64_t)L * M) return;
  const int l = (int)(w / M), m = (int)(w - (int64_t)l * M);
  if (l < 2) { if (lane == 0) importance[w] = INFINITY; return; }      // first two layers: always selected
  long long sum = 0, entries = 0;
  for (int b = 0; b < B; ++b) {
    const int64_t c0 = cu[b], N = cu[b + 1] - c0;
    // tokens with floor(t*M/N) == m:  ceil(m*N/M) <= t < ceil((m+1)*N/M)
    const int64_t t_beg = ((int64_t)m * N + M - 1) / M, t_end = ((int64_t)(m + 1) * N + M - 1) / M;
    entries += (t_end - t_beg) * Hkv;
    for (int64_t e = lane; e < (t_end - t_beg) * Hkv; e += 32) {
      const int64_t t = t_beg + e / Hkv;
      const int g = (int)(e % Hkv);
      sum += counts[((int64_t)l * Hkv + g) * T + c0 + t];
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
  if (lane == 0) importance[w] = entries ? (float)((double)sum / (double)entries) : 0.0f;
}

__global__ void __launch_bounds__(kProfThreads) proactive_mask_kernel(const int32_t* __restrict__ cu,
                                                                       const int32_t* __restrict__ selected, int8_t* mask,
                                                                       int B, int M, int layer, int K_r, int64_t T) {
  const int64_t i = (int64_t)blockIdx.x * kProfThreads + threadIdx.x;
  if (i >= T) return;
  const int b = upper_segment(cu, B, i);
  const int64_t N = cu[b + 1] - cu[b], t = i - cu[b];
  const int32_t id = (int32_t)((int64_t)layer * M + t * M / N);
  int lo = 0, hi = K_r;                                  // binary search in the ascending list
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (selected[mid] < id) lo = mid + 1; else hi = mid;
  }
  mask[i] = (lo < K_r && selected[lo] == id) ? 1 : 2;
}

}  // namespace
}  // namespace sg

extern "C" sg_status sg_profile_accumulate(const sg_shape* shape, const int32_t* kv_index, const int32_t* cu_k,
                                           int32_t total_sel, int32_t* counts, int32_t* dev_status, void* stream) {
  using namespace sg;
  sg_status st = check_shape(shape, false);
  if (st != SG_OK) return st;
  if (shape->num_layers != 1 || total_sel < 0) return SG_ERR_INVALID;
  if (total_sel == 0) return SG_OK;
  if (!kv_index || !cu_k || !counts || !aligned16(kv_index) || !aligned16(cu_k) || !aligned16(counts)) return SG_ERR_INVALID;
  const int64_t n = (int64_t)shape->num_kv_heads * total_sel;
  const int64_t grid = (n + kProfThreads - 1) / kProfThreads;
  if (grid > 0x7fffffffLL) return SG_ERR_UNSUPPORTED;
  profile_accumulate_kernel<<<(unsigned)grid, kProfThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      kv_index, shape->cu_seqlens, cu_k, counts, dev_status, shape->batch, shape->num_kv_heads, total_sel, shape->total_tokens);
  SG_CUDA_TRY(cudaGetLastError());
  return SG_OK;
}

extern "C" sg_status sg_block_importance(const sg_shape* shape, const int32_t* counts, int32_t num_blocks,
                                         float* importance, void* stream) {
  using namespace sg;
  sg_status st = check_shape(shape, false);
  if (st != SG_OK) return st;
  if (num_blocks < 1 || !counts || !importance || !aligned16(counts) || !aligned16(importance)) return SG_ERR_INVALID;
  const int64_t warps = (int64_t)shape->num_layers * num_blocks;
  const int64_t grid = (warps + kProfThreads / 32 - 1) / (kProfThreads / 32);
  if (grid > 0x7fffffffLL) return SG_ERR_UNSUPPORTED;
  block_importance_kernel<<<(unsigned)grid, kProfThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      counts, shape->cu_seqlens, importance, shape->num_layers, shape->batch, shape->num_kv_heads, num_blocks,
      shape->total_tokens);
  SG_CUDA_TRY(cudaGetLastError());
  return SG_OK;
}

extern "C" int64_t sg_transfer_budget(int32_t num_layers, int32_t num_blocks, double t_prefill, double t_transfer) {
  double k = (double)num_blocks * (double)(num_layers - 1) * t_prefill / t_transfer;
  const double lo = 2.0 * num_blocks, hi = (double)num_layers * num_blocks;
  if (!(k >= lo)) k = lo;
  if (k > hi) k = hi;
  if (num_layers < 2) k = hi;
  return (int64_t)floor(k);
}

extern "C" int64_t sg_speculative_delivered(int32_t num_layers, int32_t num_blocks, int64_t k_r, double ratio,
                                            int32_t iteration) {
  const int64_t total = (int64_t)num_layers * num_blocks;
  int64_t quota = (int64_t)floor(ratio * (double)total);
  if (quota < 1) quota = 1;
  int64_t n = k_r + (int64_t)iteration * quota;
  if (n > total) n = total;
  if (n < 0) n = 0;
  return n;
}

extern "C" sg_status sg_proactive_mask(const sg_shape* shape, int32_t num_blocks, int32_t layer, const int32_t* selected,
                                       int32_t num_selected, int8_t* kv_mask, void* stream) {
  using namespace sg;
  sg_status st = check_shape(shape, false);
  if (st != SG_OK) return st;
  if (num_blocks < 1 || layer < 0 || num_selected < 0 || !kv_mask) return SG_ERR_INVALID;
  if (num_selected > 0 && (!selected || !aligned16(selected))) return SG_ERR_INVALID;
  if (shape->total_tokens == 0) return SG_OK;
  const int64_t grid = ((int64_t)shape->total_tokens + kProfThreads - 1) / kProfThreads;
  proactive_mask_kernel<<<(unsigned)grid, kProfThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      shape->cu_seqlens, selected ? selected : shape->cu_seqlens, kv_mask, shape->batch, num_blocks, layer, num_selected,
      shape->total_tokens);
  SG_CUDA_TRY(cudaGetLastError());
  return SG_OK;
}
