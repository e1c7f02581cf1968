// sg_split_index: Algorithm 1 (KV index splitting and reordering) on the device.
//
// One CTA owns one row of the KV index (one sequence, one KV head).  It looks up the int8 class of every
// selected token in the KV mask (2 = remote, 1 = local, 0 = padding) and forms a stable three-way partition of
// the row by class -- remote first, then local, then padding -- with ballots and prefix counts: no atomics, so
// the output order is a pure function of the input.  The partitioned row (when asked for) and the local and
// remote index lists with their counts are written.  Integer work only, bound by latency (a row is a few KB).
#include "common.cuh"

namespace sg {
namespace {

constexpr int kSplitThreads = 256;
constexpr int kSplitWarps = kSplitThreads / 32;

struct SplitParams {
  const int32_t* kv_index;
  const int8_t* kv_mask;
  const int32_t* cu;
  const int32_t* cu_k;
  int32_t* reordered;
  int32_t* local_index;
  int32_t* remote_index;
  int32_t* n_local;
  int32_t* n_remote;
  int32_t* dev_status;
  int32_t K_tot, B, Hkv, reorder;
};

__global__ void __launch_bounds__(kSplitThreads) split_index_kernel(const SplitParams p) {
  __shared__ uint32_t w_cnt[3][kSplitWarps];     // per-warp counts of classes remote / local / padding
  __shared__ uint32_t w_base[3][kSplitWarps];
  __shared__ uint32_t tot[3];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.x / p.Hkv, g = blockIdx.x - b * p.Hkv;
  const int c0 = p.cu[b], N = p.cu[b + 1] - c0;
  const int ck = p.cu_k[b], kb = p.cu_k[b + 1] - ck;
  const int64_t base = (int64_t)g * p.K_tot + ck;
  // warp w owns positions [w*C, (w+1)*C) of the row, C a multiple of 32
  const int C = (((kb + kSplitWarps - 1) / kSplitWarps) + 31) & ~31;
  const int beg = warp * C, end = min(kb, beg + C);
  auto classify = [&](int j, int& t) -> int {       // 0 remote, 1 local, 2 padding (or invalid), 3 nothing
    if (j >= end) return 3;
    t = p.kv_index[base + j];
    if (t < 0 || t >= N) { raise(p.dev_status, SG_ERR_INDEX); return 2; }
    const int m = p.kv_mask[c0 + t];
    return m == 2 ? 0 : (m == 1 ? 1 : 2);
  };
  uint32_t cnt[3] = {0, 0, 0};
  for (int j0 = beg; j0 < end; j0 += 32) {
    int t;
    const int cls = classify(j0 + lane, t);
#pragma unroll
    for (int c = 0; c < 3; ++c) cnt[c] += __popc(__ballot_sync(0xffffffffu, cls == c));
  }
  if (lane == 0) { w_cnt[0][warp] = cnt[0]; w_cnt[1][warp] = cnt[1]; w_cnt[2][warp] = cnt[2]; }
  __syncthreads();
  if (tid < 3) {
    uint32_t run = 0;
    for (int w = 0; w < kSplitWarps; ++w) { w_base[tid][w] = run; run += w_cnt[tid][w]; }
    tot[tid] = run;
  }
  __syncthreads();
  const uint32_t n_rem = tot[0], n_loc = tot[1];
  if (tid == 0) { p.n_remote[b * p.Hkv + g] = (int32_t)n_rem; p.n_local[b * p.Hkv + g] = (int32_t)n_loc; }
  uint32_t run[3] = {w_base[0][warp], w_base[1][warp], w_base[2][warp]};
  const uint32_t lt = (1u << lane) - 1u;
  for (int j0 = beg; j0 < end; j0 += 32) {
    int t = 0;
    const int j = j0 + lane;
    const int cls = classify(j, t);
    uint32_t bal[3];
#pragma unroll
    for (int c = 0; c < 3; ++c) bal[c] = __ballot_sync(0xffffffffu, cls == c);
    if (cls < 3) {
      const uint32_t rank = run[cls] + __popc(bal[cls] & lt);
      if (cls == 0) p.remote_index[base + rank] = t;
      if (cls == 1) p.local_index[base + rank] = t;
      if (p.reordered) {
        const uint32_t dst = p.reorder ? (cls == 0 ? rank : (cls == 1 ? n_rem + rank : n_rem + n_loc + rank)) : (uint32_t)j;
        p.reordered[base + dst] = t;
      }
    }
#pragma unroll
    for (int c = 0; c < 3; ++c) run[c] += __popc(bal[c]);
  }
}

}  // namespace
}  // namespace sg

extern "C" sg_status sg_split_index(const sg_shape* shape, const int32_t* kv_index, const int32_t* cu_k,
                                    int32_t total_sel, const int8_t* kv_mask, int32_t reorder, int32_t* reordered,
                                    int32_t* local_index, int32_t* remote_index, int32_t* n_local, int32_t* n_remote,
                                    int32_t* dev_status, void* stream) {
  using namespace sg;
  sg_status st = check_shape(shape, false);
  if (st != SG_OK) return st;
  if (shape->num_layers != 1 || total_sel < 0) return SG_ERR_INVALID;
  if (!cu_k || !n_local || !n_remote) return SG_ERR_INVALID;
  if (total_sel > 0 && (!kv_index || !kv_mask || !local_index || !remote_index)) return SG_ERR_INVALID;
  if (!aligned16(kv_index) || !aligned16(cu_k) || !aligned16(local_index) || !aligned16(remote_index) ||
      !aligned16(reordered) || (reinterpret_cast<uintptr_t>(n_local) & 3u) || (reinterpret_cast<uintptr_t>(n_remote) & 3u))
    return SG_ERR_INVALID;
  const int64_t rows = (int64_t)shape->batch * shape->num_kv_heads;
  if (rows > 0x7fffffffLL) return SG_ERR_UNSUPPORTED;
  SplitParams p;
  p.kv_index = kv_index;
  p.kv_mask = kv_mask;
  p.cu = shape->cu_seqlens;
  p.cu_k = cu_k;
  p.reordered = reordered;
  p.local_index = local_index;
  p.remote_index = remote_index;
  p.n_local = n_local;
  p.n_remote = n_remote;
  p.dev_status = dev_status;
  p.K_tot = total_sel;
  p.B = shape->batch;
  p.Hkv = shape->num_kv_heads;
  p.reorder = reorder ? 1 : 0;
  split_index_kernel<<<(unsigned)rows, kSplitThreads, 0, static_cast<cudaStream_t>(stream)>>>(p);
  SG_CUDA_TRY(cudaGetLastError());
  return SG_OK;
}
