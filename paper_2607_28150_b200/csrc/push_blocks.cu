// sg_push_blocks: the online proactive transfer at block granularity (Section 4.1).
//
// Every KV block of the call's layers whose flat id l*M + m is in the selected set is copied, all KV heads,
// K and V, to the same token positions of the decode-side cache.  Pure byte movement, bound by HBM: a
// selected row is read once and written once.  One CTA per (block, sequence, layer): it looks its block up
// in the ascending selected list once (a uniform binary search, L2-resident) and leaves if the block is not
// selected or holds no token of the sequence -- unselected blocks cost no cache traffic.  Otherwise one
// group of d/8 threads moves one (token, head) row with 16-byte vectors, a warp covers whole 128-byte
// lines, and each group has kUnroll independent rows (2*kUnroll loads) in flight before the first store.
// The rows of a block form one contiguous run when the cache is dense.  Optionally the same CTA marks the
// block's tokens as local (1) in the decode-side KV mask, the update the paper sends behind every pushed block.
#include "common.cuh"

namespace sg {
namespace {

constexpr int kPushThreads = 256;
constexpr int kUnroll = 4;

struct PushParams {
  const uint16_t* src_k;
  const uint16_t* src_v;
  uint16_t* dst_k;
  uint16_t* dst_v;
  const int32_t* cu;
  const int32_t* selected;
  int8_t* kv_mask;         // [layers][T] decode-side KV mask to update (1 = local) for the pushed tokens, or null
  int64_t T;
  int64_t ls, ts, hs;
  int32_t B, Hkv, M, layer, K_r;
};

template <int D>
__global__ void __launch_bounds__(kPushThreads) push_blocks_kernel(const PushParams p) {
  constexpr int kTPR = D / 8;                       // threads per row, 16 bytes each
  constexpr int kRowsPerPass = kPushThreads / kTPR;
  const int m = blockIdx.x, b = blockIdx.y, l = blockIdx.z;
  const int32_t id = (int32_t)(((int64_t)p.layer + l) * p.M + m);
  int lo = 0, hi = p.K_r;                           // binary search in the ascending list, uniform over the CTA
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (p.selected[mid] < id) lo = mid + 1; else hi = mid;
  }
  if (lo >= p.K_r || p.selected[lo] != id) return;
  const int64_t c0 = p.cu[b], N = p.cu[b + 1] - c0;
  // tokens t with floor(t * M / N) == m
  const int64_t t0 = ((int64_t)m * N + p.M - 1) / p.M, t1 = ((int64_t)(m + 1) * N + p.M - 1) / p.M;
  const int rows = (int)(t1 - t0) * p.Hkv;
  if (p.kv_mask)                                    // the pushed tokens are locally available from now on
    for (int t = threadIdx.x; t < (int)(t1 - t0); t += kPushThreads) p.kv_mask[(int64_t)l * p.T + c0 + t0 + t] = 1;
  const int lane_in_row = threadIdx.x % kTPR;
  const int group = threadIdx.x / kTPR;
  const int64_t base = (int64_t)l * p.ls + (c0 + t0) * p.ts + lane_in_row * 8;
  for (int r0 = group; r0 < rows; r0 += kRowsPerPass * kUnroll) {
    int4 kv[kUnroll][2];
    int64_t off[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int r = r0 + u * kRowsPerPass;
      off[u] = -1;
      if (r < rows) {
        const int t = r / p.Hkv, g = r - t * p.Hkv;
        off[u] = base + (int64_t)t * p.ts + (int64_t)g * p.hs;
        kv[u][0] = __ldcs(reinterpret_cast<const int4*>(p.src_k + off[u]));
        kv[u][1] = __ldcs(reinterpret_cast<const int4*>(p.src_v + off[u]));
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      if (off[u] >= 0) {
        __stcs(reinterpret_cast<int4*>(p.dst_k + off[u]), kv[u][0]);
        __stcs(reinterpret_cast<int4*>(p.dst_v + off[u]), kv[u][1]);
      }
    }
  }
}

}  // namespace
}  // namespace sg

extern "C" sg_status sg_push_blocks(const sg_shape* shape, int32_t num_blocks, int32_t layer, const int32_t* selected,
                                    int32_t num_selected, const void* src_k, const void* src_v, void* dst_k, void* dst_v,
                                    int8_t* kv_mask, void* stream) {
  using namespace sg;
  sg_status st = check_shape(shape, false);
  if (st != SG_OK) return st;
  if (num_blocks < 1 || layer < 0 || num_selected < 0) return SG_ERR_INVALID;
  if (((int64_t)layer + shape->num_layers) * num_blocks > 0x7fffffffLL) return SG_ERR_UNSUPPORTED;
  if (num_selected == 0 || shape->total_tokens == 0) return SG_OK;
  if (!selected || !src_k || !src_v || !dst_k || !dst_v) return SG_ERR_INVALID;
  if (!aligned16(selected) || !aligned16(src_k) || !aligned16(src_v) || !aligned16(dst_k) || !aligned16(dst_v))
    return SG_ERR_INVALID;
  PushParams p;
  p.src_k = static_cast<const uint16_t*>(src_k);
  p.src_v = static_cast<const uint16_t*>(src_v);
  p.dst_k = static_cast<uint16_t*>(dst_k);
  p.dst_v = static_cast<uint16_t*>(dst_v);
  p.cu = shape->cu_seqlens;
  p.selected = selected;
  p.kv_mask = kv_mask;
  p.T = shape->total_tokens;
  p.ls = shape->cache_layer_stride;
  p.ts = shape->cache_token_stride;
  p.hs = shape->cache_head_stride;
  p.B = shape->batch;
  p.Hkv = shape->num_kv_heads;
  p.M = num_blocks;
  p.layer = layer;
  p.K_r = num_selected;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (shape->batch > 65535 || shape->num_layers > 65535) return SG_ERR_UNSUPPORTED;
  const dim3 grid((unsigned)num_blocks, (unsigned)shape->batch, (unsigned)shape->num_layers);
  if (shape->head_dim == 128) push_blocks_kernel<128><<<grid, kPushThreads, 0, s>>>(p);
  else push_blocks_kernel<64><<<grid, kPushThreads, 0, s>>>(p);
  SG_CUDA_TRY(cudaGetLastError());
  return SG_OK;
}
