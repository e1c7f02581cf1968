// sg_pack_kv: index-driven gather of selected K/V rows into a contiguous buffer.
//
// Pure byte movement, bound by HBM: every selected row (2*d bytes of K, 2*d bytes of V) is read
// once and written once.  One group of d/8 threads moves one row with 16-byte vectors, so a
// warp's accesses cover whole 128-byte lines on both sides; each group has kUnroll independent
// rows (2*kUnroll loads) in flight before the first store.
#include "common.cuh"

namespace sg {
namespace {

constexpr int kPackThreads = 256;
constexpr int kUnroll = 4;

struct PackParams {
  const uint16_t* k_cache;
  const uint16_t* v_cache;
  const int32_t* sel_idx;
  const int32_t* cu;
  const int32_t* cu_k;
  const int32_t* sel_count;   // [L][B][Hkv] entries selected per row, or null: every entry of the row
  uint16_t* packed_k;
  uint16_t* packed_v;
  int32_t* dev_status;
  int64_t ls, ts, hs;
  int64_t total_rows;      // L * K_tot * H_kv
  int64_t rows_per_layer;  // K_tot * H_kv
  int32_t K_tot, B, Hkv;
};

// kCounted: rows beyond a head's count (PackParams::sel_count) are skipped; the plain instantiation carries none of it.
template <int D, bool kCounted>
__global__ void __launch_bounds__(kPackThreads) pack_kv_kernel(const PackParams p) {
  constexpr int kTPR = D / 8;                       // threads per row, 16 bytes each
  constexpr int kRowsPerPass = kPackThreads / kTPR;
  const int lane_in_row = threadIdx.x % kTPR;
  const int group = threadIdx.x / kTPR;
  const int64_t row0 = (int64_t)blockIdx.x * (kRowsPerPass * kUnroll) + group;

  int4 kv[kUnroll][2];
  bool ok[kUnroll], skip[kUnroll];
#pragma unroll
  for (int u = 0; u < kUnroll; ++u) {
    const int64_t r = row0 + (int64_t)u * kRowsPerPass;
    ok[u] = false;
    skip[u] = false;
    kv[u][0] = make_int4(0, 0, 0, 0);
    kv[u][1] = make_int4(0, 0, 0, 0);
    if (r < p.total_rows) {
      const int64_t l = r / p.rows_per_layer;
      const int64_t rr = r - l * p.rows_per_layer;
      const int b = upper_segment(p.cu_k, p.B, rr, p.Hkv);
      const int ck = p.cu_k[b];
      const int kb = p.cu_k[b + 1] - ck;
      const int rem = (int)(rr - (int64_t)ck * p.Hkv);
      const int g = rem / kb;
      const int j = rem - g * kb;
      const int c0 = p.cu[b];
      const int n = p.cu[b + 1] - c0;
      if (kCounted && j >= p.sel_count[(l * p.B + b) * p.Hkv + g]) { skip[u] = true; continue; }   // not selected: slot left as it is
      const int t = p.sel_idx[(l * p.Hkv + g) * (int64_t)p.K_tot + ck + j];
      if (t >= 0 && t < n) {
        ok[u] = true;
        const int64_t src = l * p.ls + ((int64_t)c0 + t) * p.ts + (int64_t)g * p.hs + lane_in_row * 8;
        kv[u][0] = __ldcs(reinterpret_cast<const int4*>(p.k_cache + src));
        kv[u][1] = __ldcs(reinterpret_cast<const int4*>(p.v_cache + src));
      } else if (lane_in_row == 0) {
        raise(p.dev_status, SG_ERR_INDEX);
      }
    }
  }
#pragma unroll
  for (int u = 0; u < kUnroll; ++u) {
    const int64_t r = row0 + (int64_t)u * kRowsPerPass;
    if (r < p.total_rows && !(kCounted && skip[u])) {
      const int64_t dst = r * D + lane_in_row * 8;
      __stcs(reinterpret_cast<int4*>(p.packed_k + dst), kv[u][0]);
      __stcs(reinterpret_cast<int4*>(p.packed_v + dst), kv[u][1]);
    }
  }
  (void)ok;
}

}  // namespace
}  // namespace sg

namespace sg {
namespace {
sg_status pack_kv_launch(const sg_shape* shape, const void* k_cache, const void* v_cache, const int32_t* sel_idx,
                         const int32_t* cu_k, int32_t total_sel, const int32_t* sel_count, void* packed_k, void* packed_v,
                         int32_t* dev_status, void* stream);
}
}  // namespace sg

extern "C" sg_status sg_pack_kv(const sg_shape* shape, const void* k_cache, const void* v_cache,
                                const int32_t* sel_idx, const int32_t* cu_k, int32_t total_sel,
                                void* packed_k, void* packed_v, int32_t* dev_status, void* stream) {
  return sg::pack_kv_launch(shape, k_cache, v_cache, sel_idx, cu_k, total_sel, nullptr, packed_k, packed_v, dev_status, stream);
}

extern "C" sg_status sg_pack_kv_counted(const sg_shape* shape, const void* k_cache, const void* v_cache,
                                        const int32_t* sel_idx, const int32_t* cu_cap, int32_t total_cap,
                                        const int32_t* sel_count, void* packed_k, void* packed_v, int32_t* dev_status,
                                        void* stream) {
  if (!sel_count || !sg::aligned16(sel_count)) return SG_ERR_INVALID;
  return sg::pack_kv_launch(shape, k_cache, v_cache, sel_idx, cu_cap, total_cap, sel_count, packed_k, packed_v, dev_status, stream);
}

namespace sg {
namespace {
sg_status pack_kv_launch(const sg_shape* shape, const void* k_cache, const void* v_cache, const int32_t* sel_idx,
                         const int32_t* cu_k, int32_t total_sel, const int32_t* sel_count, void* packed_k, void* packed_v,
                         int32_t* dev_status, void* stream) {
  using namespace sg;
  sg_status st = check_shape(shape, false);
  if (st != SG_OK) return st;
  if (total_sel < 0) return SG_ERR_INVALID;
  if (total_sel == 0) return SG_OK;
  if (!k_cache || !v_cache || !sel_idx || !cu_k || !packed_k || !packed_v) return SG_ERR_INVALID;
  if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(sel_idx) || !aligned16(cu_k) ||
      !aligned16(packed_k) || !aligned16(packed_v))
    return SG_ERR_INVALID;
  PackParams p;
  p.k_cache = static_cast<const uint16_t*>(k_cache);
  p.v_cache = static_cast<const uint16_t*>(v_cache);
  p.sel_idx = sel_idx;
  p.cu = shape->cu_seqlens;
  p.cu_k = cu_k;
  p.sel_count = sel_count;
  p.packed_k = static_cast<uint16_t*>(packed_k);
  p.packed_v = static_cast<uint16_t*>(packed_v);
  p.dev_status = dev_status;
  p.ls = shape->cache_layer_stride;
  p.ts = shape->cache_token_stride;
  p.hs = shape->cache_head_stride;
  p.K_tot = total_sel;
  p.B = shape->batch;
  p.Hkv = shape->num_kv_heads;
  p.rows_per_layer = (int64_t)total_sel * shape->num_kv_heads;
  p.total_rows = p.rows_per_layer * shape->num_layers;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (shape->head_dim == 128) {
    const int64_t rows_per_cta = (kPackThreads / 16) * kUnroll;
    const int64_t grid = (p.total_rows + rows_per_cta - 1) / rows_per_cta;
    if (grid > 0x7fffffffLL) return SG_ERR_UNSUPPORTED;
    if (sel_count) pack_kv_kernel<128, true><<<(unsigned)grid, kPackThreads, 0, s>>>(p);
    else pack_kv_kernel<128, false><<<(unsigned)grid, kPackThreads, 0, s>>>(p);
  } else {
    const int64_t rows_per_cta = (kPackThreads / 8) * kUnroll;
    const int64_t grid = (p.total_rows + rows_per_cta - 1) / rows_per_cta;
    if (grid > 0x7fffffffLL) return SG_ERR_UNSUPPORTED;
    if (sel_count) pack_kv_kernel<64, true><<<(unsigned)grid, kPackThreads, 0, s>>>(p);
    else pack_kv_kernel<64, false><<<(unsigned)grid, kPackThreads, 0, s>>>(p);
  }
  SG_CUDA_TRY(cudaGetLastError());
  return SG_OK;
}
}  // namespace
}  // namespace sg
