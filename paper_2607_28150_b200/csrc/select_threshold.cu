// sg_select_threshold: threshold (alpha) selection under a cap.
//
// Per (layer, sequence, KV head): the tokens whose score exceeds the row maximum minus alpha, at most cap_b
// of them (the largest, ties to the lower index), emitted in ascending order with their count.  A threshold
// set is an upper set of the score order, so it is the exact top-cap_b set (sg_select_topk's exact selection,
// run first with the cap as its budget) cut at the threshold: one CTA per row finds the row maximum among the
// cap_b candidates, keeps the candidates above max - alpha with a stable block-wide compaction in place,
// pads the rest of the row with -1 and writes the count.  Comparisons run on the order-preserving integer
// image of the scores, so subnormal scores are not flushed; a NaN is never selected (but may have taken one of
// the cap_b candidate slots: NaN-free scores are part of the contract).
#include "common.cuh"

namespace sg {
namespace {

constexpr int kTrimThreads = 256;

__device__ __forceinline__ uint32_t order_key(uint32_t u) { return (u & 0x80000000u) ? ~u : (u | 0x80000000u); }
__device__ __forceinline__ uint32_t key_to_bits(uint32_t k) { return (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k; }
__device__ __forceinline__ bool is_nan_bits(uint32_t u) { return (u & 0x7f800000u) == 0x7f800000u && (u & 0x007fffffu) != 0u; }

struct TrimParams {
  const float* scores;
  const int32_t* cu;
  const int32_t* cu_cap;
  int32_t* sel_idx;
  int32_t* sel_count;
  int32_t* dev_status;
  int64_t T;
  int32_t cap_tot, B, Hkv;
  float alpha;
};

__global__ void __launch_bounds__(kTrimThreads) threshold_trim_kernel(const TrimParams p) {
  __shared__ uint32_t s_red[kTrimThreads / 32];
  __shared__ int s_scan[kTrimThreads / 32 + 1];
  __shared__ int s_running;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row = blockIdx.x;
  const int l = row / (p.B * p.Hkv);
  const int rem = row - l * (p.B * p.Hkv);
  const int b = rem / p.Hkv;
  const int g = rem - b * p.Hkv;
  const int N = p.cu[b + 1] - p.cu[b];
  const int cc = p.cu_cap[b];
  const int cap = p.cu_cap[b + 1] - cc;
  int32_t* idx = p.sel_idx + ((int64_t)l * p.Hkv + g) * p.cap_tot + cc;
  const uint32_t* x = reinterpret_cast<const uint32_t*>(p.scores) + ((int64_t)l * p.Hkv + g) * p.T + p.cu[b];
  int32_t* count_out = p.sel_count + ((int64_t)l * p.B + b) * p.Hkv + g;
  if (cap <= 0) { if (tid == 0) *count_out = 0; return; }

  // row maximum among the candidates (NaNs ignored); 0 = none found (every real key is > 0 ... except -NaN, ignored too)
  uint32_t kmax = 0;
  for (int j = tid; j < cap; j += kTrimThreads) {
    const int t = idx[j];
    if (t >= 0 && t < N) {
      const uint32_t u = __ldg(x + t);
      if (!is_nan_bits(u)) kmax = max(kmax, order_key(u));
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, off));
  if (lane == 0) s_red[warp] = kmax;
  if (tid == 0) s_running = 0;
  __syncthreads();
  kmax = 0;
#pragma unroll
  for (int w = 0; w < kTrimThreads / 32; ++w) kmax = max(kmax, s_red[w]);
  const bool have_max = kmax != 0;
  float thr;                                                  // IEEE subtraction without flush-to-zero, whatever the compile flags
  asm("sub.rn.f32 %0, %1, %2;" : "=f"(thr) : "f"(__uint_as_float(key_to_bits(kmax))), "f"(p.alpha));
  uint32_t thr_bits = __float_as_uint(thr);
  if ((thr_bits & 0x7fffffffu) == 0u) thr_bits = 0u;           // -0 and +0 compare equal as floats: use +0's key
  const uint32_t kthr = order_key(thr_bits);

  // stable compaction in place, one chunk of kTrimThreads candidates at a time (writes never pass the reads)
  for (int j0 = 0; j0 < cap; j0 += kTrimThreads) {
    const int j = j0 + tid;
    int t = -1;
    bool keep = false;
    if (j < cap) {
      t = idx[j];
      if (have_max && t >= 0 && t < N) {
        const uint32_t u = __ldg(x + t);
        keep = !is_nan_bits(u) && order_key(u) > kthr;
      }
    }
    const uint32_t ballot = __ballot_sync(0xffffffffu, keep);
    if (lane == 0) s_scan[warp] = __popc(ballot);
    __syncthreads();                                          // every read of this chunk is done; warp counts are visible
    int before = s_running;
#pragma unroll
    for (int w = 0; w < kTrimThreads / 32; ++w) before += w < warp ? s_scan[w] : 0;
    int chunk_total = 0;
#pragma unroll
    for (int w = 0; w < kTrimThreads / 32; ++w) chunk_total += s_scan[w];
    if (keep) idx[before + __popc(ballot & ((1u << lane) - 1u))] = t;
    __syncthreads();
    if (tid == 0) s_running += chunk_total;
    __syncthreads();
  }
  const int n = s_running;
  for (int j = n + tid; j < cap; j += kTrimThreads) idx[j] = -1;
  if (tid == 0) *count_out = n;
}

}  // namespace
}  // namespace sg

extern "C" sg_status sg_select_threshold(const sg_shape* shape, const float* scores, float alpha, const int32_t* cu_cap,
                                         int32_t total_cap, int32_t* sel_idx, int32_t* sel_count, int32_t* dev_status,
                                         void* stream) {
  using namespace sg;
  sg_status st = check_shape(shape, false);
  if (st != SG_OK) return st;
  if (total_cap < 0 || !(alpha >= 0.f)) return SG_ERR_INVALID;
  if (!scores || !cu_cap || !sel_count || !aligned16(scores) || !aligned16(cu_cap) || !aligned16(sel_count)) return SG_ERR_INVALID;
  if (total_cap > 0 && (!sel_idx || !aligned16(sel_idx))) return SG_ERR_INVALID;
  const int64_t rows = (int64_t)shape->num_layers * shape->batch * shape->num_kv_heads;
  if (rows > 0x7fffffffLL) return SG_ERR_UNSUPPORTED;
  if (total_cap > 0) {
    st = sg_select_topk(shape, scores, cu_cap, total_cap, sel_idx, nullptr, 0, dev_status, stream);
    if (st != SG_OK) return st;
  }
  TrimParams p;
  p.scores = scores;
  p.cu = shape->cu_seqlens;
  p.cu_cap = cu_cap;
  p.sel_idx = sel_idx;
  p.sel_count = sel_count;
  p.dev_status = dev_status;
  p.T = shape->total_tokens;
  p.cap_tot = total_cap;
  p.B = shape->batch;
  p.Hkv = shape->num_kv_heads;
  p.alpha = alpha;
  threshold_trim_kernel<<<(unsigned)rows, kTrimThreads, 0, static_cast<cudaStream_t>(stream)>>>(p);
  SG_CUDA_TRY(cudaGetLastError());
  return SG_OK;
}
