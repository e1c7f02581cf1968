// sg_select_topk: per-(layer, sequence, KV head) top-k by MSB-first radix select.
//
// One CTA owns one importance row.  The row's fp32 values are mapped to order-preserving uint32
// keys and kept in shared memory (rows of up to ~55K tokens; longer rows are re-read from L2).
// Four 8-bit histogram passes find the k-th largest key exactly; a final ordered compaction
// (ballot + prefix counts, no atomics) emits the selected positions in ascending order, taking
// equal-to-threshold entries from the lowest positions first.  The result is therefore a pure
// function of the input row: identical on every run and identical to a full sort.
#include "common.cuh"

namespace sg {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kHistCopies = 8;
constexpr int kMaxSmemBytes = 227 * 1024;
constexpr int kSelFixedSmem = (kHistCopies * 256 + 256 + 4 * kSelWarps + 8) * 4;
constexpr int kSelKeyCap = (kMaxSmemBytes - kSelFixedSmem) / 4;

struct SelParams {
  const float* importance;
  const int32_t* cu;
  const int32_t* cu_k;
  int32_t* sel_idx;
  int32_t* dev_status;
  int64_t T;
  int32_t K_tot, B, Hkv;
};

// Takes the raw bit pattern: the row is read as uint32 so that no float instruction (and no
// flush-to-zero of subnormals) ever touches the values.
__device__ __forceinline__ uint32_t order_key(uint32_t u) {
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <bool kInSmem>
__global__ void __launch_bounds__(kSelThreads, 1) select_topk_kernel(const SelParams p) {
  extern __shared__ __align__(16) uint32_t smem[];
  uint32_t* hist = smem;                              // [kHistCopies][256]
  uint32_t* total = hist + kHistCopies * 256;         // [256]
  uint32_t* wgt = total + 256;                        // [kSelWarps] per-warp counts / bases
  uint32_t* weq = wgt + kSelWarps;
  uint32_t* wgt_base = weq + kSelWarps;
  uint32_t* weq_base = wgt_base + kSelWarps;
  uint32_t* sh = weq_base + kSelWarps;                // [0] chosen bin, [1] remaining need
  uint32_t* keys = sh + 8;                            // [N] when kInSmem

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row = blockIdx.x;
  const int l = row / (p.B * p.Hkv);
  const int rem = row - l * (p.B * p.Hkv);
  const int b = rem / p.Hkv;
  const int g = rem - b * p.Hkv;
  const int c0 = p.cu[b];
  const int N = p.cu[b + 1] - c0;
  const int ck = p.cu_k[b];
  const int kb = p.cu_k[b + 1] - ck;
  if (kb <= 0) return;
  int32_t* out = p.sel_idx + ((int64_t)l * p.Hkv + g) * p.K_tot + ck;
  if (kb >= N) {                                      // whole prompt (or an over-sized budget)
    if (kb > N && tid == 0) raise(p.dev_status, SG_ERR_INVALID);
    for (int j = tid; j < kb; j += kSelThreads) out[j] = j < N ? j : -1;
    return;
  }
  const uint32_t* x = reinterpret_cast<const uint32_t*>(p.importance) + ((int64_t)l * p.Hkv + g) * p.T + c0;

  if (kInSmem) {
    for (int t = tid; t < N; t += kSelThreads) keys[t] = order_key(__ldg(x + t));
  }
  auto key_at = [&](int t) -> uint32_t { return kInSmem ? keys[t] : order_key(__ldg(x + t)); };

  // ---- radix select: find the kb-th largest key ----
  uint32_t prefix = 0, decided = 0, need = (uint32_t)kb;
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int i = tid; i < kHistCopies * 256; i += kSelThreads) hist[i] = 0;
    __syncthreads();
    uint32_t* my_hist = hist + (warp % kHistCopies) * 256;
    for (int t = tid; t < N; t += kSelThreads) {
      const uint32_t k = key_at(t);
      if ((k & decided) == prefix) atomicAdd(&my_hist[(k >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid < 256) {
      uint32_t s = 0;
#pragma unroll
      for (int c = 0; c < kHistCopies; ++c) s += hist[c * 256 + tid];
      total[tid] = s;
    }
    __syncthreads();
    if (warp == 0) {
      uint32_t c[8], s = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { c[i] = total[255 - (lane * 8 + i)]; s += c[i]; }
      uint32_t inc = s;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += v;
      }
      const uint32_t exc = inc - s;                   // candidates in bins above this lane's bins
      if (exc < need && need <= inc) {
        uint32_t run = exc;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (run < need && need <= run + c[i]) { sh[0] = 255u - (uint32_t)(lane * 8 + i); sh[1] = need - run; }
          run += c[i];
        }
      }
    }
    __syncthreads();
    prefix |= sh[0] << shift;
    decided |= 255u << shift;
    need = sh[1];
    __syncthreads();
  }
  const uint32_t tau = prefix;                        // the kb-th largest key
  const uint32_t need_eq = need;                      // entries equal to tau to keep, lowest positions first

  // ---- ordered compaction: warp w owns positions [w*C, (w+1)*C) ----
  const int C = (((N + kSelWarps - 1) / kSelWarps) + 31) & ~31;
  const int beg = warp * C;
  const int end = min(N, beg + C);
  uint32_t ngt = 0, neq = 0;
  for (int t0 = beg; t0 < end; t0 += 32) {
    const int t = t0 + lane;
    const uint32_t k = t < end ? key_at(t) : 0u;
    ngt += __popc(__ballot_sync(0xffffffffu, t < end && k > tau));
    neq += __popc(__ballot_sync(0xffffffffu, t < end && k == tau));
  }
  if (lane == 0) { wgt[warp] = ngt; weq[warp] = neq; }
  __syncthreads();
  if (warp == 0) {
    uint32_t a = wgt[lane], e = weq[lane], ia = a, ie = e;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t va = __shfl_up_sync(0xffffffffu, ia, off);
      const uint32_t ve = __shfl_up_sync(0xffffffffu, ie, off);
      if (lane >= off) { ia += va; ie += ve; }
    }
    wgt_base[lane] = ia - a;
    weq_base[lane] = ie - e;
  }
  __syncthreads();
  uint32_t gt_run = wgt_base[warp], eq_run = weq_base[warp];
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (int t0 = beg; t0 < end; t0 += 32) {
    const int t = t0 + lane;
    const uint32_t k = t < end ? key_at(t) : 0u;
    const bool is_gt = t < end && k > tau;
    const bool is_eq = t < end && k == tau;
    const uint32_t bg = __ballot_sync(0xffffffffu, is_gt);
    const uint32_t be = __ballot_sync(0xffffffffu, is_eq);
    const uint32_t gt_before = gt_run + __popc(bg & lt_mask);
    const uint32_t eq_before = eq_run + __popc(be & lt_mask);
    if (is_gt || (is_eq && eq_before < need_eq)) out[gt_before + min(eq_before, need_eq)] = t;
    gt_run += __popc(bg);
    eq_run += __popc(be);
  }
}


// ------------------------------------------------------------------------------------------------
// Register-resident variant for rows of up to 32768 tokens: thread t owns E consecutive positions
// [t*E, (t+1)*E) and keeps their keys in registers (the row is read coalesced into a padded shared-memory
// staging buffer first, then each thread picks up its segment with 16-byte loads).  Three MSB-first
// passes (11 + 11 + 10 bits) find the k-th largest key; after the first pass only the few keys inside
// the threshold bin take part.  Because ownership is contiguous, one block-wide prefix sum over
// per-thread (greater, equal) counts gives every thread the output offset of its first selected
// position, and it writes its positions in ascending order.
constexpr int kRegBins = 2048;
constexpr int kRegCopies = 2;

// Block-wide exclusive prefix sum of one value per thread (T threads); `wsum` holds 2*T/32 words.
template <int T>
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* wsum, int lane, int warp) {
  uint32_t inc = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t u = __shfl_up_sync(0xffffffffu, inc, off);
    if (lane >= off) inc += u;
  }
  if (lane == 31) wsum[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    const uint32_t w = lane < T / 32 ? wsum[lane] : 0u;
    uint32_t wi = w;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t u = __shfl_up_sync(0xffffffffu, wi, off);
      if (lane >= off) wi += u;
    }
    if (lane < T / 32) wsum[T / 32 + lane] = wi - w;
  }
  __syncthreads();
  return wsum[T / 32 + warp] + inc - v;
}

template <int E, int T>
__global__ void __launch_bounds__(T) select_topk_reg_kernel(const SelParams p) {
  extern __shared__ __align__(16) uint32_t smem[];
  uint32_t* hist = smem;                               // [kRegCopies][kRegBins]
  uint32_t* wsum = hist + kRegCopies * kRegBins;       // [2][T/32]
  uint32_t* sh = wsum + 2 * (T / 32);                  // [0] chosen bin, [1] remaining need  (8 words)
  uint32_t* stage = sh + 8;                            // [T][E + 4] keys, each thread's segment padded by 16 bytes

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row = blockIdx.x;
  const int l = row / (p.B * p.Hkv);
  const int rem = row - l * (p.B * p.Hkv);
  const int b = rem / p.Hkv;
  const int g = rem - b * p.Hkv;
  const int c0 = p.cu[b];
  const int N = p.cu[b + 1] - c0;
  const int ck = p.cu_k[b];
  const int kb = p.cu_k[b + 1] - ck;
  if (kb <= 0) return;
  int32_t* out = p.sel_idx + ((int64_t)l * p.Hkv + g) * p.K_tot + ck;
  if (kb >= N) {                                      // whole prompt (or an over-sized budget)
    if (kb > N && tid == 0) raise(p.dev_status, SG_ERR_INVALID);
    for (int j = tid; j < kb; j += T) out[j] = j < N ? j : -1;
    return;
  }
  const uint32_t* x = reinterpret_cast<const uint32_t*>(p.importance) + ((int64_t)l * p.Hkv + g) * p.T + c0;
  for (int i = tid; i < kRegCopies * kRegBins; i += T) hist[i] = 0;
  {
    uint32_t v[E];                                     // all E loads of the thread are issued before the first store
#pragma unroll
    for (int e = 0; e < E; ++e) { const int i = tid + e * T; v[e] = i < N ? __ldg(x + i) : 0u; }
#pragma unroll
    for (int e = 0; e < E; ++e) { const int i = tid + e * T; stage[i + 4 * (i / E)] = i < N ? order_key(v[e]) : 0u; }
  }
  __syncthreads();
  const int first = tid * E;
  uint32_t key[E];
#pragma unroll
  for (int e = 0; e < E; e += 4) {
    const uint4 v = *reinterpret_cast<const uint4*>(stage + tid * (E + 4) + e);
    key[e] = v.x; key[e + 1] = v.y; key[e + 2] = v.z; key[e + 3] = v.w;
  }

  uint32_t prefix = 0, decided = 0, need = (uint32_t)kb;
#pragma unroll 1
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    const int nbins = pass == 2 ? 1024 : 2048;
    const int copies = pass == 0 ? kRegCopies : 1;     // later passes see few candidates: one copy is enough
    uint32_t* my_hist = hist + (warp % copies) * kRegBins;
#pragma unroll
    for (int e = 0; e < E; ++e)
      if (first + e < N && (key[e] & decided) == prefix) atomicAdd(&my_hist[(key[e] >> shift) & (uint32_t)(nbins - 1)], 1u);
    __syncthreads();
    // suffix search: thread t looks at bins nbins-1-t*bpt ... (descending); the bin holding the need-th largest
    constexpr int kBpt = kRegBins / T;                 // bins per thread in an 11-bit pass (half as many in the 10-bit pass)
    const int bpt = nbins / T;
    uint32_t c[kBpt], c2[kBpt];
    const int bin0 = nbins - 1 - tid * bpt;            // this thread's highest bin; it owns bin0, bin0-1, ...
#pragma unroll
    for (int i = 0; i < kBpt; ++i) {                   // all loads first (independent), then the clears for the next pass
      c[i] = i < bpt ? hist[bin0 - i] : 0u;
      c2[i] = (i < bpt && copies > 1) ? hist[kRegBins + bin0 - i] : 0u;
    }
    uint32_t ssum = 0;
#pragma unroll
    for (int i = 0; i < kBpt; ++i) {
      if (i < bpt) { hist[bin0 - i] = 0; if (copies > 1) hist[kRegBins + bin0 - i] = 0; }
      c[i] += c2[i];
      ssum += c[i];
    }
    const uint32_t exc = block_exclusive_scan<T>(ssum, wsum, lane, warp);   // candidates in bins above this thread's
    if (exc < need && need <= exc + ssum) {
      uint32_t run = exc;
#pragma unroll
      for (int i = 0; i < kBpt; ++i) {
        if (run < need && need <= run + c[i]) { sh[0] = (uint32_t)(bin0 - i); sh[1] = need - run; }
        run += c[i];
      }
    }
    __syncthreads();
    prefix |= sh[0] << shift;
    decided |= (uint32_t)(nbins - 1) << shift;
    need = sh[1];
  }
  const uint32_t tau = prefix, need_eq = need;

  // per-thread counts, packed (greater in the low half, equal in the high half), block-wide exclusive prefix
  uint32_t cnt = 0;
#pragma unroll
  for (int e = 0; e < E; ++e)
    if (first + e < N) cnt += (key[e] > tau ? 1u : 0u) + (key[e] == tau ? 0x10000u : 0u);
  const uint32_t before = block_exclusive_scan<T>(cnt, wsum, lane, warp);
  uint32_t gt_before = before & 0xffffu, eq_before = before >> 16;
#pragma unroll
  for (int e = 0; e < E; ++e) {
    if (first + e < N) {
      const bool is_gt = key[e] > tau, is_eq = key[e] == tau;
      if (is_gt || (is_eq && eq_before < need_eq)) out[gt_before + min(eq_before, need_eq)] = first + e;
      gt_before += is_gt ? 1u : 0u;
      eq_before += is_eq ? 1u : 0u;
    }
  }
}

template <int E, int T>
constexpr int select_reg_smem_bytes() { return (kRegCopies * kRegBins + 2 * (T / 32) + 8 + T * (E + 4)) * 4; }

}  // namespace
}  // namespace sg

extern "C" sg_status sg_select_topk(const sg_shape* shape, const float* importance, const int32_t* cu_k,
                                    int32_t total_sel, int32_t* sel_idx, void* workspace,
                                    size_t workspace_bytes, int32_t* dev_status, void* stream) {
  using namespace sg;
  (void)workspace;
  (void)workspace_bytes;
  sg_status st = check_shape(shape, false);
  if (st != SG_OK) return st;
  if (total_sel < 0) return SG_ERR_INVALID;
  if (total_sel == 0) return SG_OK;
  if (!importance || !cu_k || !sel_idx) return SG_ERR_INVALID;
  if (!aligned16(importance) || !aligned16(cu_k) || !aligned16(sel_idx)) return SG_ERR_INVALID;
  SelParams p;
  p.importance = importance;
  p.cu = shape->cu_seqlens;
  p.cu_k = cu_k;
  p.sel_idx = sel_idx;
  p.dev_status = dev_status;
  p.T = shape->total_tokens;
  p.K_tot = total_sel;
  p.B = shape->batch;
  p.Hkv = shape->num_kv_heads;
  const int64_t rows = (int64_t)shape->num_layers * shape->batch * shape->num_kv_heads;
  if (rows > 0x7fffffffLL) return SG_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
#define SG_LAUNCH_SELECT_REG(E, T)                                                         \
  do {                                                                                   \
    SG_ENSURE_SMEM((select_topk_reg_kernel<E, T>), (select_reg_smem_bytes<E, T>()));      \
    select_topk_reg_kernel<E, T><<<(unsigned)rows, T, select_reg_smem_bytes<E, T>(), s>>>(p); \
  } while (0)
  if (shape->max_seqlen <= 4096) {
    SG_LAUNCH_SELECT_REG(8, 512);
  } else if (shape->max_seqlen <= 8192) {
    SG_LAUNCH_SELECT_REG(16, 512);
  } else if (shape->max_seqlen <= 16384) {
    SG_LAUNCH_SELECT_REG(16, 1024);
  } else if (shape->max_seqlen <= 32768) {
    SG_LAUNCH_SELECT_REG(32, 1024);
  } else if (shape->max_seqlen <= kSelKeyCap) {
    const int smem = kSelFixedSmem + shape->max_seqlen * 4;
    SG_ENSURE_SMEM(select_topk_kernel<true>, smem);
    select_topk_kernel<true><<<(unsigned)rows, kSelThreads, smem, s>>>(p);
  } else {
    select_topk_kernel<false><<<(unsigned)rows, kSelThreads, kSelFixedSmem, s>>>(p);
  }
#undef SG_LAUNCH_SELECT_REG
  SG_CUDA_TRY(cudaGetLastError());
  return SG_OK;
}
