// sg_select_topk: per-(layer, sequence, KV head) top-k by exact selection of the k-th largest key.
//
// One CTA owns one importance row.  The row's fp32 values are mapped to order-preserving uint32 keys.
// Rows of up to 32768 tokens keep their keys in registers (second kernel below: histograms over a shrinking
// key interval, direct ranking of the last few keys, output from bit masks; optionally fused with the gather
// of the selected K/V rows).  Longer rows keep the keys in shared memory (up to ~55K tokens) or re-read them
// from L2 (first kernel): four 8-bit MSB-first histogram passes find the k-th largest key exactly and a final
// ordered compaction (ballot + prefix counts, no atomics) emits the selected positions in ascending order.
// Both take equal-to-threshold entries from the lowest positions first.  The result is therefore a pure
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
  int32_t capacity;        // longest row the launched kernel variant can hold (from shape->max_seqlen); 0 = any length
  // fused packing (select_topk_reg_kernel with PD > 0): the CTA that selected a row also gathers its K/V rows
  const uint16_t* k_cache;
  const uint16_t* v_cache;
  uint16_t* packed_k;
  uint16_t* packed_v;
  int64_t ls, ts, hs;
};

// Takes the raw bit pattern: the row is read as uint32 so that no float instruction (and no
// flush-to-zero of subnormals) ever touches the values.
__device__ __forceinline__ uint32_t order_key(uint32_t u) {
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// The selection kernels are launched with programmatic stream serialization: when the kernel before them in the
// stream (normally the scoring kernel) lets its dependents go early, their CTAs are placed while it drains, and
// the launch latency disappears behind it.  Nothing is read before this wait, which returns once that kernel has
// completed and its writes are visible; after a kernel that does not take part it returns at once.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <bool kInSmem>
__global__ void __launch_bounds__(kSelThreads, 1) select_topk_kernel(const SelParams p) {
  pdl_wait();
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
  if (p.capacity > 0 && N > p.capacity) {
    // The row is longer than the shape's max_seqlen promised (the key array was sized from it): flag it and
    // emit an empty row instead of touching memory the launch did not provide.
    if (tid == 0) raise(p.dev_status, SG_ERR_INVALID);
    for (int j = tid; j < kb; j += kSelThreads) out[j] = -1;
    return;
  }
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
// [t*E, (t+1)*E) and keeps their keys in registers (16-byte loads of its own segment when the row is 16-byte
// aligned, else coalesced through a padded shared-memory staging buffer).  At most three histogram passes of
// 2048 bins over a shrinking key interval find the k-th largest key exactly; after the first pass only the few
// keys inside the threshold bin take part.  Because ownership is contiguous, one block-wide prefix sum over
// per-thread (greater, equal) counts gives every thread the output offset of its first selected position, and
// it writes its positions in ascending order from two bit masks.
//
// PD > 0 (head dimension 64 or 128) fuses the packing: the positions also go to shared memory and the same CTA
// copies the row's kb selected K and V rows (16 bytes per thread, kPackUnroll rows in flight per thread group)
// into the packed buffers.  Rows are independent, so while one CTA of an SM is in its latency-bound
// selection another streams rows: the two phases overlap across CTAs without any inter-CTA wait.
constexpr int kPackUnroll = 4;
constexpr int kFinishMax = 64;                         // interval populations up to this are finished by direct ranking
constexpr int64_t kFuseMinRows = kNumSMs;               // fewer rows than SMs cannot fill the machine with their gathers
constexpr int kRegBins = 2048;
constexpr int kRegCopies = 2;

// Block-wide exclusive prefix sum of one value per thread (T threads); `wsum` holds T/32 words.  One barrier: every
// warp adds up the totals of the warps before it by itself.  The caller keeps a barrier between two calls.
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
  const uint32_t before = __reduce_add_sync(0xffffffffu, (lane < T / 32 && lane < warp) ? wsum[lane] : 0u);
  return before + inc - v;
}

template <int E, int T, int PD>
__global__ void __launch_bounds__(T) select_topk_reg_kernel(const SelParams p) {
  pdl_wait();
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
  // fused packing: thread group `grp` (D/8 threads, 16 bytes each) copies selected row j of this (layer, sequence, head)
  auto pack_rows = [&](auto pos_of) {
    if constexpr (PD > 0) {
      constexpr int kTPR = PD / 8, kGroups = T / kTPR;
      const int lane_in_row = tid % kTPR, grp = tid / kTPR;
      const int64_t src0 = (int64_t)l * p.ls + (int64_t)c0 * p.ts + (int64_t)g * p.hs + lane_in_row * 8;
      const int64_t dst0 = (((int64_t)l * p.K_tot + ck) * p.Hkv + (int64_t)g * kb) * PD + lane_in_row * 8;
      // rotating pipeline: kPackUnroll rows per thread group stay in flight; a row's registers are refilled right
      // after its store is issued, so loads never drain while stores go out
      auto load_row = [&](int j, int4& a, int4& b) {
        a = make_int4(0, 0, 0, 0);
        b = make_int4(0, 0, 0, 0);
        if (j < kb) {
          const int t = pos_of(j);
          if (t >= 0) {                                // -1 only behind the end of an over-sized budget: zero rows
            const int64_t src = src0 + (int64_t)t * p.ts;
            a = __ldcs(reinterpret_cast<const int4*>(p.k_cache + src));
            b = __ldcs(reinterpret_cast<const int4*>(p.v_cache + src));
          }
        }
      };
      int4 kv[kPackUnroll][2];
#pragma unroll
      for (int u = 0; u < kPackUnroll; ++u) load_row(grp + u * kGroups, kv[u][0], kv[u][1]);
      for (int j0 = grp; j0 < kb; j0 += kGroups * kPackUnroll) {
#pragma unroll
        for (int u = 0; u < kPackUnroll; ++u) {
          const int j = j0 + u * kGroups;
          if (j < kb) {
            const int64_t dst = dst0 + (int64_t)j * PD;
            __stcs(reinterpret_cast<int4*>(p.packed_k + dst), kv[u][0]);
            __stcs(reinterpret_cast<int4*>(p.packed_v + dst), kv[u][1]);
          }
          load_row(j + kGroups * kPackUnroll, kv[u][0], kv[u][1]);
        }
      }
    }
  };
  if (N > p.capacity) {
    // Longer than the E*T positions this variant holds (it was chosen from shape->max_seqlen, which the row
    // exceeds): flag it, emit an empty row (and zero rows in the fused gather) and leave.
    if (tid == 0) {
      raise(p.dev_status, SG_ERR_INVALID);
      if (PD > 0) raise(p.dev_status, SG_ERR_INDEX);
    }
    for (int j = tid; j < kb; j += T) out[j] = -1;
    pack_rows([&](int) { return -1; });
    return;
  }
  if (kb >= N) {                                      // whole prompt (or an over-sized budget)
    if (kb > N && tid == 0) {
      raise(p.dev_status, SG_ERR_INVALID);
      if (PD > 0) raise(p.dev_status, SG_ERR_INDEX);   // what the packing kernel reports for the -1 entries
    }
    for (int j = tid; j < kb; j += T) out[j] = j < N ? j : -1;
    pack_rows([&](int j) { return j < N ? j : -1; });
    return;
  }
  const uint32_t* x = reinterpret_cast<const uint32_t*>(p.importance) + ((int64_t)l * p.Hkv + g) * p.T + c0;
  for (int i = tid; i < kRegCopies * kRegBins; i += T) hist[i] = 0;
  const int first = tid * E;
  const int nvalid = min(max(N - first, 0), E);        // this thread's positions inside the row
  const uint32_t vmask = nvalid >= 32 ? 0xffffffffu : ((1u << nvalid) - 1u);
  uint32_t key[E];
  if ((reinterpret_cast<uintptr_t>(x) & 15u) == 0) {
    // 16-byte aligned row: every thread reads its own E consecutive values with 16-byte loads (the lines of a
    // warp's first load serve its later ones from L1); no staging, no barrier
    uint4 v[E / 4];
#pragma unroll
    for (int q = 0; q < E / 4; ++q) {
      const int i = first + 4 * q;
      if (i + 3 < N) {
        v[q] = __ldg(reinterpret_cast<const uint4*>(x + i));
      } else {
        v[q].x = i < N ? __ldg(x + i) : 0u;
        v[q].y = i + 1 < N ? __ldg(x + i + 1) : 0u;
        v[q].z = i + 2 < N ? __ldg(x + i + 2) : 0u;
        v[q].w = 0u;
      }
    }
#pragma unroll
    for (int q = 0; q < E / 4; ++q) {
      key[4 * q] = order_key(v[q].x); key[4 * q + 1] = order_key(v[q].y);
      key[4 * q + 2] = order_key(v[q].z); key[4 * q + 3] = order_key(v[q].w);
    }
    __syncthreads();                                   // histogram cleared
  } else {
    {
      uint32_t v[E];                                   // all E loads of the thread are issued before the first store
#pragma unroll
      for (int e = 0; e < E; ++e) { const int i = tid + e * T; v[e] = i < N ? __ldg(x + i) : 0u; }
#pragma unroll
      for (int e = 0; e < E; ++e) { const int i = tid + e * T; stage[i + 4 * (i / E)] = i < N ? order_key(v[e]) : 0u; }
    }
    __syncthreads();
#pragma unroll
    for (int e = 0; e < E; e += 4) {
      const uint4 v = *reinterpret_cast<const uint4*>(stage + tid * (E + 4) + e);
      key[e] = v.x; key[e + 1] = v.y; key[e + 2] = v.z; key[e + 3] = v.w;
    }
  }

  // ---- exact k-th largest key by narrowing a key interval [lo, hi] that holds it, 11 bits of the interval per pass.
  // The digit of a pass is (key - lo) >> shift with shift chosen so that the interval spans at most 2048 bins:
  // unlike the fixed top bits of a float, it spreads whatever range the row really has over all bins, so the
  // threshold bin of the first pass keeps tens of keys, not a quarter of the row, and the later passes touch few.
  uint32_t kmin = 0xffffffffu, kmax = 0u;
#pragma unroll
  for (int e = 0; e < E; ++e)
    if ((vmask >> e) & 1u) { kmin = min(kmin, key[e]); kmax = max(kmax, key[e]); }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if (lane == 0) { wsum[warp] = kmin; wsum[T / 32 + warp] = kmax; }
  __syncthreads();
  kmin = __reduce_min_sync(0xffffffffu, lane < T / 32 ? wsum[lane] : 0xffffffffu);
  kmax = __reduce_max_sync(0xffffffffu, lane < T / 32 ? wsum[T / 32 + lane] : 0u);
  __syncthreads();                                     // wsum is reused by the scans below
  uint32_t lo = kmin, hi = kmax, need = (uint32_t)kb;
#pragma unroll 1
  for (int pass = 0; lo != hi; ++pass) {
    const uint32_t width = hi - lo;
    const int shift = max(0, 32 - __clz(width) - 11);
    const int copies = pass == 0 ? kRegCopies : 1;     // later passes see few candidates: one copy is enough
    uint32_t* my_hist = hist + (warp % copies) * kRegBins;
#pragma unroll
    for (int e = 0; e < E; ++e) {
      const uint32_t rel = key[e] - lo;
      if (((vmask >> e) & 1u) && rel <= width) atomicAdd(&my_hist[rel >> shift], 1u);
    }
    __syncthreads();
    // suffix search: thread t looks at bins 2047-t*bpt ... (descending) for the bin holding the need-th largest
    constexpr int kBpt = kRegBins / T;
    uint32_t c[kBpt];
    const int bin0 = kRegBins - 1 - tid * kBpt;        // this thread's highest bin; it owns bin0, bin0-1, ...
    uint32_t ssum = 0;
#pragma unroll
    for (int i = 0; i < kBpt; ++i) {
      c[i] = hist[bin0 - i];
      if (copies > 1) c[i] += hist[kRegBins + bin0 - i];
    }
#pragma unroll
    for (int i = 0; i < kBpt; ++i) {                   // cleared for the next pass
      hist[bin0 - i] = 0;
      if (copies > 1) hist[kRegBins + bin0 - i] = 0;
      ssum += c[i];
    }
    const uint32_t exc = block_exclusive_scan<T>(ssum, wsum, lane, warp);   // candidates in bins above this thread's
    if (exc < need && need <= exc + ssum) {
      uint32_t run = exc;
#pragma unroll
      for (int i = 0; i < kBpt; ++i) {
        if (run < need && need <= run + c[i]) { sh[0] = (uint32_t)(bin0 - i); sh[1] = need - run; sh[2] = c[i]; sh[3] = 0; }
        run += c[i];
      }
    }
    __syncthreads();
    lo += sh[0] << shift;
    hi = lo + min(hi - lo, (1u << shift) - 1u);
    need = sh[1];
    const uint32_t ncand = sh[2];
    if (lo != hi && ncand <= (uint32_t)kFinishMax) {
      // Few keys left in the interval: instead of more block-wide passes, gather them and let one thread per key
      // count the keys above it and equal to it; the key whose rank range covers `need` is the threshold.
      uint32_t* list = stage;
      const uint32_t w = hi - lo;
#pragma unroll
      for (int e = 0; e < E; ++e)
        if (((vmask >> e) & 1u) && key[e] - lo <= w) list[atomicAdd(&sh[3], 1u)] = key[e];
      __syncthreads();
      if (tid < (int)ncand) {
        const uint32_t k = list[tid];
        uint32_t above = 0, same = 0;
        for (uint32_t j = 0; j < ncand; ++j) {
          const uint32_t o = list[j];
          above += o > k ? 1u : 0u;
          same += o == k ? 1u : 0u;
        }
        if (above < need && need <= above + same) { sh[4] = k; sh[5] = need - above; }   // equal keys write equal values
      }
      __syncthreads();
      lo = hi = sh[4];
      need = sh[5];
    }
  }
  const uint32_t tau = lo, need_eq = need;

  // per-thread bit masks of the positions above / equal to the threshold; their counts, packed (greater in the low half,
  // equal in the high half), go through one block-wide exclusive prefix sum
  uint32_t mgt = 0, meq = 0;
#pragma unroll
  for (int e = 0; e < E; ++e) {
    mgt |= (key[e] > tau ? 1u : 0u) << e;
    meq |= (key[e] == tau ? 1u : 0u) << e;
  }
  mgt &= vmask;
  meq &= vmask;
  const uint32_t cnt = (uint32_t)__popc(mgt) | ((uint32_t)__popc(meq) << 16);
  const uint32_t before = block_exclusive_scan<T>(cnt, wsum, lane, warp);
  const uint32_t gt_before = before & 0xffffu, eq_before = before >> 16;
  // of this thread's equal entries only the first (need_eq - eq_before) are kept: drop the highest ones beyond that
  int extra = __popc(meq) - (int)(need_eq > eq_before ? min(need_eq - eq_before, (uint32_t)E) : 0u);
  while (extra > 0) { meq &= ~(0x80000000u >> __clz(meq)); --extra; }
  uint32_t m = mgt | meq;
  uint32_t slot = gt_before + min(eq_before, need_eq);
  while (m) {                                          // ascending positions
    const int e = __ffs(m) - 1;
    m &= m - 1;
    out[slot] = first + e;
    if constexpr (PD > 0) stage[slot] = (uint32_t)(first + e);
    ++slot;
  }
  if constexpr (PD > 0) {
    __syncthreads();
    pack_rows([&](int j) { return (int)stage[j]; });
  }
}

template <int E, int T>
constexpr int select_reg_smem_bytes() { return (kRegCopies * kRegBins + 2 * (T / 32) + 8 + T * (E + 4)) * 4; }

}  // namespace
}  // namespace sg

namespace sg {
namespace {
// Launches the selection; with `fuse` the register-resident kernels also pack (the caller has checked that the rows fit them).
sg_status select_launch(const sg_shape* shape, SelParams& p, bool fuse, void* stream) {
  const int64_t rows = (int64_t)shape->num_layers * shape->batch * shape->num_kv_heads;
  if (rows > 0x7fffffffLL) return SG_ERR_UNSUPPORTED;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.stream = static_cast<cudaStream_t>(stream);
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3((unsigned)rows);
  const int pd = fuse ? shape->head_dim : 0;
#define SG_LAUNCH_SELECT_REG_PD(E, T, PD)                                                       \
  do {                                                                                          \
    p.capacity = (E) * (T);                                                                     \
    SG_ENSURE_SMEM((select_topk_reg_kernel<E, T, PD>), (select_reg_smem_bytes<E, T>()));         \
    cfg.blockDim = dim3(T);                                                                     \
    cfg.dynamicSmemBytes = select_reg_smem_bytes<E, T>();                                       \
    SG_CUDA_TRY(cudaLaunchKernelEx(&cfg, select_topk_reg_kernel<E, T, PD>, p));                  \
  } while (0)
#define SG_LAUNCH_SELECT_REG(E, T)                        \
  do {                                                    \
    if (pd == 128) SG_LAUNCH_SELECT_REG_PD(E, T, 128);    \
    else if (pd == 64) SG_LAUNCH_SELECT_REG_PD(E, T, 64); \
    else SG_LAUNCH_SELECT_REG_PD(E, T, 0);                \
  } while (0)
  if (rows < kNumSMs && !fuse && shape->max_seqlen <= 8192 && shape->max_seqlen > 4096) {
    // fewer rows than SMs: one CTA per SM anyway, so twice the threads per row (half the keys each) shorten the chains
    SG_LAUNCH_SELECT_REG_PD(8, 1024, 0);
  } else if (shape->max_seqlen <= 4096) {
    SG_LAUNCH_SELECT_REG(8, 512);
  } else if (shape->max_seqlen <= 8192) {
    SG_LAUNCH_SELECT_REG(16, 512);
  } else if (shape->max_seqlen <= 16384) {
    SG_LAUNCH_SELECT_REG(16, 1024);
  } else if (shape->max_seqlen <= 32768) {
    SG_LAUNCH_SELECT_REG(32, 1024);
  } else if (fuse) {
    return SG_ERR_UNSUPPORTED;
  } else if (shape->max_seqlen <= kSelKeyCap) {
    const int smem = kSelFixedSmem + shape->max_seqlen * 4;
    p.capacity = shape->max_seqlen;
    SG_ENSURE_SMEM(select_topk_kernel<true>, smem);
    cfg.blockDim = dim3(kSelThreads);
    cfg.dynamicSmemBytes = smem;
    SG_CUDA_TRY(cudaLaunchKernelEx(&cfg, select_topk_kernel<true>, p));
  } else {
    p.capacity = 0;                                    // keys are re-read from global memory: any length
    cfg.blockDim = dim3(kSelThreads);
    cfg.dynamicSmemBytes = kSelFixedSmem;
    SG_CUDA_TRY(cudaLaunchKernelEx(&cfg, select_topk_kernel<false>, p));
  }
#undef SG_LAUNCH_SELECT_REG
#undef SG_LAUNCH_SELECT_REG_PD
  SG_CUDA_TRY(cudaGetLastError());
  return SG_OK;
}
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
  SelParams p = {};
  p.importance = importance;
  p.cu = shape->cu_seqlens;
  p.cu_k = cu_k;
  p.sel_idx = sel_idx;
  p.dev_status = dev_status;
  p.T = shape->total_tokens;
  p.K_tot = total_sel;
  p.B = shape->batch;
  p.Hkv = shape->num_kv_heads;
  return select_launch(shape, p, false, stream);
}

extern "C" sg_status sg_select_pack_kv(const sg_shape* shape, const float* importance, const int32_t* cu_k,
                                       int32_t total_sel, const void* k_cache, const void* v_cache, int32_t* sel_idx,
                                       void* packed_k, void* packed_v, int32_t* dev_status, void* stream) {
  using namespace sg;
  sg_status st = check_shape(shape, false);
  if (st != SG_OK) return st;
  if (total_sel < 0) return SG_ERR_INVALID;
  if (total_sel == 0) return SG_OK;
  if (!importance || !cu_k || !sel_idx || !k_cache || !v_cache || !packed_k || !packed_v) return SG_ERR_INVALID;
  if (!aligned16(importance) || !aligned16(cu_k) || !aligned16(sel_idx) || !aligned16(k_cache) || !aligned16(v_cache) ||
      !aligned16(packed_k) || !aligned16(packed_v))
    return SG_ERR_INVALID;
  // One fused launch pays when the rows fit the register-resident kernels and there are enough of them to keep every SM
  // streaming while others select; otherwise the two kernels run back to back.
  const int64_t rows = (int64_t)shape->num_layers * shape->batch * shape->num_kv_heads;
  const bool fuse = shape->max_seqlen <= 32768 && rows >= kFuseMinRows;
  if (!fuse) {
    st = sg_select_topk(shape, importance, cu_k, total_sel, sel_idx, nullptr, 0, dev_status, stream);
    if (st != SG_OK) return st;
    return sg_pack_kv(shape, k_cache, v_cache, sel_idx, cu_k, total_sel, packed_k, packed_v, dev_status, stream);
  }
  SelParams p = {};
  p.importance = importance;
  p.cu = shape->cu_seqlens;
  p.cu_k = cu_k;
  p.sel_idx = sel_idx;
  p.dev_status = dev_status;
  p.T = shape->total_tokens;
  p.K_tot = total_sel;
  p.B = shape->batch;
  p.Hkv = shape->num_kv_heads;
  p.k_cache = static_cast<const uint16_t*>(k_cache);
  p.v_cache = static_cast<const uint16_t*>(v_cache);
  p.packed_k = static_cast<uint16_t*>(packed_k);
  p.packed_v = static_cast<uint16_t*>(packed_v);
  p.ls = shape->cache_layer_stride;
  p.ts = shape->cache_token_stride;
  p.hs = shape->cache_head_stride;
  return select_launch(shape, p, true, stream);
}
