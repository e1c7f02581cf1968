// sg_sparse_decode_attn: split-KV decode attention over a packed source plus an index-gathered source.
//
// Memory-bound: every attended token costs 2*d*2 bytes of K+V per KV head and only 4*G*d flops.
// The token list of a (sequence, KV head) -- packed rows first, then local rows addressed through
// local_idx -- is cut into slices of 16 tokens.  The slices are dealt out round robin over all warps of all
// CTAs that share a (sequence, KV head), so every CTA gets the same mix of packed and gathered slices; a warp
// streams its slices through a ring of three K/V slices of its own in shared memory (16-byte cp.async copies, XOR-swizzled rows so ldmatrix is
// conflict-free; gathered rows are whole 2*d-byte lines, so sector efficiency stays 100 %).  The ring is
// private to the warp, so the loop has no block-wide barrier: a warp waits only for its own copies.
// S = Q K^T and O += P V run on bf16 tensor-core MMAs with the G query rows of the KV head padded to
// 16; the online softmax (base 2) stays in registers.
// The split-KV partials (m, l, unnormalised O) never leave the chip: the warps of a CTA merge through
// shared memory, and the CTAs of a (sequence, KV head) form a thread-block cluster (1, 2, 4 or 8 CTAs);
// every CTA owns a slice of the G*d outputs and receives the other CTAs' partials of that slice in its own
// shared memory (remote stores that report their bytes to an mbarrier of the owner, so only the owner's merging
// threads wait, and only for what is addressed to them), then merges them with the log-sum-exp rule
// (m = max m_j, l = sum l_j 2^(m_j-m), o = sum o_j 2^(m_j-m) / l) and writes bf16 out and fp32 lse.
// One launch, no workspace.
// (Measured and dropped: a two-kernel variant with partials in HBM, 2x slower on long single-sequence
// lists; clusters of 16, few of which can be co-scheduled; a block-wide ring of 64-token tiles with a
// barrier per tile, 10-25 % slower at every size.)
// The launch uses programmatic dependent launch, so back-to-back decode calls overlap their launch
// latency and prologue with the previous call's tail.
#include "common.cuh"
#include "launch.h"

namespace sg {
namespace {

constexpr int kSlice = 16;         // tokens per warp step (one m16n8k16 k-extent of P V)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct DecParams {
  const uint16_t* q;
  const uint16_t* packed_k;
  const uint16_t* packed_v;
  const uint16_t* local_k;
  const uint16_t* local_v;
  const int32_t* cu;
  const int32_t* cu_k;
  const int32_t* cu_nloc;
  const int32_t* local_idx;
  const int32_t* packed_count;   // [B][Hkv] packed rows of a (sequence, KV head) that are in the list, or null: all k_b
  const int32_t* local_skip;     // [B][Hkv] leading entries of the head's local-index row that are not in the list, or null
  uint16_t* out;
  float* lse;
  int32_t* dev_status;
  int64_t ts, hs;
  int32_t B, Hq, Hkv, G, K_tot, NL_tot;
  int32_t n_tokens;  // total tokens of the batch: with one sequence every prefix array is {0, total}, known on the host
  int32_t csize;     // CTAs per (sequence, KV head) = cluster size
  float scale_log2;
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory"); }
// Remote stores that report their bytes to an mbarrier of the destination CTA: the owner of an output slice waits on
// its own barrier for everybody's partials instead of the whole cluster meeting at a barrier.
__device__ __forceinline__ void st_async_f32(float* local_ptr, uint64_t* local_bar, uint32_t cta_rank, float v) {
  uint32_t raddr, rbar;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(raddr) : "r"(smem_u32(local_ptr)), "r"(cta_rank));
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(rbar) : "r"(smem_u32(local_bar)), "r"(cta_rank));
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];\n" ::"r"(raddr), "f"(v), "r"(rbar) : "memory");
}
__device__ __forceinline__ void st_async_f32x2(float* local_ptr, uint64_t* local_bar, uint32_t cta_rank, float a, float b) {
  uint32_t raddr, rbar;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(raddr) : "r"(smem_u32(local_ptr)), "r"(cta_rank));
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(rbar) : "r"(smem_u32(local_bar)), "r"(cta_rank));
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];\n" ::"r"(raddr), "f"(a), "f"(b), "r"(rbar) : "memory");
}
__device__ __forceinline__ void cluster_arrive_release() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
}
// Bounded wait for phase 0 of an mbarrier whose bytes come from other CTAs of the cluster; false when it gave up.
__device__ __forceinline__ bool mbar_wait_cluster_bounded(uint64_t* bar) {
  const uint32_t addr = smem_u32(bar);
  const long long t0 = clock64();
  do {                                                      // the senders run concurrently (same cluster): microseconds; the limit is ~0.5 s
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(done) : "r"(addr) : "memory");
    if (done) return true;
  } while (clock64() - t0 < 1000000000LL);
  return false;
}
// Programmatic dependent launch: let the next kernel in the stream start its prologue now, and wait
// for the previous kernel's memory before touching anything it may have written.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// kHi: the KV head has more than 8 query rows, so MMA rows 8..15 carry data too.
// kDecWarps warps per CTA, each with a private ring of kBuf slices: (8, 3) gives one CTA per SM, (4, 3) two.
template <int D, bool kHi, int kDecWarps, int kBuf>
__global__ void __launch_bounds__(kDecWarps * 32, kDecWarps == 4 ? 2 : 1) decode_partial_kernel(const DecParams p) {
  constexpr int kDecThreads = kDecWarps * 32;
  constexpr int kRowBytes = D * 2;
  constexpr int kChunksPerRow = D / 8;                       // 16-byte chunks
  constexpr int kSliceBytes = kSlice * kRowBytes;            // K (or V) rows of one slice
  constexpr int kCopiesPerLane = kSlice * kChunksPerRow / 32;
  constexpr uint32_t kFull = 0xffffffffu;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  // per warp: kBuf slices of K, then kBuf slices of V, rows XOR-swizzled; after all rings one validity
  // word per (warp, buffer)
  uint32_t* s_mask = reinterpret_cast<uint32_t*>(smem_raw + kDecWarps * kBuf * 2 * kSliceBytes);
  // Receive area for the cluster merge, never aliased by the rings: the slice of the G*d outputs this CTA
  // owns, as every rank's partial: rx_o [8][per], rx_m [8][16], rx_l [8][16].
  float* rx_m = reinterpret_cast<float*>(s_mask + kDecWarps * kBuf);
  float* rx_l = rx_m + 8 * 16;
  float* rx_o = rx_l + 8 * 16;
  uint64_t* rx_bar = reinterpret_cast<uint64_t*>(rx_o + 16 * D);   // counts the bytes of the partials pushed into the three arrays

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = blockIdx.y;
  pdl_launch_dependents();
  if (p.csize > 1) {
    if (tid == 0) {
      // every rank sends this CTA its partial of the slice owned here and its (M, L) of the G rows
      const int per0 = (p.G * D + p.csize - 1) / p.csize;
      const int c_rank = blockIdx.x % p.csize;
      const int own = max(0, min(p.G * D, (c_rank + 1) * per0) - c_rank * per0);
      const uint32_t bytes = (uint32_t)p.csize * (uint32_t)(own + 2 * p.G) * 4u;
      const uint32_t bar = smem_u32(rx_bar);
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(bar) : "memory");
      asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
    }
    cluster_arrive_release();                                  // "this CTA runs, its barrier is set up": awaited before the first remote store
  }
  const int b = blockIdx.x / p.csize;                          // grid.x = B * cluster size
  const int c = blockIdx.x - b * p.csize;                      // rank in the cluster
  // A single sequence (the latency-critical case) needs no prefix loads: a dependent round trip to L2 less before the
  // first copy can be issued.
  const bool one = p.B == 1;
  const int ck0 = one ? 0 : p.cu_k[b];
  const int kb = one ? p.K_tot : p.cu_k[b + 1] - ck0;          // packed rows per KV head (the slot size in the buffer)
  const int kbe = p.packed_count ? min(kb, max(0, __ldg(p.packed_count + (int64_t)b * p.Hkv + g))) : kb;   // ... of which in the list
  const int cl0 = one ? 0 : p.cu_nloc[b];
  const int nl_row = one ? p.NL_tot : p.cu_nloc[b + 1] - cl0;
  const int lskip = p.local_skip ? min(nl_row, max(0, __ldg(p.local_skip + (int64_t)b * p.Hkv + g))) : 0;
  const int nl = nl_row - lskip;
  const int c0 = one ? 0 : p.cu[b];
  const int nseq = one ? p.n_tokens : p.cu[b + 1] - c0;

  const uint16_t* pk_base = p.packed_k + ((int64_t)ck0 * p.Hkv + (int64_t)g * kb) * D;
  const uint16_t* pv_base = p.packed_v + ((int64_t)ck0 * p.Hkv + (int64_t)g * kb) * D;
  const uint16_t* lk_base = p.local_k + (int64_t)c0 * p.ts + (int64_t)g * p.hs;
  const uint16_t* lv_base = p.local_v + (int64_t)c0 * p.ts + (int64_t)g * p.hs;
  const uint32_t wk_u32 = smem_u32(smem_raw) + warp * (kBuf * 2 * kSliceBytes);   // this warp's K ring
  const uint32_t wv_u32 = wk_u32 + kBuf * kSliceBytes;                            // and its V ring

  // The slices of the list [packed rows ++ local rows] of (b, g) are dealt out round robin over all warps of all CTAs of
  // the cluster (slice s goes to rank s % csize, warp (s / csize) % warps): every CTA gets the same mix of contiguous
  // packed slices and slower gathered ones, whatever the split of the list.
  constexpr int pos_beg = 0;
  const int ntok = kbe + nl;
  const int nslices = (ntok + kSlice - 1) / kSlice;
  const int first_slice = warp * p.csize + c, slice_stride = kDecWarps * p.csize;
  const int nmine = nslices > first_slice ? (nslices - first_slice + slice_stride - 1) / slice_stride : 0;
  const int32_t* idx_base = p.local_idx + (int64_t)g * p.NL_tot + cl0 + lskip - kbe;   // indexed by list position
  // Lane r (and r + 16) holds the local index of row r of the warp's j-th slice, read one slice ahead.
  auto fetch_idx = [&](int j) -> int {
    const int li = (first_slice + j * slice_stride) * kSlice + (lane & 15);
    const int pos = pos_beg + li;
    return (j < nmine && li < ntok && pos >= kbe) ? __ldg(idx_base + pos) : 0;
  };
  auto load_slice = [&](int j, int buf, int idx_reg) {
    const int li0 = (first_slice + j * slice_stride) * kSlice;
    if (li0 + kSlice <= ntok && pos_beg + li0 + kSlice <= kbe) {
      // the whole slice lies in the packed buffer: 16 consecutive rows are one contiguous run of 16-byte pieces
      if (lane == 0) s_mask[warp * kBuf + buf] = 0xffffu;
      const uint16_t* srck = pk_base + (int64_t)(pos_beg + li0) * D + lane * 8;
      const uint16_t* srcv = pv_base + (int64_t)(pos_beg + li0) * D + lane * 8;
#pragma unroll
      for (int i = 0; i < kCopiesPerLane; ++i) {
        const int qid = lane + i * 32;
        const int row = qid / kChunksPerRow;
        const int col = qid % kChunksPerRow;
        const uint32_t off = buf * kSliceBytes + row * kRowBytes + ((col ^ (row & 7)) << 4);
        cp_async16(wk_u32 + off, srck + i * 256, 16);
        cp_async16(wv_u32 + off, srcv + i * 256, 16);
      }
      return;
    }
    {
      const int li = li0 + (lane & 15), pos = pos_beg + li;
      const bool in_list = li < ntok;
      const bool ok = in_list && (pos < kbe || (idx_reg >= 0 && idx_reg < nseq));
      if (in_list && !ok && lane < 16) raise(p.dev_status, SG_ERR_INDEX);
      const uint32_t mask = __ballot_sync(kFull, ok) & 0xffffu;
      if (lane == 0) s_mask[warp * kBuf + buf] = mask;        // bit r: row r holds a real token
    }
#pragma unroll
    for (int i = 0; i < kCopiesPerLane; ++i) {
      const int qid = lane + i * 32;
      const int row = qid / kChunksPerRow;
      const int col = qid % kChunksPerRow;
      const int li = li0 + row;
      const int pos = pos_beg + li;
      const int t = __shfl_sync(kFull, idx_reg, row);
      const uint16_t* srck = p.packed_k;
      const uint16_t* srcv = p.packed_v;
      int bytes = 0;
      if (li < ntok) {
        if (pos < kbe) {
          srck = pk_base + (int64_t)pos * D + col * 8;
          srcv = pv_base + (int64_t)pos * D + col * 8;
          bytes = 16;
        } else if (t >= 0 && t < nseq) {
          srck = lk_base + (int64_t)t * p.ts + col * 8;
          srcv = lv_base + (int64_t)t * p.ts + col * 8;
          bytes = 16;
        }
      }
      const uint32_t off = buf * kSliceBytes + row * kRowBytes + ((col ^ (row & 7)) << 4);
      cp_async16(wk_u32 + off, srck, bytes);                  // bytes == 0 zero-fills the row
      cp_async16(wv_u32 + off, srcv, bytes);
    }
  };

  float o_acc[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) { o_acc[i][0] = o_acc[i][1] = o_acc[i][2] = o_acc[i][3] = 0.f; }
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

  int idx_next;
  {
    int idx_pro[kBuf - 1];
#pragma unroll
    for (int s = 0; s < kBuf - 1; ++s) idx_pro[s] = fetch_idx(s);
    idx_next = fetch_idx(kBuf - 1);
    static_assert(kBuf == 3, "the prologue below passes two index registers by selection");
#pragma unroll 1
    for (int s = 0; s < kBuf - 1; ++s) {                      // not unrolled: this code runs once per call, from a cold instruction cache
      if (s < nmine) load_slice(s, s, s ? idx_pro[1] : idx_pro[0]);
      cp_async_commit();
    }
  }

  // Everything in this kernel up to its output stores reads only inputs of the decode step -- the KV sources, the
  // index lists, the prefix arrays and the query rows -- which the contract treats as stable: they must not be
  // written by a kernel that itself lets its dependents start early (such as the previous layer's call of this
  // kernel).  So nothing waits here: the dependency wait sits in front of the stores of out / lse, and consecutive
  // calls overlap everything but those stores.
  // Q fragments (A operand, 16 x D, rows >= G are zero).
  const int r_lo = lane >> 2, r_hi = r_lo + 8;
  uint32_t qa[D / 16][4];
  {
    const uint16_t* qb = p.q + ((int64_t)b * p.Hq + (int64_t)g * p.G) * D;
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
      const int col = kk * 16 + 2 * (lane & 3);
      qa[kk][0] = r_lo < p.G ? *reinterpret_cast<const uint32_t*>(qb + r_lo * D + col) : 0u;
      qa[kk][2] = r_lo < p.G ? *reinterpret_cast<const uint32_t*>(qb + r_lo * D + col + 8) : 0u;
      qa[kk][1] = (kHi && r_hi < p.G) ? *reinterpret_cast<const uint32_t*>(qb + r_hi * D + col) : 0u;
      qa[kk][3] = (kHi && r_hi < p.G) ? *reinterpret_cast<const uint32_t*>(qb + r_hi * D + col + 8) : 0u;
    }
  }

  // The ring is private to the warp: no block-wide barrier inside the loop, the warps drift freely.
#pragma unroll 1
  for (int j = 0; j < nmine; ++j) {
    cp_async_wait<kBuf - 2>();
    __syncwarp();
    {
      const int nj = j + kBuf - 1;
      if (nj < nmine) load_slice(nj, nj % kBuf, idx_next);
      cp_async_commit();
      idx_next = fetch_idx(nj + 1);
    }
    const int buf = j % kBuf;
    const uint32_t k_st = wk_u32 + buf * kSliceBytes;
    const uint32_t v_st = wv_u32 + buf * kSliceBytes;
    const uint32_t vmask = s_mask[warp * kBuf + buf];
    constexpr int wrow = 0;

    // S = Q K^T for 16 tokens (two n8 tiles)
    // (even and odd k-steps accumulate separately: two dependent chains of half the length; a warp has only one or two
    // slices at small batch, so the length of this chain is what it waits for)
    float s_acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    {
      float s_odd[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      const int mi = lane >> 3;
      const int row = wrow + (mi >> 1) * 8 + (lane & 7);
      // all fragment loads of the slice first, then the tensor-core chain: the statements are volatile and keep their
      // order, so loading inside the chain would expose one shared-memory latency per k-step
      uint32_t kf[D / 16][4];
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        const int chunk = kk * 2 + (mi & 1);
        ldmatrix_x4(kf[kk], k_st + row * kRowBytes + ((chunk ^ (row & 7)) << 4));
      }
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        mma_bf16((kk & 1) ? s_odd[0] : s_acc[0], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], kf[kk][0], kf[kk][1]);
        mma_bf16((kk & 1) ? s_odd[1] : s_acc[1], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], kf[kk][2], kf[kk][3]);
      }
#pragma unroll
      for (int j = 0; j < 2; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) s_acc[j][e] += s_odd[j][e];
      }
    }
    // the V fragments are fetched now, ahead of the softmax arithmetic that P V has to wait for anyway
    uint32_t vf[D / 16][4];
    {
      const int mi = lane >> 3;
      const int row = wrow + (mi & 1) * 8 + (lane & 7);
#pragma unroll
      for (int dc = 0; dc < D / 16; ++dc) {
        const int chunk = dc * 2 + (mi >> 1);
        ldmatrix_x4_trans(vf[dc], v_st + row * kRowBytes + ((chunk ^ (row & 7)) << 4));
      }
    }
    // online softmax in base 2; mask padding and skipped indices
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const bool valid = (vmask >> (j * 8 + 2 * (lane & 3) + e)) & 1u;
        s_acc[j][e] = valid ? s_acc[j][e] * p.scale_log2 : -INFINITY;
        mx_lo = fmaxf(mx_lo, s_acc[j][e]);
        if (kHi) {
          s_acc[j][2 + e] = valid ? s_acc[j][2 + e] * p.scale_log2 : -INFINITY;
          mx_hi = fmaxf(mx_hi, s_acc[j][2 + e]);
        }
      }
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    const float mn_lo = fmaxf(m_lo, mx_lo);
    const float mu_lo = mn_lo == -INFINITY ? 0.f : mn_lo;
    const float al_lo = exp2f(m_lo - mu_lo);
    m_lo = mn_lo;
    float mu_hi = 0.f, al_hi = 1.f;
    if (kHi) {
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
      const float mn_hi = fmaxf(m_hi, mx_hi);
      mu_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
      al_hi = exp2f(m_hi - mu_hi);
      m_hi = mn_hi;
    }
    float sum_lo = 0.f, sum_hi = 0.f;
    uint32_t pa[4];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const float p0 = exp2f(s_acc[j][0] - mu_lo), p1 = exp2f(s_acc[j][1] - mu_lo);
      sum_lo += p0 + p1;
      pa[2 * j] = pack_bf16(p0, p1);
      if (kHi) {
        const float p2 = exp2f(s_acc[j][2] - mu_hi), p3 = exp2f(s_acc[j][3] - mu_hi);
        sum_hi += p2 + p3;
        pa[2 * j + 1] = pack_bf16(p2, p3);
      } else {
        pa[2 * j + 1] = 0u;
      }
    }
    // the four lanes of a row keep their own part of the row sum (the rescale factor is the same for all four);
    // the parts are added up once, after the last slice
    l_lo = l_lo * al_lo + sum_lo;
    if (kHi) l_hi = l_hi * al_hi + sum_hi;
    const bool rescale = kHi ? (al_lo != 1.f || al_hi != 1.f) : (al_lo != 1.f);
    if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
      for (int i = 0; i < D / 8; ++i) {
        o_acc[i][0] *= al_lo; o_acc[i][1] *= al_lo;
        if (kHi) { o_acc[i][2] *= al_hi; o_acc[i][3] *= al_hi; }
      }
    }
    // O += P V
#pragma unroll
    for (int dc = 0; dc < D / 16; ++dc) {
      mma_bf16(o_acc[2 * dc], pa[0], pa[1], pa[2], pa[3], vf[dc][0], vf[dc][1]);
      mma_bf16(o_acc[2 * dc + 1], pa[0], pa[1], pa[2], pa[3], vf[dc][2], vf[dc][3]);
    }
  }
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  if (kHi) {
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  }
  cp_async_wait<0>();
  __syncthreads();

  // merge the warps through shared memory (the rings are free now)
  constexpr int kOStride = D + 8;                             // row stride of the partials: the rows of a store land in different banks
  float* sm_o = reinterpret_cast<float*>(smem_raw);           // [kDecWarps][16][kOStride]
  float* sm_m = sm_o + kDecWarps * 16 * kOStride;             // [kDecWarps][16]
  float* sm_l = sm_m + kDecWarps * 16;
  const bool w_lo = r_lo < p.G, w_hi = kHi && r_hi < p.G;      // rows >= G are padding and never read
  if ((lane & 3) == 0) {
    if (w_lo) { sm_m[warp * 16 + r_lo] = m_lo; sm_l[warp * 16 + r_lo] = l_lo; }
    if (w_hi) { sm_m[warp * 16 + r_hi] = m_hi; sm_l[warp * 16 + r_hi] = l_hi; }
  }
#pragma unroll
  for (int i = 0; i < D / 8; ++i) {
    const int col = i * 8 + 2 * (lane & 3);
    float* dst = sm_o + (warp * 16 + r_lo) * kOStride + col;
    if (w_lo) *reinterpret_cast<float2*>(dst) = make_float2(o_acc[i][0], o_acc[i][1]);
    if (w_hi) *reinterpret_cast<float2*>(dst + 8 * kOStride) = make_float2(o_acc[i][2], o_acc[i][3]);
  }
  __syncthreads();
  // CTA-level partial of every output; with a cluster, each rank owns a slice of the G*d outputs and
  // every CTA pushes its partial of a slice into the owner's receive area (distributed shared memory).
  const int cs = p.csize;
  const int per = (p.G * D + cs - 1) / cs;
  __nv_bfloat16* outp = reinterpret_cast<__nv_bfloat16*>(p.out) + ((int64_t)b * p.Hq + (int64_t)g * p.G) * D;
  float* lsep = p.lse ? p.lse + (int64_t)b * p.Hq + (int64_t)g * p.G : nullptr;
  if (cs > 1) cluster_wait();                                  // every CTA of the cluster has started
  if (cs == 1) pdl_wait();                                     // out / lse are written below: all earlier work in the stream first
  // two neighbouring outputs per thread (same row, same owner: D and the owners' slices are even)
  for (int e = 2 * tid; e < p.G * D; e += 2 * kDecThreads) {
    const int r = e / D, col = e - r * D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, sm_m[w * 16 + r]);
    const float Mu = M == -INFINITY ? 0.f : M;
    float L = 0.f, O0 = 0.f, O1 = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
      const float f = exp2f(sm_m[w * 16 + r] - Mu);
      const float2 o = *reinterpret_cast<const float2*>(sm_o + (w * 16 + r) * kOStride + col);
      L += sm_l[w * 16 + r] * f;
      O0 += o.x * f;
      O1 += o.y * f;
    }
    if (cs == 1) {
      *reinterpret_cast<__nv_bfloat162*>(outp + e) = __floats2bfloat162_rn(L > 0.f ? O0 / L : 0.f, L > 0.f ? O1 / L : 0.f);
      if (lsep && col == 0) lsep[r] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
    } else {
      const int owner = e / per;
      st_async_f32x2(rx_o + c * per + (e - owner * per), rx_bar, owner, O0, O1);
      if ((col >> 1) < cs) {                                  // the row's (M, L) goes to every rank: one thread per rank
        st_async_f32(rx_m + c * 16 + r, rx_bar, col >> 1, M);
        st_async_f32(rx_l + c * 16 + r, rx_bar, col >> 1, L);
      }
    }
  }
  if (cs > 1) {
    // Only the threads that merge wait, and only for the bytes addressed to this CTA.  Once they are all here nobody
    // writes into this CTA's shared memory any more, so it may finish without meeting the others again.
    const int e_beg = c * per, e_end = min(p.G * D, e_beg + per);
    if ((e_beg + tid < e_end || tid == 0) && !mbar_wait_cluster_bounded(rx_bar)) {   // thread 0 keeps the CTA alive for its senders in any case
      raise(p.dev_status, SG_ERR_TIMEOUT);
      return;
    }
    pdl_wait();                                                // out / lse are written below: all earlier work in the stream first
    for (int e = e_beg + tid; e < e_end; e += kDecThreads) {
      const int r = e / D, col = e - r * D;
      float mj[8], lj[8], oj[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const bool on = j < cs;
        mj[j] = on ? rx_m[j * 16 + r] : -INFINITY;
        lj[j] = on ? rx_l[j * 16 + r] : 0.f;
        oj[j] = on ? rx_o[j * per + (e - e_beg)] : 0.f;
      }
      float M = -INFINITY;
#pragma unroll
      for (int j = 0; j < 8; ++j) M = fmaxf(M, mj[j]);
      const float Mu = M == -INFINITY ? 0.f : M;
      float L = 0.f, O = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float f = exp2f(mj[j] - Mu);
        L += lj[j] * f;
        O += oj[j] * f;
      }
      outp[e] = __float2bfloat16_rn(L > 0.f ? O / L : 0.f);
      if (lsep && col == 0) lsep[r] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
    }
  }
}

template <int D, int kDecWarps, int kBuf>
constexpr int decode_smem_bytes() {
  return kDecWarps * kBuf * 2 * kSlice * D * 2 + kDecWarps * kBuf * 4 + (2 * 8 * 16 + 16 * D) * 4 + 16;   // rings, masks, receive area, its barrier
}

}  // namespace

// Launch shape, from what a sweep over batch sizes and list lengths measured.  CTAs beyond one wave
// of resident CTAs never paid, so a (sequence, KV head) pair is split over a cluster only while all
// clusters fit on the SMs at one CTA each.
//  * pairs <= SMs: warps = 8, one CTA per SM; csize = the cluster size (a power of two <= 8, the
//    portable limit) that gives each warp about one slice, capped by the SM count (12 warps per CTA
//    measured slower than 8: the merge grows faster than the streaming shrinks);
//  * more pairs: csize = 1 and warps = 4, two CTAs per SM, so that one CTA's prologue and merge overlap
//    the other's streaming -- except long lists whose CTA count fills waves of one CTA per SM better.
void decode_plan(const sg_shape* shape, int32_t total_sel, int32_t total_loc, int* csize, int* warps) {
  const int64_t pairs = (int64_t)shape->batch * shape->num_kv_heads;
  const int64_t avg_tokens = ((int64_t)total_sel + total_loc) / shape->batch;
  int W = 4, cs = 1;
  if (pairs <= kNumSMs) {
    // largest cluster whose CTAs are all resident at once; clusters of eight one-CTA-per-SM CTAs must also leave half
    // of the SMs to the next call, whose clusters cannot be placed otherwise while this call drains (2x slower)
    int fit = 1;
    while (fit < 8 && pairs * fit * 2 <= kNumSMs) fit *= 2;
    const int fit8 = (fit == 8 && pairs * 16 > kNumSMs) ? 4 : fit;
    // short lists: four warps per CTA already give every warp at most ~1.75 slices, and the merge is half as wide
    W = 4 * avg_tokens <= 7 * 4 * kSlice * fit ? 4 : 8;
    if (W == 8) fit = fit8;
    int work = 1;
    while (work < 8 && (int64_t)work * W * kSlice < avg_tokens) work *= 2;
    cs = fit < work ? fit : work;
    // many short lists: one 8-warp CTA per list has a slice or two per warp already, and no cluster to merge
    if (pairs >= 64 && avg_tokens <= 14 * kSlice) { W = 8; cs = 1; }
  } else {
    auto fill = [&](int64_t slots) { return (double)pairs / (double)(((pairs + slots - 1) / slots) * slots); };
    W = (avg_tokens >= 1024 && fill(kNumSMs) > fill(2 * kNumSMs) + 0.05) ? 8 : 4;
  }
  *csize = cs;
  *warps = W;
}

size_t decode_workspace_bytes(const sg_shape*, int32_t, int32_t) { return 0; }   // partials stay on chip

}  // namespace sg

namespace sg {
namespace {
// Testing hook (sg_testing_decode_overlap): 0 launches the decode kernel fully ordered behind earlier work.
std::atomic<int> g_test_decode_overlap{1};
sg_status decode_launch(const sg_shape* shape, const void* q, const void* packed_k, const void* packed_v, const int32_t* cu_k,
                        int32_t total_sel, const int32_t* packed_count, const int32_t* local_skip, const void* local_k,
                        const void* local_v, const int32_t* local_idx, const int32_t* cu_nloc, int32_t total_loc,
                        float softmax_scale, void* out, float* lse, void* workspace, size_t workspace_bytes,
                        int32_t* dev_status, void* stream);
}
}  // namespace sg

extern "C" void sg_testing_decode_overlap(int32_t allowed) {
  sg::g_test_decode_overlap.store(allowed, std::memory_order_relaxed);
}

extern "C" sg_status sg_sparse_decode_attn(const sg_shape* shape, const void* q, const void* packed_k,
                                           const void* packed_v, const int32_t* cu_k, int32_t total_sel,
                                           const void* local_k, const void* local_v, const int32_t* local_idx,
                                           const int32_t* cu_nloc, int32_t total_loc, float softmax_scale,
                                           void* out, float* lse, void* workspace, size_t workspace_bytes,
                                           int32_t* dev_status, void* stream) {
  return sg::decode_launch(shape, q, packed_k, packed_v, cu_k, total_sel, nullptr, nullptr, local_k, local_v, local_idx,
                           cu_nloc, total_loc, softmax_scale, out, lse, workspace, workspace_bytes, dev_status, stream);
}

extern "C" sg_status sg_sparse_decode_attn_counted(const sg_shape* shape, const void* q, const void* packed_k,
                                                   const void* packed_v, const int32_t* cu_cap, int32_t total_cap,
                                                   const int32_t* packed_count, const void* local_k, const void* local_v,
                                                   const int32_t* local_idx, const int32_t* cu_nloc, int32_t total_loc,
                                                   const int32_t* local_skip, float softmax_scale, void* out, float* lse,
                                                   int32_t* dev_status, void* stream) {
  if ((!packed_count && !local_skip) || !sg::aligned16(packed_count) || !sg::aligned16(local_skip)) return SG_ERR_INVALID;
  return sg::decode_launch(shape, q, packed_k, packed_v, cu_cap, total_cap, packed_count, local_skip, local_k, local_v,
                           local_idx, cu_nloc, total_loc, softmax_scale, out, lse, nullptr, 0, dev_status, stream);
}

namespace sg {
namespace {
sg_status decode_launch(const sg_shape* shape, const void* q, const void* packed_k, const void* packed_v, const int32_t* cu_k,
                        int32_t total_sel, const int32_t* packed_count, const int32_t* local_skip, const void* local_k,
                        const void* local_v, const int32_t* local_idx, const int32_t* cu_nloc, int32_t total_loc,
                        float softmax_scale, void* out, float* lse, void* workspace, size_t workspace_bytes,
                        int32_t* dev_status, void* stream) {
  using namespace sg;
  sg_status st = check_shape(shape, false);
  if (st != SG_OK) return st;
  if (shape->num_layers != 1 || total_sel < 0 || total_loc < 0) return SG_ERR_INVALID;
  if (!q || !out || !cu_k || !cu_nloc) return SG_ERR_INVALID;
  if (total_sel > 0 && (!packed_k || !packed_v)) return SG_ERR_INVALID;
  if (total_loc > 0 && (!local_k || !local_v || !local_idx)) return SG_ERR_INVALID;
  if (!aligned16(q) || !aligned16(out) || !aligned16(cu_k) || !aligned16(cu_nloc) || !aligned16(packed_k) ||
      !aligned16(packed_v) || !aligned16(local_k) || !aligned16(local_v) || !aligned16(local_idx) ||
      !aligned16(workspace) || (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)))
    return SG_ERR_INVALID;
  if (!(softmax_scale >= 0.f)) return SG_ERR_INVALID;
  (void)workspace_bytes;                                      // no workspace is needed: partials stay on chip
  const int D = shape->head_dim;
  const int G = shape->num_q_heads / shape->num_kv_heads;
  DecParams p;
  p.q = static_cast<const uint16_t*>(q);
  p.packed_k = static_cast<const uint16_t*>(packed_k ? packed_k : q);
  p.packed_v = static_cast<const uint16_t*>(packed_v ? packed_v : q);
  p.local_k = static_cast<const uint16_t*>(local_k ? local_k : q);
  p.local_v = static_cast<const uint16_t*>(local_v ? local_v : q);
  p.cu = shape->cu_seqlens;
  p.cu_k = cu_k;
  p.cu_nloc = cu_nloc;
  p.local_idx = local_idx ? local_idx : cu_nloc;
  p.packed_count = packed_count;
  p.local_skip = local_skip;
  p.out = static_cast<uint16_t*>(out);
  p.lse = lse;
  p.dev_status = dev_status;
  p.ts = shape->cache_token_stride;
  p.hs = shape->cache_head_stride;
  p.B = shape->batch;
  p.Hq = shape->num_q_heads;
  p.Hkv = shape->num_kv_heads;
  p.G = G;
  p.K_tot = total_sel;
  p.NL_tot = total_loc;
  p.n_tokens = shape->total_tokens;
  int warps = 4;
  decode_plan(shape, total_sel, total_loc, &p.csize, &warps);
  p.scale_log2 = (softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D)) * kLog2e;
  const int64_t grid_x = (int64_t)shape->batch * p.csize;
  if (grid_x > 0x7fffffffLL || shape->num_kv_heads > 65535) return SG_ERR_UNSUPPORTED;

  cudaLaunchAttribute attrs[2];
  attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attrs[0].val.programmaticStreamSerializationAllowed = g_test_decode_overlap.load(std::memory_order_relaxed) ? 1 : 0;
  attrs[1].id = cudaLaunchAttributeClusterDimension;
  attrs[1].val.clusterDim.x = (unsigned)p.csize;
  attrs[1].val.clusterDim.y = 1;
  attrs[1].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.stream = static_cast<cudaStream_t>(stream);
  cfg.attrs = attrs;
  cfg.numAttrs = p.csize > 1 ? 2 : 1;
  cfg.blockDim = dim3((unsigned)warps * 32);
  // one launch: sequences with empty lists still get out = 0 and lse = -inf
  cfg.gridDim = dim3((unsigned)grid_x, (unsigned)shape->num_kv_heads);
#define SG_LAUNCH_DECODE(DD, HI, WW, BB)                                                      \
  do {                                                                                        \
    SG_ENSURE_SMEM((decode_partial_kernel<DD, HI, WW, BB>), (decode_smem_bytes<DD, WW, BB>())); \
    cfg.dynamicSmemBytes = decode_smem_bytes<DD, WW, BB>();                                   \
    SG_CUDA_TRY(cudaLaunchKernelEx(&cfg, decode_partial_kernel<DD, HI, WW, BB>, p));          \
  } while (0)
#define SG_LAUNCH_DECODE_W(DD, HI)                         \
  do {                                                     \
    if (warps == 8) SG_LAUNCH_DECODE(DD, HI, 8, 3);        \
    else SG_LAUNCH_DECODE(DD, HI, 4, 3);                   \
  } while (0)
  if (D == 128) { if (G > 8) SG_LAUNCH_DECODE_W(128, true); else SG_LAUNCH_DECODE_W(128, false); }
  else          { if (G > 8) SG_LAUNCH_DECODE_W(64, true);  else SG_LAUNCH_DECODE_W(64, false); }
#undef SG_LAUNCH_DECODE_W
#undef SG_LAUNCH_DECODE
  return SG_OK;
}
}  // namespace
}  // namespace sg
