// sg_score: window-query x key-cache scoring with a fused softmax and row-reduce (sm_100a).
//
// For one (layer, sequence, KV head) the R = G*W window queries are scored against all N keys:
// a dense R x N x d contraction, so it runs on the 5th-generation tensor cores.  importance[t] =
// sum_r softmax_row_r(s)[t] needs every row's normaliser before any probability can be summed
// down a column, so the work is two passes over the keys:
//
//   pass 1 (row statistics)  D[row r][key t]  = Q_blk (A, 128 rows) x K_tile^T (B, 128 keys):
//          each epilogue thread owns one query row (one TMEM lane) and keeps a running
//          (max, sum-of-exp2) over the key columns -- no cross-thread reduction.
//   pass 2 (column sums)     D[key t][row r]  = K_tile (A, 128 keys) x Q_blk^T (B, <=128 rows):
//          each epilogue thread owns one key (one TMEM lane) and adds exp2(s*c - lse_r) over the
//          query-row columns; lse_r is a per-column constant read from shared memory.
//
// One persistent kernel runs both passes: one warp feeds Q and 128-key K tiles with TMA into 128-byte-swizzled
// shared memory, one thread issues tcgen05.mma into four 128-column TMEM accumulator stages (one per epilogue
// warpgroup), sixteen epilogue warps (four warpgroups, each owning every fourth block) drain them with tcgen05.ld.
// The score matrix never leaves the SM.  Work items (a pass, a layer/KV head, a chunk of key tiles of one sequence)
// are laid out so that pass 2 of a (layer, KV head) unit follows its pass 1 by a lag of a few units: close enough that
// the unit's keys are still in L2 for the second read (K crosses HBM once), far enough that the statistics pass 2
// needs are already published.  The epilogue warpgroups never meet at a CTA-wide barrier: each walks the items on its
// own and only waits for accumulators; two helper warps do everything else at item boundaries -- they merge and
// publish the row statistics of finished pass-1 items, bump a per-unit counter, wait (bounded) on that counter for
// the CTA's next pass-2 item and merge the chunks' statistics into its rows' log-sum-exps, one item ahead of the
// epilogue.  A pass-2 item only depends on items at smaller schedule positions and pass-1 items never wait, so the
// schedule cannot deadlock for any grid size.
//
// Every wait is bounded: on expiry the CTA raises SG_ERR_TIMEOUT in the status word, stops issuing work, waits
// (bounded) for its own TMA copies and MMAs, frees its TMEM and returns.
#include <cuda.h>

#include <vector>

#include "common.cuh"
#include "launch.h"

namespace sg {
namespace {

constexpr int kEpiGroups = 4;             // epilogue warpgroups (four warps each, one per TMEM lane quarter)
constexpr int kEpiThreads = 128 * kEpiGroups;
// Warp roles: warps 0-15 are the epilogue (four hardware-aligned warpgroups), warp 16 feeds TMA, warp 17 issues the MMAs and owns the TMEM allocation, warps 18 and 19 (the helpers)
// merge row statistics off the epilogue's path.
constexpr int kTmaWarp = kEpiThreads / 32;
constexpr int kMmaWarp = kTmaWarp + 1;
constexpr int kHelperWarp = kTmaWarp + 2;
constexpr int kScoreThreads = kEpiThreads + 128;
constexpr int kTileKeys = 128;
constexpr int kAccStages = 4;             // 4 x 128 fp32 columns = the whole 512-column TMEM
constexpr int kPartSlots = 8;             // pass 2, several row blocks per key tile: partial column sums of up to 8 tiles in flight
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxKStages = 4;
constexpr int kSmemLimit = 232448;        // 227 KB opt-in dynamic shared memory per CTA
constexpr float kLog2e = 1.4426950408889634f;

// Profiling build (-DSG_SCORE_PROFILE): selected threads add up the clocks they spend in each kind of wait and
// write the sums behind the CTA's four clock words of the testing clock buffer (32 words per CTA).
#ifdef SG_SCORE_PROFILE
#define SG_PROF_DECL(...) long long __VA_ARGS__
#define SG_PROF_BEGIN(t) const long long t = clock64()
#define SG_PROF_ADD(acc, t) acc += clock64() - (t)
#define SG_PROF_INC(acc) acc += 1
#define SG_PROF_STORE(slot, v) do { if (p.clock_out) p.clock_out[32 * (size_t)blockIdx.x + (slot)] = (unsigned long long)(v); } while (0)
constexpr int kClockWords = 32;
#else
#define SG_PROF_DECL(...)
#define SG_PROF_BEGIN(t)
#define SG_PROF_ADD(acc, t)
#define SG_PROF_INC(acc)
#define SG_PROF_STORE(slot, v)
constexpr int kClockWords = 4;
#endif

// Debug build (-DSG_CHECKS): device-side checks of the shared-memory carve-up, of every TMA coordinate (16-byte
// aligned innermost coordinate, tile inside the tensor or hanging over its end only where the fill value is
// wanted) and of every TMEM address against the allocation.  A failed check never traps: it sets the
// SG_ERR_INVALID bit of the status word and the access is still made only if it is known to be harmless (TMA
// loads past the end are zero-filled by the hardware), so a debug run ends like any other and reports the bit.
#ifdef SG_CHECKS
#define SG_CHECK(cond) do { if (!(cond)) raise(p.dev_status, SG_ERR_INVALID); } while (0)
#else
#define SG_CHECK(cond) do { } while (0)
#endif

struct ScoreParams {
  const int32_t* cu;
  float* importance;
  int* p1_done;            // [U] per unit: two counts per published pass-1 item, one per helper warp (zeroed by the host call)
  float2* part;            // [U][max_items][Ralloc] per-item row statistics (log2-domain max, sum of exp2)
  int32_t* dev_status;
  int64_t T;
  int32_t B, Hkv, G, W, R, Rpad, Ralloc;
  int32_t U;               // units = layers x KV heads
  int32_t lag;             // pass 2 of unit u is scheduled `lag` units after its pass 1
  int32_t compact;         // schedule layout: 0 = every slot 2*C positions, 1 = positions without an item removed
  int32_t tiles_per_chunk, max_items, k_stages, q_bufs;
  int32_t smem_bytes;      // dynamic shared memory of the launch (debug checks)
  int32_t wgslots;         // statistics slots per item: 4 (one per epilogue warpgroup) or 1 (every row block has one owner)
  int32_t withhold_unit;   // testing only: pass-1 items of this unit are never counted as done (-1 = none)
  uint32_t wait_ns;        // limit of every bounded wait, nanoseconds
  unsigned long long* clock_out;   // testing only: per CTA {clock64 start, end, globaltimer start, end}, or null
  float scale_log2;
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// One try_wait: true when the phase has completed.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: gives up after `limit_ns` (about one second in normal use), or once another thread has set
// *abort_flag.  try_wait comes back after a short, hardware-chosen time whether or not the phase has completed, so a
// thread that simply retries spins through a dozen instructions per attempt -- issue slots and, worse, entries of the
// queue that the SFU instructions of the working warps go through (measured: one retry per 11 clocks and SM, 60 % of
// all executed instructions, SFU pipe at 51 %).  A waiter therefore sleeps `sleep_ns` between attempts (chosen per
// role: short on the MMA thread's critical path, long for the producer that runs ahead) and looks at the clock and the
// abort flag only every 64th attempt.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t limit_ns,
                                          uint32_t sleep_ns) {
  if (mbar_test(bar, parity)) return true;
  uint64_t t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (sleep_ns) __nanosleep(sleep_ns);
    if (mbar_test(bar, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > (uint64_t)limit_ns) { *abort_flag = 1; return false; }
    }
  }
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] = A[smem] * B[smem], bf16 x bf16 -> fp32, issued by one thread; the operands are shared-memory matrix
// descriptors given as their low words (address field), the high word is the same for every operand.
// All MMAs of one accumulator block in a single statement: NK k-steps of 16 elements, four per 128-byte
// sub-tile (descriptor low word += 2 per step inside a sub-tile, += a_sub / b_sub to the next sub-tile).  The first
// MMA overwrites the accumulator, the others add to it.  One statement keeps the issuing thread's instruction
// stream to the bare minimum between two blocks: the tensor pipe drains its short queue within ~200 clocks of the
// last issue, so every clock spent between blocks is an idle clock of the pipe.
template <int NK>
__device__ __forceinline__ void umma_block(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t a_sub, uint32_t b_sub,
                                           uint32_t desc_hi, uint32_t idesc) {
  static_assert(NK == 4 || NK == 8, "one or two 64-element sub-tiles along d");
  if (NK == 8) {
    asm volatile(
        "{\n\t.reg .b64 da, db;\n\t.reg .b32 a, b;\n\t.reg .pred pf, pt;\n\t"
        "setp.ne.u32 pf, %0, %0;\n\tsetp.eq.u32 pt, %0, %0;\n\t"
        "mov.b64 da, {%1, %5};\n\tmov.b64 db, {%2, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, pf;\n\t"
        "add.u32 a, %1, 2;\n\tadd.u32 b, %2, 2;\n\tmov.b64 da, {a, %5};\n\tmov.b64 db, {b, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, pt;\n\t"
        "add.u32 a, %1, 4;\n\tadd.u32 b, %2, 4;\n\tmov.b64 da, {a, %5};\n\tmov.b64 db, {b, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, pt;\n\t"
        "add.u32 a, %1, 6;\n\tadd.u32 b, %2, 6;\n\tmov.b64 da, {a, %5};\n\tmov.b64 db, {b, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, pt;\n\t"
        "add.u32 a, %1, %3;\n\tadd.u32 b, %2, %4;\n\tmov.b64 da, {a, %5};\n\tmov.b64 db, {b, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, pt;\n\t"
        "add.u32 a, a, 2;\n\tadd.u32 b, b, 2;\n\tmov.b64 da, {a, %5};\n\tmov.b64 db, {b, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, pt;\n\t"
        "add.u32 a, a, 2;\n\tadd.u32 b, b, 2;\n\tmov.b64 da, {a, %5};\n\tmov.b64 db, {b, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, pt;\n\t"
        "add.u32 a, a, 2;\n\tadd.u32 b, b, 2;\n\tmov.b64 da, {a, %5};\n\tmov.b64 db, {b, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, pt;\n\t}"
        ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(a_sub), "r"(b_sub), "r"(desc_hi), "r"(idesc) : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .b64 da, db;\n\t.reg .b32 a, b;\n\t.reg .pred pf, pt;\n\t"
        "setp.ne.u32 pf, %0, %0;\n\tsetp.eq.u32 pt, %0, %0;\n\t"
        "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pf;\n\t"
        "add.u32 a, %1, 2;\n\tadd.u32 b, %2, 2;\n\tmov.b64 da, {a, %3};\n\tmov.b64 db, {b, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
        "add.u32 a, %1, 4;\n\tadd.u32 b, %2, 4;\n\tmov.b64 da, {a, %3};\n\tmov.b64 db, {b, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
        "add.u32 a, %1, 6;\n\tadd.u32 b, %2, 6;\n\tmov.b64 da, {a, %3};\n\tmov.b64 db, {b, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t}"
        ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc) : "memory");
  }
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// TMEM load of 32 consecutive fp32 columns of this thread's lane, issued without waiting: the registers hold
// the data only after tmem_ld_wait().  A warp issues the load of its next 32 columns before it works on the
// current ones, so the load's latency is covered by arithmetic.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t (&r)[32], uint32_t taddr) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
// Waits for the thread's outstanding TMEM loads.  The empty statements that follow tie the 32 registers of the
// load that has just completed to this point of the program: volatile statements keep their order, and every
// later use of the registers depends on them, so the compiler cannot schedule arithmetic on the data ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; i += 8)
    asm volatile("" : "+r"(r[i]), "+r"(r[i + 1]), "+r"(r[i + 2]), "+r"(r[i + 3]), "+r"(r[i + 4]), "+r"(r[i + 5]),
                      "+r"(r[i + 6]), "+r"(r[i + 7]) :: "memory");
}

// Shared-memory matrix descriptor of a K-major bf16 tile stored as rows of 128 bytes with the
// 128-byte swizzle (what TMA writes with CU_TENSOR_MAP_SWIZZLE_128B).  High word: 8-row groups are 1024
// bytes apart (stride byte offset, bits [32,46)), descriptor version 1 for sm_100 (bit 46), layout type
// SWIZZLE_128B = 2 (bits [61,64)); the leading byte offset is unused for this layout.  Low word: the start
// address in 16-byte units (bits [0,14)); advancing 16 elements along K inside the 128-byte span adds 2.
constexpr uint32_t kSmemDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t addr) { return (addr & 0x3FFFFu) >> 4; }
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__device__ __forceinline__ uint32_t make_idesc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Position in the persistent schedule -> work item.  The schedule is a sequence of slots; slot s holds the
// pass-2 items of unit (s - lag) followed by the pass-1 items of unit s, a unit being one (layer, KV head)
// with all its sequences (C items per pass).  CTA k walks positions k, k + grid, k + 2*grid, ...  A pass-2
// item depends only on pass-1 items at smaller positions, and pass-1 items never wait, so the item at the
// smallest unfinished position can always run: the schedule cannot deadlock whatever the grid size.
// With few units (lag >= U) the schedule is simply all pass-1 items followed by all pass-2 items.
struct SchedPos { int pass, unit, j; };    // pass 0 = no item at this position
__host__ __device__ __forceinline__ long long schedule_length(int U, int C, int lag, bool compact) {
  return (lag >= U || compact) ? (long long)U * 2 * C : (long long)(U + lag) * 2 * C;
}
// Three layouts.  lag >= U (few units): all pass-1 items, then all pass-2 items.  Padded: every slot has
// 2*C positions, those of units that do not exist are empty (the first and the last `lag` slots are half
// empty).  Compact: the same order with the empty positions removed.  Which of the last two finishes first
// depends on how the items fall on the CTAs; the host simulates both and picks (see choose_layout).
__host__ __device__ __forceinline__ SchedPos schedule_position(long long pos, int U, int C, int lag, bool compact) {
  SchedPos sp;
  if (lag >= U) {
    const long long half = (long long)U * C;
    const long long q = pos < half ? pos : pos - half;
    sp.unit = (int)(q / C); sp.j = (int)(q - (long long)sp.unit * C); sp.pass = pos < half ? 1 : 2;
    return sp;
  }
  if (compact) {
    const long long head = (long long)lag * C, mid = (long long)(U - lag) * 2 * C;
    if (pos < head) {
      sp.unit = (int)(pos / C); sp.j = (int)(pos - (long long)sp.unit * C); sp.pass = 1;
      return sp;
    }
    if (pos >= head + mid) {
      const long long q = pos - head - mid;
      const int k = (int)(q / C);
      sp.unit = U - lag + k; sp.j = (int)(q - (long long)k * C); sp.pass = 2;
      return sp;
    }
    pos += head;                                   // inside the middle part both layouts agree up to this shift
  }
  const int slot = (int)(pos / (2 * C));
  const int r = (int)(pos - (long long)slot * (2 * C));
  if (r < C) { sp.unit = slot - lag; sp.j = r; sp.pass = 2; } else { sp.unit = slot; sp.j = r - C; sp.pass = 1; }
  if (sp.unit < 0 || sp.unit >= U) sp.pass = 0;
  return sp;
}

struct ScoreItem {
  int pass;          // 1 or 2; 0 = no item at this position
  int unit, l, g, b;
  int c0, N;         // first token and length of sequence b
  int tile_beg, tile_end;
  int item_in_unit;  // this item's index among the unit's C items (its partial-statistics slot)
  int first_item_b;  // index of sequence b's first item in the unit
  int nch_b;         // number of items (chunks) of sequence b
};

// s_cu[b] = cu_seqlens[b]; s_prefix[b] = number of items of the sequences before b (s_prefix[B] = C).
__device__ __forceinline__ ScoreItem decode_position(const ScoreParams& p, long long pos, const int* s_cu, const int* s_prefix) {
  ScoreItem it;
  it.pass = 0;
  const int C = s_prefix[p.B];
  const SchedPos sp = schedule_position(pos, p.U, C, p.lag, p.compact != 0);
  it.pass = sp.pass;
  const int unit = sp.unit, j = sp.j;
  if (it.pass == 0) return it;
  it.unit = unit;
  it.l = unit / p.Hkv;
  it.g = unit - it.l * p.Hkv;
  it.item_in_unit = j;
  int lo = 0, hi = p.B;                                  // largest b with s_prefix[b] <= j
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (s_prefix[mid] <= j) lo = mid; else hi = mid;
  }
  it.b = lo;
  it.first_item_b = s_prefix[lo];
  it.nch_b = s_prefix[lo + 1] - it.first_item_b;
  it.c0 = s_cu[lo];
  it.N = s_cu[lo + 1] - it.c0;
  const int tiles_total = (it.N + kTileKeys - 1) / kTileKeys;
  it.tile_beg = (j - it.first_item_b) * p.tiles_per_chunk;
  it.tile_end = min(tiles_total, it.tile_beg + p.tiles_per_chunk);
  return it;
}

__device__ __forceinline__ int ld_acquire_gpu(const int* ptr) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
  return v;
}
// Rare path of pass 1: the sum of a 32-column chunk against the running reference m left the safe range (a value far
// above m, or m still -inf at the start of a work item).  Takes the chunk's maximum, rescales the running sum and adds
// the chunk against the new reference.  Kept out of line so that the hot loop holds nothing but its 32 x (fma, ex2, add).
// (Everything is passed and returned by value: taking the address of the chunk's registers or of the running statistics
// would move them to local memory in the hot loop as well.)
__device__ __noinline__ float2 refresh_reference(float scale_log2, float m, float lsum, uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t c4, uint32_t c5, uint32_t c6, uint32_t c7, uint32_t c8, uint32_t c9, uint32_t c10, uint32_t c11, uint32_t c12, uint32_t c13, uint32_t c14, uint32_t c15, uint32_t c16, uint32_t c17, uint32_t c18, uint32_t c19, uint32_t c20, uint32_t c21, uint32_t c22, uint32_t c23, uint32_t c24, uint32_t c25, uint32_t c26, uint32_t c27, uint32_t c28, uint32_t c29, uint32_t c30, uint32_t c31) {
  const uint32_t cur[32] = {c0, c1, c2, c3, c4, c5, c6, c7, c8, c9, c10, c11, c12, c13, c14, c15, c16, c17, c18, c19, c20, c21, c22, c23, c24, c25, c26, c27, c28, c29, c30, c31};
  float mx = __uint_as_float(cur[0]);
#pragma unroll
  for (int c = 1; c < 32; ++c) mx = fmaxf(mx, __uint_as_float(cur[c]));
  const float mn = fmaxf(m, mx * scale_log2);
  float r0 = 0.f, r1 = 0.f;
#pragma unroll
  for (int c = 0; c < 32; c += 2) {
    r0 += exp2f(fmaf(__uint_as_float(cur[c]), scale_log2, -mn));
    r1 += exp2f(fmaf(__uint_as_float(cur[c + 1]), scale_log2, -mn));
  }
  return make_float2(mn, lsum * exp2f(m - mn) + (r0 + r1));
}

template <int D>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k, const ScoreParams p) {
  constexpr int kSub = D / 64;                        // 64-element (128-byte) sub-tiles along d
  constexpr int kKSubBytes = kTileKeys * 128;         // one sub-tile of a K stage
  constexpr int kKStageBytes = kSub * kKSubBytes;
  extern __shared__ uint8_t smem_dyn[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  const int q_sub_bytes = p.Ralloc * 128;
  const int q_buf_bytes = kSub * q_sub_bytes;
  uint8_t* q_smem = smem;                                            // [q_bufs] Q operands
  uint8_t* k_smem = q_smem + p.q_bufs * q_buf_bytes;                  // [k_stages] K tiles
  uint8_t* tail = k_smem + p.k_stages * kKStageBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tail);                 // 29 barriers (29 slots; the words behind them follow)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 29 * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 29 * 8 + 4);
  float* lse_buf = reinterpret_cast<float*>(tail + 240);              // [2][Ralloc] row log-sum-exps of two pass-2 items
  float* sm_stat = lse_buf + 2 * p.Ralloc;                            // pass 1: [2 buffers]{m[wgslots][Ralloc], l[wgslots][Ralloc]}
  float* sm_part = sm_stat + 4 * p.wgslots * p.Ralloc;                // pass 2, several blocks per tile: [slots][groups][128] partial column sums
  const int part_slots = p.Rpad > 384 ? 4 : (p.Rpad > 128 ? 8 : 0);   // tiles in flight (see the pass-2 combine)
  int* sm_cnt = reinterpret_cast<int*>(sm_part + part_slots * kEpiGroups * 128);   // [kPartSlots][4 lane quarters] partials written
  int* s_cu = sm_cnt + kPartSlots * 4 + 8;                            // [B+1] (eight spare words before it)                                            // [B+1]
  int* s_prefix = s_cu + p.B + 1;                                     // [B+1]

  auto bar_qfull = [&](int s) { return smem_u32(&bars[s]); };
  auto bar_qempty = [&](int s) { return smem_u32(&bars[2 + s]); };
  auto bar_kfull = [&](int s) { return smem_u32(&bars[4 + s]); };
  auto bar_kempty = [&](int s) { return smem_u32(&bars[8 + s]); };
  auto bar_afull = [&](int s) { return smem_u32(&bars[12 + s]); };
  auto bar_aempty = [&](int s) { return smem_u32(&bars[16 + s]); };
  auto bar_lse_ready = [&](int s) { return smem_u32(&bars[20 + s]); };   // helper -> epilogue: lse_buf[s] holds the item's rows
  auto bar_lse_free = [&](int s) { return smem_u32(&bars[22 + s]); };    // epilogue (16 warps) -> helper: lse_buf[s] may be rewritten
  const uint32_t bar_drain = smem_u32(&bars[24]);
  auto bar_stat_full = [&](int s) { return smem_u32(&bars[25 + s]); };   // epilogue (16 warps) -> helpers: the item's statistics are complete
  auto bar_stat_free = [&](int s) { return smem_u32(&bars[27 + s]); };   // helpers -> epilogue: the statistics buffer was published                        // MMA thread: every MMA it issued has completed

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    SG_CHECK(reinterpret_cast<uint8_t*>(s_prefix + p.B + 1) <= smem_dyn + p.smem_bytes);     // carve-up fits the launch's shared memory
    SG_CHECK((smem_u32(q_smem) & 1023u) == 0 && (smem_u32(k_smem) & 1023u) == 0);            // swizzled operands on 1024-byte boundaries
    SG_CHECK((smem_u32(bars) & 7u) == 0 && (smem_u32(lse_buf) & 15u) == 0);
  }

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar_qfull(s), 1); mbar_init(bar_qempty(s), 1);
    }
    for (int s = 0; s < kMaxKStages; ++s) { mbar_init(bar_kfull(s), 1); mbar_init(bar_kempty(s), 1); }
    for (int s = 0; s < kAccStages; ++s) { mbar_init(bar_afull(s), 1); mbar_init(bar_aempty(s), 4); }
    for (int s = 0; s < 2; ++s) { mbar_init(bar_lse_ready(s), 2); mbar_init(bar_lse_free(s), kEpiThreads / 32); }
    mbar_init(bar_drain, 1);
    for (int s = 0; s < 2; ++s) { mbar_init(bar_stat_full(s), kEpiThreads / 32); mbar_init(bar_stat_free(s), 2); }
    *abort_flag = 0;
    for (int i = 0; i < kPartSlots * 4; ++i) sm_cnt[i] = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == kMmaWarp) {
    tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  if (warp == 0) {
    // sequence offsets and the per-sequence item prefix, once per CTA
    int acc = 0;
    for (int b0 = 0; b0 <= p.B; b0 += 32) {
      const int b = b0 + lane;
      int nch = 0;
      if (b <= p.B) s_cu[b] = p.cu[b];
      if (b < p.B) {
        const int tiles = (p.cu[b + 1] - p.cu[b] + kTileKeys - 1) / kTileKeys;
        nch = (tiles + p.tiles_per_chunk - 1) / p.tiles_per_chunk;
      }
      int inc = nch;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += v;
      }
      if (b < p.B) s_prefix[b + 1] = acc + inc;
      acc += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (lane == 0) s_prefix[0] = 0;
  }
  if (p.R < p.Ralloc) {
    // Rows R..Ralloc-1 of the Q operands are never written by TMA: zero them once so that padded MMA
    // rows/columns are finite.  (The 128-byte swizzle only permutes 16-byte chunks inside a row's own 128 bytes.)
    const int words = (p.Ralloc - p.R) * 32;
    for (int qb = 0; qb < p.q_bufs; ++qb)
      for (int dc = 0; dc < kSub; ++dc) {
        uint32_t* z = reinterpret_cast<uint32_t*>(q_smem + qb * q_buf_bytes + dc * q_sub_bytes + p.R * 128);
        for (int i = tid; i < words; i += kScoreThreads) z[i] = 0u;
      }
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int C = s_prefix[p.B];
  const long long npos = schedule_length(p.U, C, p.lag, p.compact != 0);
  volatile int never = 0;

  unsigned long long clk0 = 0, gt0 = 0;
  if (p.clock_out && tid == 0) { clk0 = (unsigned long long)clock64(); gt0 = global_timer_ns(); }

  if (warp == kTmaWarp) {
    // ------------------------------------------------------------ TMA producer (one thread)
    if (lane == 0) {
      int stage = 0, n_item = 0;
      uint32_t phase = 0;
      long long n_loads = 0;                          // K tiles requested so far
      bool ok = true;
      SG_PROF_DECL(w_kempty = 0, w_qempty = 0);
      for (long long pos = blockIdx.x; pos < npos && ok; pos += gridDim.x) {
        const ScoreItem it = decode_position(p, pos, s_cu, s_prefix);
        if (it.pass == 0) continue;
        const int qb = n_item % p.q_bufs;
        const uint32_t qph = (uint32_t)((n_item / p.q_bufs) & 1);
        SG_PROF_BEGIN(tq);
        ok = mbar_wait(bar_qempty(qb), qph ^ 1u, abort_flag, p.wait_ns, 200u);
        SG_PROF_ADD(w_qempty, tq);
        if (!ok) break;
        ++n_item;
        SG_CHECK(qb >= 0 && qb < p.q_bufs && (it.g + 1) * p.G <= p.Hkv * p.G && it.b < p.B && p.G * p.W <= p.Ralloc);
        mbar_arrive_expect_tx(bar_qfull(qb), (uint32_t)(kSub * p.G * p.W * 128));
#pragma unroll
        for (int dc = 0; dc < kSub; ++dc)
          tma_load_4d(smem_u32(q_smem + qb * q_buf_bytes + dc * q_sub_bytes), &tmap_q, bar_qfull(qb), dc * 64, it.g * p.G, 0,
                      it.l * p.B + it.b);
        for (int tile = it.tile_beg; tile < it.tile_end && ok; ++tile) {
          SG_PROF_BEGIN(tk);
          ok = mbar_wait(bar_kempty(stage), phase ^ 1u, abort_flag, p.wait_ns, 200u);
          SG_PROF_ADD(w_kempty, tk);
          if (!ok) break;
          SG_CHECK(stage >= 0 && stage < p.k_stages && it.c0 + tile * kTileKeys < p.T && it.g < p.Hkv && it.l * p.Hkv < p.U);
          mbar_arrive_expect_tx(bar_kfull(stage), (uint32_t)kKStageBytes);
#pragma unroll
          for (int dc = 0; dc < kSub; ++dc)
            tma_load_4d(smem_u32(k_smem + stage * kKStageBytes + dc * kKSubBytes), &tmap_k, bar_kfull(stage), dc * 64, it.g,
                        it.c0 + tile * kTileKeys, it.l);
          ++n_loads;
          if (++stage == p.k_stages) { stage = 0; phase ^= 1u; }
        }
      }
      SG_PROF_STORE(4, w_kempty); SG_PROF_STORE(5, w_qempty);
      if (ok) {
        // Wait until the MMAs have released every K stage and Q buffer: no barrier arrival and no copy of this
        // CTA is pending when it exits.
        for (int i = 0; i < p.k_stages; ++i) {
          if (!mbar_wait(bar_kempty(stage), phase ^ 1u, abort_flag, p.wait_ns, 200u)) break;
          if (++stage == p.k_stages) { stage = 0; phase ^= 1u; }
        }
        for (int i = 0; i < p.q_bufs; ++i) {
          const int n = n_item + i;
          if (!mbar_wait(bar_qempty(n % p.q_bufs), (uint32_t)(((n / p.q_bufs) & 1) ^ 1), abort_flag, p.wait_ns, 200u)) break;
        }
      } else {
        // Aborted: nobody may consume what was requested, so wait (bounded, ignoring the abort flag) for the copies
        // themselves -- the `full` barrier of every K stage and Q buffer that still has a request outstanding --
        // before this CTA's shared memory is given up.
        const int back = (int)(n_loads < p.k_stages ? n_loads : p.k_stages);
        for (int i = 1; i <= back; ++i) {
          const long long n = n_loads - i;             // the i-th last request: stage n % k_stages, use n / k_stages
          if (!mbar_wait(bar_kfull((int)(n % p.k_stages)), (uint32_t)((n / p.k_stages) & 1), &never, p.wait_ns, 200u)) break;
        }
        const int qback = n_item < p.q_bufs ? n_item : p.q_bufs;
        for (int i = 1; i <= qback; ++i) {
          const int n = n_item - i;
          if (!mbar_wait(bar_qfull(n % p.q_bufs), (uint32_t)((n / p.q_bufs) & 1), &never, p.wait_ns, 200u)) break;
        }
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------ MMA issuer (one thread)
    // Accumulator stage w feeds epilogue warpgroup w; block n of the CTA's running count goes to stage n mod 4.
    // Each stage is consumed by one warpgroup only, so no waiter ever falls more than one mbarrier phase behind.
    if (lane == 0) {
      int ks = 0, n_item = 0;
      uint32_t kph = 0, phbits = 0, tile_count = 0;   // phbits: one phase bit per accumulator stage
      bool ok = true;
      SG_PROF_DECL(w_qfull = 0, w_kfull = 0, w_aempty = 0);
      const uint32_t k_lo0 = smem_desc_lo(smem_u32(k_smem));
      const uint32_t k_stage_lo = (uint32_t)kKStageBytes >> 4;
      const uint32_t bar_afull0 = bar_afull(0), bar_aempty0 = bar_aempty(0);
      for (long long pos = blockIdx.x; pos < npos && ok; pos += gridDim.x) {
        const ScoreItem it = decode_position(p, pos, s_cu, s_prefix);
        if (it.pass == 0) continue;
        const int qb = n_item % p.q_bufs;
        const uint32_t qph = (uint32_t)((n_item / p.q_bufs) & 1);
        ++n_item;
        SG_PROF_BEGIN(tq);
        ok = mbar_wait(bar_qfull(qb), qph, abort_flag, p.wait_ns, 0u);
        SG_PROF_ADD(w_qfull, tq);
        if (!ok) break;
        tc_fence_after();
        // per-item constants of the issue loop
        const bool pass1 = it.pass == 1;
        const int nblk = pass1 ? (p.R + 127) / 128 : (p.Rpad + 127) / 128;
        const uint32_t q_lo0 = smem_desc_lo(smem_u32(q_smem + qb * q_buf_bytes));
        const uint32_t q_blk_lo = (128u * 128u) >> 4;                      // next row block of the Q operand
        const uint32_t a_sub = (uint32_t)(pass1 ? q_sub_bytes : kKSubBytes) >> 4;
        const uint32_t b_sub = (uint32_t)(pass1 ? kKSubBytes : q_sub_bytes) >> 4;
        const uint32_t idesc_full = make_idesc(128, 128);
        const uint32_t idesc_last = pass1 ? idesc_full : make_idesc(128, p.Rpad - (nblk - 1) * 128);
        for (int tile = it.tile_beg; tile < it.tile_end && ok; ++tile) {
          SG_PROF_BEGIN(tk);
          if (!mbar_test(bar_kfull(ks), kph)) ok = mbar_wait(bar_kfull(ks), kph, abort_flag, p.wait_ns, 0u);
          SG_PROF_ADD(w_kfull, tk);
          if (!ok) break;
          tc_fence_after();
          const uint32_t k_lo = k_lo0 + (uint32_t)ks * k_stage_lo;
          uint32_t q_lo = q_lo0;
          for (int blk = 0; blk < nblk; ++blk, q_lo += q_blk_lo) {
            const uint32_t as = (tile_count++) % kEpiGroups;               // blocks go to the warpgroups in rotation
            const uint32_t par = ((phbits >> as) & 1u) ^ 1u;
            SG_PROF_BEGIN(ta);
            ok = mbar_wait(bar_aempty0 + as * 8u, par, abort_flag, p.wait_ns, 0u);
            SG_PROF_ADD(w_aempty, ta);
            if (!ok) break;
            tc_fence_after();
            umma_block<4 * kSub>(tmem_base + as * 128u, pass1 ? q_lo : k_lo, pass1 ? k_lo : q_lo, a_sub, b_sub, kSmemDescHi,
                                 blk == nblk - 1 ? idesc_last : idesc_full);
            umma_commit(bar_afull0 + as * 8u);
            phbits ^= 1u << as;
          }
          if (ok) umma_commit(bar_kempty(ks));
          if (++ks == p.k_stages) { ks = 0; kph ^= 1u; }
        }
        if (ok) umma_commit(bar_qempty(qb));
      }
      // Every MMA this thread issued has completed before the CTA frees its tensor memory, also on an aborted run
      // (the commit arrives when all earlier MMAs are done; the wait ignores the abort flag and is bounded).
      SG_PROF_STORE(6, w_qfull); SG_PROF_STORE(7, w_kfull); SG_PROF_STORE(8, w_aempty);
      umma_commit(bar_drain);
      mbar_wait(bar_drain, 0u, &never, p.wait_ns, 0u);
    }
  } else if (warp < kTmaWarp) {
    // ------------------------------------------------------------ epilogue warps
    // Four warpgroups of four warps; each owns one accumulator stage and every fourth block (a key tile, or one
    // row block of a key tile) of the CTA's running block count.  A thread sees all 128 accumulator columns of
    // its TMEM lane.  The warpgroups never meet at a CTA-wide barrier: each walks the CTA's items on its own,
    // publishes its own pass-1 statistics and waits only for accumulators and (pass 2) for the helper warp's
    // log-sum-exps, so the others keep the SFU busy while one of them is between items.
    const int wg = warp >> 2;
    const int wg_tid = tid & 127;
    (void)wg_tid;                                      // only the profiling build reads it
    const int lane_grp = warp & 3;                     // TMEM lane quarter this warp may access
    const int row_in_tile = lane_grp * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)(lane_grp * 32) << 16);
    const int as = wg;                                 // this warpgroup's accumulator stage
    const uint32_t t_acc = t_lane + (uint32_t)(as * 128);
    const int wgslot = p.wgslots == 4 ? wg : 0;
    uint32_t aph = 0, tile_count = 0;
    int n_p2 = 0;                                      // pass-2 items seen so far (selects the lse buffer)
    int n_p1 = 0;                                      // pass-1 items seen so far (selects the statistics buffer)
    bool ok = true;
    SG_PROF_DECL(w_afull = 0, w_lse = 0, w_pub = 0, n_blocks = 0, w_sfree = 0);
    // Releases the accumulator: called right after the block's last TMEM load has completed, before the
    // arithmetic on those columns, so the MMAs of this warpgroup's next block overlap it.
    auto release_acc = [&]() {
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_aempty(as));
      aph ^= 1u;
    };
    for (long long pos = blockIdx.x; pos < npos; pos += gridDim.x) {   // no early exit: every thread meets its warpgroup's barriers
      const ScoreItem it = decode_position(p, pos, s_cu, s_prefix);
      if (it.pass == 0) continue;
      const int N = it.N;
      const int Weff = min(p.W, N);
      const int first_win = N - Weff;                  // position of window row 0; keys <= it are visible to all rows

      if (it.pass == 1) {
        const int nblk = (p.R + 127) / 128;
        const bool blockwise = nblk > 1;
        const uint32_t n_item0 = tile_count;           // running block count at the start of the item
        // Running statistics live in one of two shared-memory buffers (alternating pass-1 items, because the
        // warpgroups drift apart by up to an item).  The buffer's previous item must have been merged and published
        // by the helper warps (practically always true already; the wait is bounded).
        const int sbuf = n_p1 & 1, suse = n_p1 >> 1;
        ++n_p1;
        SG_PROF_BEGIN(tsf);
        if (ok && suse > 0) ok = mbar_wait(bar_stat_free(sbuf), (uint32_t)((suse - 1) & 1), abort_flag, p.wait_ns, 32u);
        SG_PROF_ADD(w_sfree, tsf);
        float* sm_m = sm_stat + (size_t)(sbuf * 2 * p.wgslots + wgslot) * p.Ralloc;   // this warpgroup's slot: max ...
        float* sm_l = sm_m + p.wgslots * p.Ralloc;                                     // ... and sum of exp2
        // Slot (wgslot, blk*128 + row_in_tile) is only ever touched by this thread during the item, so the running
        // statistics need no barrier: with one slot per warpgroup every block's rows are initialised, with a shared
        // slot (the number of row blocks is a multiple of four, so a row block always meets the same warpgroup)
        // only the owned ones.
        for (int blk = 0; blk < nblk; ++blk)
          if (p.wgslots == 4 || ((n_item0 + (uint32_t)blk) % kEpiGroups) == (uint32_t)wg) {
            sm_m[blk * 128 + row_in_tile] = -INFINITY;
            sm_l[blk * 128 + row_in_tile] = 0.f;
          }
        // The item's tiles in two loops.  First the tiles that every window row sees completely, when all rows of this
        // warp lie inside the window: the loop holds the hot body and nothing else -- with the masked variant compiled
        // into the same loop the kernel, which runs at its 96-register limit, was 7-10 % slower as a whole.  Then the
        // rest (the causal diagonal, or everything when some row of the warp is outside the window) in the general loop.
        bool rows_ok = true;
        for (int blk = 0; blk < nblk; ++blk) {
          const int r = blk * 128 + row_in_tile;
          rows_ok = rows_ok && r < p.R && (r / p.G) < Weff;
        }
        rows_ok = __all_sync(0xffffffffu, rows_ok);
        const int vis_end = (first_win + 1) / kTileKeys;                    // tiles [0, vis_end) are visible to every window row
        const int hot_end = rows_ok ? min(it.tile_end, max(it.tile_beg, vis_end)) : it.tile_beg;
        for (int tile = it.tile_beg; tile < hot_end; ++tile) {
          if (!blockwise && ((tile_count++) % kEpiGroups) != (uint32_t)wg) continue;   // (the wait below looks at `ok`)
          for (int blk = 0; blk < nblk; ++blk) {
            if (blockwise && (((tile_count++) % kEpiGroups) != (uint32_t)wg || !ok)) continue;
            SG_PROF_BEGIN(ta);
            if (ok) ok = mbar_wait(bar_afull(as), aph, abort_flag, p.wait_ns, 0u);
            SG_PROF_ADD(w_afull, ta);
            SG_PROF_INC(n_blocks);
            if (!ok) continue;
            tc_fence_after();
            const int r = blk * 128 + row_in_tile;
            float m = sm_m[r], lsum = sm_l[r];
            uint32_t cur[32];
            // The running reference m need not be the row maximum: fp32 keeps its relative precision for any exponent, so
            // the sum of exp2(x - m) is as accurate with a stale (lower) m as with the true maximum, as long as nothing
            // overflows.  A chunk is summed against the current m (no maximum over its 32 values); only if the sum leaves
            // the safe range -- a value more than ~60 binary orders above m, or m still -inf at the start of an item --
            // is the reference refreshed, out of line.  The loop body is 32 x (fma, ex2, add) and nothing else.
#pragma unroll 2   // measured: 1, 2 and 4 give 685 / 667 / 680 us on the long-context shape
            for (int j = 0; j < 4; ++j) {
              SG_CHECK(as * 128 + j * 32 + 32 <= (int)kTmemCols);
              tmem_ld32_issue(cur, t_acc + (uint32_t)(j * 32));
              tmem_ld_wait(cur);
              if (j == 3) release_acc();
              float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
              for (int c = 0; c < 32; c += 4) {
                s0 += exp2f(fmaf(__uint_as_float(cur[c]), p.scale_log2, -m));
                s1 += exp2f(fmaf(__uint_as_float(cur[c + 1]), p.scale_log2, -m));
                s2 += exp2f(fmaf(__uint_as_float(cur[c + 2]), p.scale_log2, -m));
                s3 += exp2f(fmaf(__uint_as_float(cur[c + 3]), p.scale_log2, -m));
              }
              const float s = (s0 + s1) + (s2 + s3);
              if (s < 0x1p60f) lsum += s;
              else { const float2 ml = refresh_reference(p.scale_log2, m, lsum, cur[0], cur[1], cur[2], cur[3], cur[4], cur[5], cur[6], cur[7], cur[8], cur[9], cur[10], cur[11], cur[12], cur[13], cur[14], cur[15], cur[16], cur[17], cur[18], cur[19], cur[20], cur[21], cur[22], cur[23], cur[24], cur[25], cur[26], cur[27], cur[28], cur[29], cur[30], cur[31]); m = ml.x; lsum = ml.y; }
            }
            sm_m[r] = m;
            sm_l[r] = lsum;
          }
        }
        for (int tile = hot_end; tile < it.tile_end; ++tile) {
          if (!blockwise && (((tile_count++) % kEpiGroups) != (uint32_t)wg || !ok)) continue;
          const int t0 = tile * kTileKeys;
          const bool all_visible = t0 + kTileKeys - 1 <= first_win;
          for (int blk = 0; blk < nblk; ++blk) {
            if (blockwise && (((tile_count++) % kEpiGroups) != (uint32_t)wg || !ok)) continue;
            SG_PROF_BEGIN(ta);
            if (ok) ok = mbar_wait(bar_afull(as), aph, abort_flag, p.wait_ns, 0u);
            SG_PROF_ADD(w_afull, ta);
            SG_PROF_INC(n_blocks);
            if (!ok) continue;
            tc_fence_after();
            const int r = blk * 128 + row_in_tile;
            const bool row_ok = r < p.R && (r / p.G) < Weff;
            const int cmax = row_ok ? (first_win + r / p.G - t0) : -1;    // last visible column of this tile
            float m = sm_m[r], lsum = sm_l[r];
            uint32_t cur[32];
            // Chunk by chunk: where every row of the warp sees all 32 keys of the chunk (all but the last chunk or two
            // of a tile on the causal diagonal, and every chunk of a fully visible tile) the hot body, else per-column
            // masks with the true maximum.  (all_visible enters only to spare the vote on fully visible tiles.)
#pragma unroll 1
            for (int j = 0; j < 4; ++j) {
              const int col0 = j * 32;
              SG_CHECK(as * 128 + col0 + 32 <= (int)kTmemCols);
              tmem_ld32_issue(cur, t_acc + (uint32_t)col0);
              tmem_ld_wait(cur);
              if (j == 3) release_acc();
              if (!__all_sync(0xffffffffu, row_ok && (all_visible || col0 + 31 <= cmax))) {
                // Some (row, key) pairs of the chunk are hidden: a thread that sees nothing of it is done; the others
                // replace their hidden scores by -inf, which the body below ignores (exp2 of it is 0, no maximum takes it).
                if (col0 > cmax) continue;
#pragma unroll
                for (int c = 0; c < 32; ++c) cur[c] = (col0 + c <= cmax) ? cur[c] : 0xff800000u;
              }
              float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
              for (int c = 0; c < 32; c += 4) {
                s0 += exp2f(fmaf(__uint_as_float(cur[c]), p.scale_log2, -m));
                s1 += exp2f(fmaf(__uint_as_float(cur[c + 1]), p.scale_log2, -m));
                s2 += exp2f(fmaf(__uint_as_float(cur[c + 2]), p.scale_log2, -m));
                s3 += exp2f(fmaf(__uint_as_float(cur[c + 3]), p.scale_log2, -m));
              }
              const float s = (s0 + s1) + (s2 + s3);
              if (s < 0x1p60f) lsum += s;      // false also for the NaN that a hidden score gives while m is still -inf
              else { const float2 ml = refresh_reference(p.scale_log2, m, lsum, cur[0], cur[1], cur[2], cur[3], cur[4], cur[5], cur[6], cur[7], cur[8], cur[9], cur[10], cur[11], cur[12], cur[13], cur[14], cur[15], cur[16], cur[17], cur[18], cur[19], cur[20], cur[21], cur[22], cur[23], cur[24], cur[25], cur[26], cur[27], cur[28], cur[29], cur[30], cur[31]); m = ml.x; lsum = ml.y; }
            }
            sm_m[r] = m;
            sm_l[r] = lsum;
          }
        }
        // End of the item for this warp: its rows' statistics are complete in shared memory.  The helper warps merge
        // the warpgroups' slots, publish the item and count it as done for its unit, off this warp's path.
        SG_PROF_BEGIN(tp);
        __syncwarp();
        if (lane == 0 && ok) mbar_arrive(bar_stat_full(sbuf));
        SG_PROF_ADD(w_pub, tp);
      } else {
        const int nblk = (p.Rpad + 127) / 128;
        const bool blockwise = nblk > 1;
        // The helper warp has merged the unit's pass-1 statistics into this item's row log-sum-exps (it waited for
        // the unit's counter); two buffers, so it works on the next pass-2 item while this one runs.  Every warp
        // waits here, also one that gets no block of the item: passing this point proves that the buffer's previous
        // use was released by all sixteen warps, which keeps the arrivals below in step with the barrier's phases.
        const int lbuf = n_p2 & 1;
        const uint32_t lph = (uint32_t)((n_p2 >> 1) & 1);
        ++n_p2;
        SG_PROF_BEGIN(tl);
        if (ok) ok = mbar_wait(bar_lse_ready(lbuf), lph, abort_flag, p.wait_ns, 32u);
        SG_PROF_ADD(w_lse, tl);
        const float* lse2 = lse_buf + lbuf * p.Ralloc;   // [Ralloc] row log-sum-exps (log2 domain) of (unit, b)
        // End of a tile for this warp: its partial (or whole) column sum goes out.
        auto finish_tile = [&](const int tile, const int t, const float a0, const float a1, const float a2, const float a3, const uint32_t n0,
                               const bool mine) {
          float total = (a0 + a1) + (a2 + a3);
          if (blockwise) {
            // The tile's row blocks were dealt to different warpgroups.  Each warpgroup that had one leaves its partial
            // column sums in shared memory; per lane quarter, the warp that writes the last partial adds them up in a
            // fixed order (bitwise reproducible) and stores the importance -- no block-wide barrier per tile.  A slot
            // is reused S tiles later: block m is issued only after blocks m-4 .. m-7 were released, and the
            // warpgroups that released them had finished everything up to block m-8; with (S-1)*nblk >= 7 all
            // partials of the slot's previous tile are summed before the slot is written again.
            if (!mine) return;
            const int nwg = nblk < kEpiGroups ? nblk : kEpiGroups;      // warpgroups that drain blocks of this tile
            const int slot = tile & (nblk >= 4 ? 3 : 7);
            float* part = sm_part + slot * (kEpiGroups * 128);
            part[wg * 128 + row_in_tile] = total;
            __threadfence_block();
            __syncwarp();
            int old = 0;
            if (lane == 0) old = atomicAdd(&sm_cnt[slot * 4 + lane_grp], 1);
            old = __shfl_sync(0xffffffffu, old, 0);
            if (old != nwg - 1) return;
            __threadfence_block();
            total = 0.f;
            for (int i = 0; i < nwg; ++i) total += part[((n0 + i) % kEpiGroups) * 128 + row_in_tile];
            __syncwarp();
            if (lane == 0) sm_cnt[slot * 4 + lane_grp] = 0;
          }
          SG_CHECK(!(ok && t < N) || (it.c0 + t < p.T && it.l * p.Hkv + it.g < p.U));
          if (ok && t < N) p.importance[((size_t)it.l * p.Hkv + it.g) * p.T + it.c0 + t] = total;
        };
        // Two loops, as in pass 1: the tiles every window row sees completely, when every row block is full (hot body
        // only), then the rest in the general loop.
        const int vis_end = (first_win + 1) / kTileKeys;
        const int hot_end = (p.Rpad & 127) == 0 ? min(it.tile_end, max(it.tile_beg, vis_end)) : it.tile_beg;
        for (int tile = it.tile_beg; tile < hot_end; ++tile) {
          if (!blockwise && ((tile_count++) % kEpiGroups) != (uint32_t)wg) continue;   // (the wait below looks at `ok`)
          const int t = tile * kTileKeys + row_in_tile;  // this thread's key
          float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
          const uint32_t n0 = tile_count;                // running block count at the start of this tile
          bool mine = false;                             // this warpgroup drains at least one block of the tile
          for (int blk = 0; blk < nblk; ++blk) {
            if (blockwise && (((tile_count++) % kEpiGroups) != (uint32_t)wg || !ok)) continue;
            mine = true;
            SG_PROF_BEGIN(ta);
            if (ok) ok = mbar_wait(bar_afull(as), aph, abort_flag, p.wait_ns, 0u);
            SG_PROF_ADD(w_afull, ta);
            SG_PROF_INC(n_blocks);
            if (!ok) continue;
            tc_fence_after();
            uint32_t cur[32];
            // nothing but 32 x (fma, ex2, add) and the rows' log-sum-exps from shared memory
#pragma unroll 2
            for (int j = 0; j < 4; ++j) {
              SG_CHECK(as * 128 + j * 32 + 32 <= (int)kTmemCols && blk * 128 + j * 32 + 32 <= p.Ralloc);
              tmem_ld32_issue(cur, t_acc + (uint32_t)(j * 32));
              tmem_ld_wait(cur);
              if (j == 3) release_acc();
              const float* ls = lse2 + blk * 128 + j * 32;
#pragma unroll
              for (int c = 0; c < 32; c += 4) {
                const float4 l4 = *reinterpret_cast<const float4*>(ls + c);
                a0 += exp2f(fmaf(__uint_as_float(cur[c]), p.scale_log2, -l4.x));
                a1 += exp2f(fmaf(__uint_as_float(cur[c + 1]), p.scale_log2, -l4.y));
                a2 += exp2f(fmaf(__uint_as_float(cur[c + 2]), p.scale_log2, -l4.z));
                a3 += exp2f(fmaf(__uint_as_float(cur[c + 3]), p.scale_log2, -l4.w));
              }
            }
          }
          finish_tile(tile, t, a0, a1, a2, a3, n0, mine);
        }
        for (int tile = hot_end; tile < it.tile_end; ++tile) {
          if (!blockwise && (((tile_count++) % kEpiGroups) != (uint32_t)wg || !ok)) continue;
          const int t = tile * kTileKeys + row_in_tile;  // this thread's key
          const bool all_visible = tile * kTileKeys + kTileKeys - 1 <= first_win;
          const int rmin = (t - first_win) * p.G;        // rows below rmin cannot see key t
          float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
          const uint32_t n0 = tile_count;                // running block count at the start of this tile
          bool mine = false;                             // this warpgroup drains at least one block of the tile
          for (int blk = 0; blk < nblk; ++blk) {
            if (blockwise && (((tile_count++) % kEpiGroups) != (uint32_t)wg || !ok)) continue;
            mine = true;
            SG_PROF_BEGIN(ta);
            if (ok) ok = mbar_wait(bar_afull(as), aph, abort_flag, p.wait_ns, 0u);
            SG_PROF_ADD(w_afull, ta);
            SG_PROF_INC(n_blocks);
            if (!ok) continue;
            tc_fence_after();
            const int ncols = min(128, p.Rpad - blk * 128);
            const int nchk = (ncols + 31) >> 5;          // 32-column chunks of this block (warp-uniform)
            uint32_t cur[32];
            // Chunk by chunk: where all 32 rows of the chunk exist and see every key of the warp (on the causal diagonal:
            // all warps but the one that holds the window's own keys) the hot body, else per-column masks.
#pragma unroll 1
            for (int j = 0; j < nchk; ++j) {
              const int col0 = j * 32;
              SG_CHECK(as * 128 + col0 + 32 <= (int)kTmemCols && blk * 128 + col0 + 32 <= p.Ralloc);
              tmem_ld32_issue(cur, t_acc + (uint32_t)col0);
              tmem_ld_wait(cur);
              if (j == nchk - 1) release_acc();
              const float* ls = lse2 + blk * 128 + col0;
              if (!(col0 + 32 <= ncols && (all_visible || __all_sync(0xffffffffu, blk * 128 + col0 >= rmin)))) {
                // rows that do not see this thread's key (those below c_lo of this chunk), or that do not exist (from c_hi
                // on, in a partial last chunk): score -inf, probability 0
                const int c_lo = rmin - blk * 128 - col0, c_hi = ncols - col0;
                if (c_hi >= 32) {
#pragma unroll
                  for (int c = 0; c < 32; ++c) cur[c] = c >= c_lo ? cur[c] : 0xff800000u;
                } else {
#pragma unroll
                  for (int c = 0; c < 32; ++c) cur[c] = (c >= c_lo && c < c_hi) ? cur[c] : 0xff800000u;
                }
              }
#pragma unroll
              for (int c = 0; c < 32; c += 4) {
                const float4 l4 = *reinterpret_cast<const float4*>(ls + c);
                a0 += exp2f(fmaf(__uint_as_float(cur[c]), p.scale_log2, -l4.x));
                a1 += exp2f(fmaf(__uint_as_float(cur[c + 1]), p.scale_log2, -l4.y));
                a2 += exp2f(fmaf(__uint_as_float(cur[c + 2]), p.scale_log2, -l4.z));
                a3 += exp2f(fmaf(__uint_as_float(cur[c + 3]), p.scale_log2, -l4.w));
              }
            }
          }
          finish_tile(tile, t, a0, a1, a2, a3, n0, mine);
        }
        __syncwarp();
        if (lane == 0 && ok) mbar_arrive(bar_lse_free(lbuf));        // this warp no longer reads lse_buf[lbuf]
      }
    }
#ifdef SG_SCORE_PROFILE
    if (wg_tid == 0) { SG_PROF_STORE(9 + wg * 4, w_afull); SG_PROF_STORE(10 + wg * 4, w_lse); SG_PROF_STORE(11 + wg * 4, w_pub + w_sfree); SG_PROF_STORE(12 + wg * 4, n_blocks); }
#endif
  } else if (warp >= kHelperWarp) {
    // ------------------------------------------------------------ helper warps (two: each handles half of the rows)
    // Everything at an item boundary that is not arithmetic on scores runs here, off the epilogue's path:
    //   publish(k), k-th pass-1 item of this CTA: when all sixteen epilogue warps have left their statistics in shared
    //     memory, merge the warpgroups' slots per row, store one (max, sum) pair per row for the item, count the item
    //     as done for its unit (stores ordered before the count by a fence), and hand the buffer back;
    //   lse(j), j-th pass-2 item: when all pass-1 items of the unit are counted (bounded wait), merge the chunks' pairs
    //     of the item's sequence into the rows' log-sum-exps for the epilogue; this runs one pass-2 item ahead of it.
    // The two sequences advance independently and neither ever blocks: a task is taken only when a test shows that it
    // can run, so a publication this CTA owes can never be held up behind a count some other CTA still owes.
    const int hw = warp - kHelperWarp;
    long long pos1 = blockIdx.x, pos2 = blockIdx.x;      // schedule cursors of the next pass-1 / pass-2 item
    int k1 = 0, j2 = 0;
    ScoreItem it1, it2;
    it1.pass = it2.pass = 0;
    auto next_item = [&](long long& pos, ScoreItem& it, int pass) {   // advance to the next item of `pass` (it.pass = 0: none left)
      for (; pos < npos; pos += gridDim.x) {
        it = decode_position(p, pos, s_cu, s_prefix);
        if (it.pass == pass) { pos += gridDim.x; return; }
      }
      it.pass = 0;
    };
    next_item(pos1, it1, 1);
    next_item(pos2, it2, 2);
    uint64_t idle_since = 0;
    uint32_t idle_iters = 0;
    SG_PROF_DECL(h_free = 0, h_cnt = 0, h_merge = 0);
    while (it1.pass != 0 || it2.pass != 0) {
      bool progressed = false;
      if (it1.pass != 0 && mbar_test(bar_stat_full(k1 & 1), (uint32_t)((k1 >> 1) & 1))) {
        SG_PROF_BEGIN(th0);
        const int sbuf = k1 & 1;
        const float* bm = sm_stat + (size_t)(sbuf * 2 * p.wgslots) * p.Ralloc;
        const float* bl = bm + p.wgslots * p.Ralloc;
        const size_t slot = ((size_t)it1.unit * p.max_items + it1.item_in_unit) * p.Ralloc;
        for (int r = hw * 32 + lane; r < p.Ralloc; r += 64) {
          float M = bm[r];
          for (int w = 1; w < p.wgslots; ++w) M = fmaxf(M, bm[w * p.Ralloc + r]);
          const float Mu = M == -INFINITY ? 0.f : M;
          float L = 0.f;
          for (int w = 0; w < p.wgslots; ++w) L += bl[w * p.Ralloc + r] * exp2f(bm[w * p.Ralloc + r] - Mu);
          p.part[slot + r] = make_float2(M, L);
        }
        // each helper warp counts its half of the rows itself (a unit is complete at 2*C counts): its stores are ordered
        // before its count by the warp barrier plus one cumulative fence, and no hand-shake between the two warps is needed
        __syncwarp();
        if (lane == 0) {
          __threadfence();
          if (!*abort_flag && it1.unit != p.withhold_unit) atomicAdd(p.p1_done + it1.unit, 1);
          mbar_arrive(bar_stat_free(sbuf));
        }
        ++k1;
        next_item(pos1, it1, 1);
        progressed = true;
        SG_PROF_ADD(h_free, th0);
      }
      if (it2.pass != 0) {
        const int lbuf = j2 & 1, use = j2 >> 1;
        bool can = use == 0 || mbar_test(bar_lse_free(lbuf), (uint32_t)((use - 1) & 1));
        if (can) {
          int cnt = 0;
          if (lane == 0) cnt = ld_acquire_gpu(p.p1_done + it2.unit);
          cnt = __shfl_sync(0xffffffffu, cnt, 0);
          can = cnt >= 2 * C;
        }
        if (can) {
          SG_PROF_BEGIN(th2);
          __syncwarp();
          __threadfence();                             // the other lanes' loads follow lane 0's acquire
          float* lse2 = lse_buf + lbuf * p.Ralloc;
          const int Weff = min(p.W, it2.N);
          const size_t part_base = ((size_t)it2.unit * p.max_items + it2.first_item_b) * p.Ralloc;
          const int nparts = it2.nch_b;
          // a lane merges two neighbouring rows at a time (one 16-byte load per chunk), eight loads in flight
          for (int r = 2 * (hw * 32 + lane); r < p.Ralloc; r += 128) {
            float M0 = -INFINITY, L0 = 0.f, M1 = -INFINITY, L1 = 0.f;
            for (int c0 = 0; c0 < nparts; c0 += 8) {
              float4 v[8];
#pragma unroll
              for (int i = 0; i < 8; ++i)
                v[i] = c0 + i < nparts ? __ldcg(reinterpret_cast<const float4*>(p.part + part_base + (size_t)(c0 + i) * p.Ralloc + r))
                                       : make_float4(-INFINITY, 0.f, -INFINITY, 0.f);
              float m0 = v[0].x, m1 = v[0].z;
#pragma unroll
              for (int i = 1; i < 8; ++i) { m0 = fmaxf(m0, v[i].x); m1 = fmaxf(m1, v[i].z); }
              if (m0 != -INFINITY) {                   // else nothing of row r is visible in these chunks
                const float Mn = fmaxf(M0, m0);
                float acc = L0 * exp2f(M0 - Mn);
#pragma unroll
                for (int i = 0; i < 8; ++i) acc += v[i].y * exp2f(v[i].x - Mn);   // a (-inf, 0) pair adds 0
                M0 = Mn; L0 = acc;
              }
              if (m1 != -INFINITY) {
                const float Mn = fmaxf(M1, m1);
                float acc = L1 * exp2f(M1 - Mn);
#pragma unroll
                for (int i = 0; i < 8; ++i) acc += v[i].w * exp2f(v[i].z - Mn);
                M1 = Mn; L1 = acc;
              }
            }
            // rows outside the window get +inf: exp2(x - inf) = 0
            lse2[r] = (r < p.R && (r / p.G) < Weff) ? M0 + log2f(L0) : INFINITY;
            lse2[r + 1] = (r + 1 < p.R && ((r + 1) / p.G) < Weff) ? M1 + log2f(L1) : INFINITY;
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_lse_ready(lbuf));
          ++j2;
          next_item(pos2, it2, 2);
          progressed = true;
          SG_PROF_ADD(h_merge, th2);
        }
      }
      if (progressed) { idle_since = 0; idle_iters = 0; continue; }
      // nothing could run: sleep a little; every 64th idle round look at the abort flag and the clock (bounded wait)
      __nanosleep(40);
      if ((++idle_iters & 63u) == 0u) {
        if (*abort_flag) break;
        const uint64_t now = global_timer_ns();
        if (idle_since == 0) idle_since = now;
        else if (now - idle_since > 2ull * p.wait_ns) { *abort_flag = 1; break; }
      }
    }
#ifdef SG_SCORE_PROFILE
    if (warp == kHelperWarp && lane == 0) { SG_PROF_STORE(25, h_free); SG_PROF_STORE(26, h_cnt); SG_PROF_STORE(27, h_merge); }
#endif
  }

  // ---------------------------------------------------------------- teardown
  // This CTA has no work left: a kernel queued behind this one with programmatic stream serialization (the selection)
  // may have its CTAs placed from now on; it still waits for this whole grid's completion before it reads anything.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
  if (tid == 0 && *abort_flag) raise(p.dev_status, SG_ERR_TIMEOUT);
  if (p.clock_out && tid == 0) {
    unsigned long long* o = p.clock_out + kClockWords * (size_t)blockIdx.x;
    o[0] = clk0; o[1] = (unsigned long long)clock64(); o[2] = gt0; o[3] = global_timer_ns();
  }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess) return nullptr;
    if (qres != cudaDriverEntryPointSuccess) return nullptr;
    return reinterpret_cast<EncodeTiledFn>(ptr);
  }();
  return fn;
}

// Testing hooks (sg_testing_score_fault, sg_testing_score_clock): process-wide, off by default.
std::atomic<int> g_test_withhold_unit{-1};
std::atomic<int> g_test_wait_limit_ms{0};
std::atomic<unsigned long long*> g_test_clock_out{nullptr};

struct ScorePlan {
  int R, Rpad, Ralloc, k_stages, q_bufs, tiles_per_chunk, max_items, smem_bytes, U, lag, wgslots;
  size_t counter_bytes, workspace_bytes;
  bool ok;
};

ScorePlan plan_score(const sg_shape* s) {
  ScorePlan pl{};
  const int D = s->head_dim;
  const int G = s->num_q_heads / s->num_kv_heads;
  pl.R = G * s->window;
  pl.Rpad = (pl.R + 15) & ~15;
  pl.Ralloc = (pl.R + 127) & ~127;
  const int q_bytes = pl.Ralloc * D * 2;
  const int k_stage = kTileKeys * D * 2;
  const int part_slots = pl.Rpad > 384 ? 4 : (pl.Rpad > 128 ? 8 : 0);
  // Row blocks are dealt to the four epilogue warpgroups in rotation.  When their number is a multiple of four a
  // row block always meets the same warpgroup, so one statistics slot per item suffices; otherwise every
  // warpgroup keeps (and publishes) its own.
  pl.wgslots = ((pl.Ralloc / 128) % kEpiGroups == 0) ? 1 : kEpiGroups;
  const int tail = (240 + (2 + 4 * pl.wgslots) * pl.Ralloc * 4 + part_slots * kEpiGroups * 128 * 4 + kPartSlots * 4 * 4 + 32 + 2 * (s->batch + 1) * 4 + 15) & ~15;
  const int avail = kSmemLimit - 1024 - tail;
  // Two Q buffers let the next item's queries load while the current item computes; fall back to one
  // when that would leave fewer than three K stages.
  pl.q_bufs = 2;
  pl.k_stages = (avail - 2 * q_bytes) / k_stage;
  if (pl.k_stages < 3) { pl.q_bufs = 1; pl.k_stages = (avail - q_bytes) / k_stage; }
  if (pl.k_stages > kMaxKStages) pl.k_stages = kMaxKStages;
  pl.ok = pl.k_stages >= 2 && s->window <= 256 && pl.R <= 1024 && s->batch <= kMaxBatchSmem;
  pl.smem_bytes = 1024 + pl.q_bufs * q_bytes + pl.k_stages * k_stage + tail;
  if (pl.smem_bytes < 120 * 1024) pl.smem_bytes = 120 * 1024;     // one CTA per SM: each CTA takes the whole TMEM
  pl.U = s->num_layers * s->num_kv_heads;
  // Chunking of the key axis.  Above the roofline ridge (R = G*W flop per K byte vs ~218) the second read of K
  // need not come from L2, so items are long (32 tiles) to amortise the per-item work; below it they are shorter
  // (16 tiles; 8 measured 16 % slower on the 8B shape) so that a unit's keys are still L2-resident when its pass 2 starts.  Either is halved while that
  // leaves fewer than ~6 items per SM and pass.
  const int64_t tiles_per_unit = (int64_t)s->total_tokens / kTileKeys + s->batch;
  int tpc = pl.R >= 256 ? 32 : 16;
  while (tpc > 4 && (tiles_per_unit / tpc + s->batch) * pl.U < 6 * kNumSMs) tpc /= 2;
  pl.tiles_per_chunk = tpc;
  pl.max_items = (int)(tiles_per_unit / tpc + s->batch + 1);
  // Pass 2 of a unit trails its pass 1 by `lag` units.  The lag must span several times more schedule positions
  // than there are CTAs (each slot holds about 2*C positions): a pass-2 item needs every pass-1 item of its unit
  // published, and the helper warps prepare it one item ahead, so with a lag of one wave pass-2 items wait for
  // statistics (measured on the 8B shape: 12-19 % of the epilogue's time at 1.25 waves, < 5 % at 3.5).  Beyond
  // that it is kept small so that the unit's keys are still in L2 for the second read; 3.5 waves is where the
  // time stops falling (8B shape 268 -> 232 us, long-context shape 808 -> 740 us from 1.25 to 3.5 waves).
  const int64_t c_est = (tiles_per_unit - s->batch) / tpc + 1;
  int64_t lag = (14 * kNumSMs / 4 + 2 * c_est - 1) / (2 * c_est) + 1;
  if (2 * lag > pl.U) lag = pl.U;     // few units: all pass-1 items first, then all pass-2 items
  pl.lag = (int)lag;
  pl.counter_bytes = ((size_t)pl.U * sizeof(int) + 255) & ~(size_t)255;
  pl.workspace_bytes = pl.counter_bytes + (size_t)2 * pl.U * pl.max_items * pl.Ralloc * sizeof(float);
  return pl;
}

// Finish time of the static schedule under a simple model (an item costs its tiles, pass 2 a little more;
// a pass-2 item starts when its CTA is free and every pass-1 item of its unit is done).  CTA k takes
// positions k, k + grid, ...; with items of 4-32 tiles, where the empty positions fall decides whether some
// CTA ends up one item behind, so the host plays both layouts through and keeps the faster.
double simulate_schedule(int U, int C, int lag, bool compact, int grid, int tiles) {
  std::vector<double> clock((size_t)grid, 0.0), done1((size_t)U, 0.0);
  const long long npos = schedule_length(U, C, lag, compact);
  double end = 0.0;
  for (long long pos = 0; pos < npos; ++pos) {
    const SchedPos sp = schedule_position(pos, U, C, lag, compact);
    if (sp.pass == 0) continue;
    double& c = clock[(size_t)(pos % grid)];
    double start = c;
    if (sp.pass == 2 && done1[(size_t)sp.unit] > start) start = done1[(size_t)sp.unit];
    c = start + (sp.pass == 2 ? 1.1 : 1.0) * tiles + 1.0;
    if (sp.pass == 1 && c > done1[(size_t)sp.unit]) done1[(size_t)sp.unit] = c;
    if (c > end) end = c;
  }
  return end;
}

bool choose_compact_layout(const sg_shape* s, const ScorePlan& pl, int grid) {
  if (pl.lag >= pl.U) return false;                               // two-phase schedule: nothing to choose
  // items per unit and pass: exact for one sequence, an estimate for a ragged batch (lengths live on the device)
  const long long tiles_per_unit = s->batch == 1 ? ((long long)s->total_tokens + kTileKeys - 1) / kTileKeys
                                                 : (long long)s->total_tokens / kTileKeys + (s->batch + 1) / 2;
  const int C = (int)((tiles_per_unit + pl.tiles_per_chunk - 1) / pl.tiles_per_chunk);
  if (schedule_length(pl.U, C, pl.lag, false) > 40000) return false;   // long schedules: the ends do not matter
  return simulate_schedule(pl.U, C, pl.lag, true, grid, pl.tiles_per_chunk) <
         simulate_schedule(pl.U, C, pl.lag, false, grid, pl.tiles_per_chunk);
}

}  // namespace

size_t score_workspace_bytes(const sg_shape* s) {
  if (s->num_kv_heads < 1 || s->num_q_heads < 1 || s->window < 1 || s->num_layers < 1) return 0;
  if (s->num_q_heads % s->num_kv_heads != 0) return 0;
  return plan_score(s).workspace_bytes;
}

}  // namespace sg

extern "C" void sg_testing_score_fault(int32_t withhold_unit, int32_t wait_limit_ms) {
  sg::g_test_withhold_unit.store(withhold_unit, std::memory_order_relaxed);
  sg::g_test_wait_limit_ms.store(wait_limit_ms, std::memory_order_relaxed);
}

extern "C" void sg_testing_score_clock(void* dev_buffer) {
  sg::g_test_clock_out.store(static_cast<unsigned long long*>(dev_buffer), std::memory_order_relaxed);
}

extern "C" int32_t sg_testing_score_grid(const sg_shape* shape) {
  using namespace sg;
  if (check_shape(shape, true) != SG_OK) return 0;
  const ScorePlan pl = plan_score(shape);
  if (!pl.ok) return 0;
  const long long max_pos = (long long)(pl.U + pl.lag) * 2 * pl.max_items;
  return (int32_t)(max_pos < kNumSMs ? max_pos : kNumSMs);
}

extern "C" sg_status sg_score(const sg_shape* shape, const void* q_win, const void* k_cache, float* importance,
                              void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream) {
  using namespace sg;
  sg_status st = check_shape(shape, true);
  if (st != SG_OK) return st;
  if (shape->total_tokens == 0) return SG_OK;
  if (!q_win || !k_cache || !importance) return SG_ERR_INVALID;
  if (!aligned16(q_win) || !aligned16(k_cache) || !aligned16(importance) || !aligned16(workspace)) return SG_ERR_INVALID;
  const ScorePlan pl = plan_score(shape);
  if (!pl.ok) return SG_ERR_UNSUPPORTED;
  const size_t need = score_workspace_bytes(shape);
  if (!workspace || workspace_bytes < need) return SG_ERR_WORKSPACE;
  EncodeTiledFn encode = encode_tiled_fn();
  if (!encode) return cuda_fail((int)cudaErrorUnknown);

  const int D = shape->head_dim;
  const int G = shape->num_q_heads / shape->num_kv_heads;
  CUtensorMap tmap_q, tmap_k;
  {
    // q_win [L*B][W][H_q][d]; box = (64 of d, G heads, W rows, 1) -> rows ordered (window row, head in group)
    const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)shape->num_q_heads, (cuuint64_t)shape->window,
                                (cuuint64_t)shape->num_layers * shape->batch};
    const cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)shape->num_q_heads * D * 2,
                                   (cuuint64_t)shape->window * shape->num_q_heads * D * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)G, (cuuint32_t)shape->window, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = encode(&tmap_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(q_win), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cuda_fail((int)r);
  }
  {
    // k_cache viewed as (d, H_kv, T, L) with the caller's strides; box = 64 of d x 1 head x 128 tokens
    const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)shape->num_kv_heads, (cuuint64_t)shape->total_tokens,
                                (cuuint64_t)shape->num_layers};
    const cuuint64_t hs = shape->num_kv_heads > 1 ? (cuuint64_t)shape->cache_head_stride * 2 : (cuuint64_t)D * 2;
    const cuuint64_t ls = shape->num_layers > 1 ? (cuuint64_t)shape->cache_layer_stride * 2
                                                : (cuuint64_t)shape->cache_token_stride * 2 * shape->total_tokens;
    const cuuint64_t strides[3] = {hs, (cuuint64_t)shape->cache_token_stride * 2, ls};
    const cuuint32_t box[4] = {64, 1, (cuuint32_t)kTileKeys, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = encode(&tmap_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(k_cache), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cuda_fail((int)r);
  }

  ScoreParams p;
  p.cu = shape->cu_seqlens;
  p.importance = importance;
  p.p1_done = static_cast<int*>(workspace);
  p.part = reinterpret_cast<float2*>(static_cast<uint8_t*>(workspace) + pl.counter_bytes);
  p.dev_status = dev_status;
  p.T = shape->total_tokens;
  p.B = shape->batch;
  p.Hkv = shape->num_kv_heads;
  p.G = G;
  p.W = shape->window;
  p.R = pl.R;
  p.Rpad = pl.Rpad;
  p.Ralloc = pl.Ralloc;
  p.U = pl.U;
  p.lag = pl.lag;
  p.tiles_per_chunk = pl.tiles_per_chunk;
  p.max_items = pl.max_items;
  p.k_stages = pl.k_stages;
  p.q_bufs = pl.q_bufs;
  p.smem_bytes = pl.smem_bytes;
  p.wgslots = pl.wgslots;
  p.withhold_unit = g_test_withhold_unit.load(std::memory_order_relaxed);
  const int limit_ms = g_test_wait_limit_ms.load(std::memory_order_relaxed);
  p.wait_ns = limit_ms > 0 ? (uint32_t)limit_ms * 1000000u : 1000000000u;
  p.clock_out = g_test_clock_out.load(std::memory_order_relaxed);
  p.scale_log2 = kLog2e / sqrtf((float)D);

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the per-unit completion counters must start at zero on every call (also on every graph replay)
  SG_CUDA_TRY(cudaMemsetAsync(workspace, 0, pl.counter_bytes, s));
  int dev = 0, sms = kNumSMs;
  SG_CUDA_TRY(cudaGetDevice(&dev));
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) sms = kNumSMs;
  const long long max_pos = (long long)(pl.U + pl.lag) * 2 * pl.max_items;
  const unsigned grid = (unsigned)(max_pos < sms ? max_pos : sms);     // persistent: one CTA per SM
  p.compact = choose_compact_layout(shape, pl, (int)grid) ? 1 : 0;
  if (D == 128) {
    SG_ENSURE_SMEM((score_kernel<128>), pl.smem_bytes);
    score_kernel<128><<<grid, kScoreThreads, pl.smem_bytes, s>>>(tmap_q, tmap_k, p);
  } else {
    SG_ENSURE_SMEM((score_kernel<64>), pl.smem_bytes);
    score_kernel<64><<<grid, kScoreThreads, pl.smem_bytes, s>>>(tmap_q, tmap_k, p);
  }
  SG_CUDA_TRY(cudaGetLastError());
  return SG_OK;
}

// ---------------------------------------------------------------------------------------------
// sg_score_static: sg_score for callers that cannot allocate device memory.
//
// The row statistics that pass 1 hands to pass 2 normally live in a caller-provided workspace.
// Here they live in a fixed array that is part of the library image, so the caller needs no
// allocator at all.  The array is shared by every call on a device and keeps the previous call's
// contents.  The per-unit completion counters at its start must be zero when the kernel begins: the
// call clears them with a memset on `stream`, exactly as sg_score does for a caller's workspace.
// Every other word is written by pass 1 before pass 2 reads it.
namespace sg {
namespace {
static __device__ __align__(256) unsigned char g_score_static_scratch[SG_SCORE_STATIC_SCRATCH_BYTES];
}  // namespace
}  // namespace sg

extern "C" sg_status sg_score_static(const sg_shape* shape, const void* q_win, const void* k_cache,
                                     float* importance, int32_t* dev_status, void* stream) {
  using namespace sg;
  sg_status st = check_shape(shape, true);
  if (st != SG_OK) return st;
  if (shape->total_tokens == 0) return SG_OK;
  if (!plan_score(shape).ok) return SG_ERR_UNSUPPORTED;      // same answer as sg_score for shapes no kernel covers
  if (score_workspace_bytes(shape) > (size_t)SG_SCORE_STATIC_SCRATCH_BYTES) return SG_ERR_WORKSPACE;
  // In host code the array's name is only a handle; the device address has to be asked for, once per
  // device, with that device current.
  static std::atomic<void*> scratch_of_device[64];
  int dev = 0;
  SG_CUDA_TRY(cudaGetDevice(&dev));
  void* scratch = (dev >= 0 && dev < 64) ? scratch_of_device[dev].load(std::memory_order_acquire) : nullptr;
  if (!scratch) {
    SG_CUDA_TRY(cudaGetSymbolAddress(&scratch, g_score_static_scratch));
    if (dev >= 0 && dev < 64) scratch_of_device[dev].store(scratch, std::memory_order_release);
  }
  return sg_score(shape, q_win, k_cache, importance, scratch, (size_t)SG_SCORE_STATIC_SCRATCH_BYTES, dev_status, stream);
}
