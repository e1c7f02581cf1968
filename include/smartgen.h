/*
 * smartgen.h -- C ABI of the selective-KV hot path on one B200 (sm_100a).
 *
 * Four calls cover the path: on the prefill side, score every prompt token's importance for each
 * (layer, KV head), pick each head's top-k tokens under a KV budget, and gather-pack the selected
 * K/V rows into one contiguous transfer-ready buffer; on the decode side, attention whose keys and
 * values come partly from that packed buffer and partly from an index-addressed local cache.
 *
 * Conventions shared by every call
 *   - Every pointer named in a signature is a DEVICE pointer unless the comment says "host".
 *     All device pointers must be 16-byte aligned.  The caller owns every buffer; the library
 *     allocates nothing, keeps no state between calls and never synchronises the stream.
 *   - bf16 tensors are passed as `const void*` / `void*` (raw bfloat16 bit patterns).
 *   - The batch is ragged: sequence b owns tokens cu_seqlens[b] .. cu_seqlens[b+1]-1 of a
 *     token-major cache; N_b = cu_seqlens[b+1] - cu_seqlens[b].
 *   - The return value reports errors the host can see before launching (bad arguments,
 *     unsupported shape, workspace too small, a failed CUDA call).  Problems only the device can
 *     see (an index outside its sequence, a budget above the prompt length, a bounded wait that
 *     expired) are OR-ed into *dev_status as (1 << sg_status) bits, if dev_status is not NULL,
 *     and the offending row is skipped or clamped -- never dereferenced.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Inputs are never modified.  Calls are thread-safe given distinct streams and workspaces.
 */
#ifndef SMARTGEN_H_
#define SMARTGEN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SG_OK = 0,
  SG_ERR_INVALID = 1,     /* null or misaligned pointer, bad shape, k_b > N_b (device bit) ...   */
  SG_ERR_UNSUPPORTED = 2, /* head_dim not 64/128, H_q % H_kv != 0, G*W beyond the built tiles ... */
  SG_ERR_WORKSPACE = 3,   /* workspace_bytes < sg_workspace_bytes(...)                            */
  SG_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed; see sg_last_cuda_error()          */
  SG_ERR_INDEX = 5,       /* device bit: an index outside its sequence was skipped                */
  SG_ERR_TIMEOUT = 6      /* device bit: a bounded wait inside a kernel expired                   */
} sg_status;

/* Operation ids for sg_workspace_bytes. */
enum { SG_OP_SCORE = 0, SG_OP_SELECT_TOPK = 1, SG_OP_PACK_KV = 2, SG_OP_SPARSE_DECODE_ATTN = 3,
       SG_OP_SPLIT_INDEX = 4 };

/* Shape of one call (host memory, passed by const pointer).  Strides are in ELEMENTS (bf16). */
typedef struct {
  int32_t num_layers;         /* layers covered by this call (>= 1); decode/split: must be 1      */
  int32_t batch;              /* B >= 1                                                           */
  int32_t num_q_heads;        /* H_q                                                              */
  int32_t num_kv_heads;       /* H_kv, H_q % H_kv == 0, G = H_q / H_kv <= 16                      */
  int32_t head_dim;           /* d in {64, 128}                                                   */
  int32_t window;             /* W, scoring window (sg_score only)                                */
  int32_t total_tokens;       /* T = cu_seqlens[B]                                                */
  int32_t max_seqlen;         /* an upper bound on every N_b (launch geometry, shared memory)     */
  const int32_t* cu_seqlens;  /* device, B+1 ascending prefix sums, cu_seqlens[0] = 0             */
  int64_t cache_layer_stride; /* elements between layers of the K (and V) cache                   */
  int64_t cache_token_stride; /* elements between tokens  (H_kv*d when dense, multiple of 8)      */
  int64_t cache_head_stride;  /* elements between KV heads (d when token-major, multiple of 8)    */
} sg_shape;

/* Bytes of device workspace the given operation needs for this shape.  total_sel = K_tot (sum of
 * the per-sequence budgets k_b), total_loc = NL_tot (sum of the per-sequence local-index counts);
 * pass 0 where an operation does not use them.  Returns 0 for operations that need none. */
size_t sg_workspace_bytes(int op, const sg_shape* shape, int32_t total_sel, int32_t total_loc);

/*
 * sg_score -- importance of every prompt token for every (layer, KV head).
 *
 * Defines: the paper ranks KV entries by attention-score magnitude and counts how often an entry
 * is picked (Section 4.1, definition of importance; S(e) in Eq. 1 is a sum over occurrences);
 * attention is softmax(Q K^T / sqrt(d)) with each query seeing itself and all previous tokens
 * (Section 2.1).  The last W prompt queries stand in for the decode queries the prefill side
 * cannot see:
 *     importance[l][g][cu[b]+t] = sum over the G query heads h of KV head g and the
 *         W_eff = min(W, N_b) window rows i of softmax_t( q_{h,i} . k_{g,t} / sqrt(d) ),
 *     the softmax of row i running over the keys t <= N_b - W_eff + i (its own position).
 *
 * q_win       bf16 [L][B][W][H_q][d], dense; row i of sequence b is the query at N_b - W_eff + i.
 * k_cache     bf16, element (l, token, g, c) at l*layer_stride + token*token_stride + g*head_stride + c.
 * importance  fp32 [L][H_kv][T], fully overwritten.
 * Supported: G*W <= 512 (d = 128) or <= 1024 (d = 64), W <= 256, B <= 1024; otherwise SG_ERR_UNSUPPORTED.
 */
sg_status sg_score(const sg_shape* shape, const void* q_win, const void* k_cache, float* importance,
                   void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream);

/*
 * sg_select_topk -- per-head top-k KV index under a budget.
 *
 * Defines: a KV index row holds the k entries selected for one head of one request
 * (Section 2.3, BH x k KV index).  For every (l, b, g) the k_b = cu_k[b+1] - cu_k[b] positions
 * of sequence b with the largest importance are kept.  Order of values: the total order of the
 * fp32 bit patterns (+0 above -0, +inf above every finite value -- so entries given infinite
 * importance as in Eq. 1 are always kept); equal values go to the lower position.  NaNs take the
 * place their bit patterns have in that order: a NaN with a clear sign bit ranks above +inf, one with
 * a set sign bit below -inf, two NaNs by payload (sg_score never produces a NaN from finite inputs).
 * Each row is emitted in ascending position order (entry order does not change attention, Section 4.2).
 *
 * importance  fp32 [L][H_kv][T].
 * cu_k        device int32 [B+1], prefix sums of k_b; total_sel = cu_k[B] (host copy of the total).
 * sel_idx     int32 [L][H_kv][K_tot]; the row segment of (l, g, b) starts at cu_k[b]; positions
 *             are sequence-local (0 .. N_b-1).  k_b > N_b sets the SG_ERR_INVALID device bit and
 *             the row is filled with 0 .. N_b-1 followed by -1.  A sequence longer than
 *             shape->max_seqlen (which sizes the kernel's key storage) sets the same bit and its
 *             rows are filled with -1; nothing outside the provided buffers is touched.
 */
sg_status sg_select_topk(const sg_shape* shape, const float* importance, const int32_t* cu_k,
                         int32_t total_sel, int32_t* sel_idx, void* workspace, size_t workspace_bytes,
                         int32_t* dev_status, void* stream);

/*
 * sg_pack_kv -- gather the selected K/V rows into a contiguous, transfer-ready buffer.
 *
 * Defines: the selected KV has shape BH x k x d, a "row" being the k entries of one head
 * (Section 4.2); the prefill node selects the required entries locally before sending them.
 *     packed_k[l][cu_k[b]*H_kv + g*k_b + j][:] = k_cache[l][cu[b] + sel_idx[l][g][cu_k[b]+j]][g][:]
 * and the same for V.  An index outside [0, N_b) sets the SG_ERR_INDEX device bit and its row is
 * written as zeros.
 *
 * packed_k/v  bf16 [L][K_tot*H_kv][d], fully overwritten.
 */
sg_status sg_pack_kv(const sg_shape* shape, const void* k_cache, const void* v_cache,
                     const int32_t* sel_idx, const int32_t* cu_k, int32_t total_sel, void* packed_k,
                     void* packed_v, int32_t* dev_status, void* stream);

/*
 * sg_select_pack_kv -- sg_select_topk followed by sg_pack_kv in one call: the prefill node selects the
 * required entries and gathers them for sending (Section 4.2).  Writes exactly what the two calls write:
 * sel_idx (the KV index, which travels with the payload) and packed_k / packed_v, with the same device status
 * bits.  When every row has at most 32768 tokens and there are at least as many (layer, sequence, KV head)
 * rows as SMs, one kernel does both: the CTA that selected a row gathers that row's K/V, so the latency-bound
 * selection of some rows overlaps the bandwidth-bound gather of others.  Otherwise the two kernels are launched
 * back to back.  Arguments as in sg_select_topk and sg_pack_kv; no workspace; asynchronous on `stream`.
 */
sg_status sg_select_pack_kv(const sg_shape* shape, const float* importance, const int32_t* cu_k,
                            int32_t total_sel, const void* k_cache, const void* v_cache, int32_t* sel_idx,
                            void* packed_k, void* packed_v, int32_t* dev_status, void* stream);

/*
 * sg_sparse_decode_attn -- one decode step of attention over a two-source KV list.
 *
 * Defines: two-lane KV fetching (Section 4.2): the entries a head needs arrive partly as
 * contiguous rows at the start of its row of the selected KV (the packed buffer) and partly by
 * gathering with a local index from the decode node's own cache.  Because the order of KV
 * entries along the sequence axis does not change softmax(q K^T / sqrt(d)) V (Section 4.2), the
 * result for (b, h), g = h / G, is plain attention (Section 2.1) over the multiset
 *     [packed rows 0..k_b-1 of (b, g)] ++ [local rows cu[b] + local_idx[g][cu_nloc[b]+j], j < n_loc_b],
 * computed as split-softmax partials merged through their log-sum-exps.  Nothing is
 * de-duplicated.  A local index outside [0, N_b) sets the SG_ERR_INDEX device bit and is skipped.
 *
 * shape       num_layers must be 1; cache strides describe local_k / local_v.
 * q           bf16 [B][H_q][d].
 * packed_k/v  bf16 [K_tot*H_kv][d], layout of sg_pack_kv for one layer; cu_k as in sg_pack_kv.
 * local_k/v   bf16, element (token, g, c) at token*token_stride + g*head_stride + c.
 * local_idx   int32 [H_kv][NL_tot]; cu_nloc device int32 [B+1]; total_loc = cu_nloc[B].
 *             The host totals are binding: with one sequence (B = 1) the kernel takes k_0 = total_sel,
 *             n_loc_0 = total_loc and N_0 = shape->total_tokens from the arguments and does not read the
 *             prefix arrays at all (they must still be valid pointers that hold {0, total}).
 * softmax_scale  0 means 1/sqrt(d).
 * out         bf16 [B][H_q][d]; lse fp32 [B][H_q] (may be NULL) = max + ln(sum) of the scaled
 *             scores.  A head with an empty list gets out = 0 and lse = -inf.
 * workspace   unused (split-KV partials are merged on chip); sg_workspace_bytes returns 0.
 *
 * Stream ordering: the kernel is launched with programmatic dependent launch and lets the next kernel
 * in the stream start early.  out / lse are written only after all earlier work in the stream has completed.
 * Every INPUT -- q, the KV sources (packed_k/v, local_k/v), local_idx, the per-head count arrays and the
 * prefix arrays (cu_seqlens, cu_k, cu_nloc) -- is treated as a stable input of the decode step and may be
 * read while an immediately preceding kernel THAT ITSELF OPTED IN to programmatic dependent launch (such as
 * the previous layer's sg_sparse_decode_attn, or sg_score) is still running: inputs must not be outputs of
 * such a kernel.  Ordinary preceding kernels (the projection that produces q, a copy, anything launched the
 * usual way) are fully ordered before this call as usual.  Independent calls issued back to back therefore
 * overlap everything but their output stores.
 */
sg_status sg_sparse_decode_attn(const sg_shape* shape, const void* q, const void* packed_k,
                                const void* packed_v, const int32_t* cu_k, int32_t total_sel,
                                const void* local_k, const void* local_v, const int32_t* local_idx,
                                const int32_t* cu_nloc, int32_t total_loc, float softmax_scale,
                                void* out, float* lse, void* workspace, size_t workspace_bytes,
                                int32_t* dev_status, void* stream);

/*
 * sg_split_index -- split a KV index into its local and remote parts (Algorithm 1).
 *
 * Defines: Algorithm 1, KV index splitting and reordering (Section 4.2).  The KV mask holds one int8 per
 * token, shared by all heads, naming the token's class: 0 = padding, 1 = the token's KV entries are locally
 * available, 2 = they reside on a remote prefill node.  Every row of the KV index (one sequence, one KV head)
 * is split by the class of its entries: local_index receives the entries of class 1 and remote_index those of
 * class 2, each in the row's own order.  With `reorder`, the row is also returned as a stable three-way
 * partition by class (remote first, then local, then padding; entries keep their relative order inside a
 * class), so that the remote entries are contiguous at the start of the row.
 * Padding entries (mask 0) are dropped from both lists; an index outside [0, N_b) sets the SG_ERR_INDEX
 * device bit and is treated as padding.
 *
 * shape        num_layers must be 1 (one call per layer's KV index).
 * kv_index     int32 [H_kv][K_tot], row segment of sequence b at cu_k[b], sequence-local positions
 *              (the layout sg_select_topk writes for one layer); cu_k device int32 [B+1].
 * kv_mask      int8 [T], ragged by cu_seqlens.
 * reordered    int32 [H_kv][K_tot] or NULL: the partitioned row (a copy when reorder == 0).
 * local_index, remote_index  int32 [H_kv][K_tot]: each row segment is filled from its start; the counts
 *              go to n_local / n_remote, int32 [B][H_kv].  Entries past the counts are left untouched.
 * The lists feed sg_sparse_decode_attn: local_index (compacted per head) is its local-lane index list,
 * remote_index is what the prefill side gathers with sg_pack_kv.
 */
sg_status sg_split_index(const sg_shape* shape, const int32_t* kv_index, const int32_t* cu_k, int32_t total_sel,
                         const int8_t* kv_mask, int32_t reorder, int32_t* reordered, int32_t* local_index,
                         int32_t* remote_index, int32_t* n_local, int32_t* n_remote, int32_t* dev_status,
                         void* stream);

/*
 * Profile-based proactive selection (Section 4.1) -- the second "next" row of the path.
 *
 * Blocks: every layer's cache is partitioned along the sequence into M = num_blocks KV blocks; token t of a
 * sequence of length N_b belongs to block floor(t * M / N_b).  A block holds its tokens' entries of all KV heads.
 *
 * sg_profile_accumulate -- S(e) of Eq. 1 (Section 4.1), the selection count of a KV entry over the profiled
 *   decode steps: adds 1 to counts[g][cu[b] + t] for every entry t of one layer's KV index of one decode
 *   step.  shape->num_layers must be 1; kv_index int32 [H_kv][K_tot] with cu_k as in sg_select_topk;
 *   counts int32 [H_kv][T] (the caller zeroes it before the first call).  Out-of-range entries set SG_ERR_INDEX.
 * sg_block_importance -- Eq. 1: importance[l][m] = +inf for l = 0, 1 (the first two layers are always
 *   selected); otherwise the mean of S(e) over the entries of block B_{l,m} (all its tokens, all KV heads, all
 *   profiled sequences), a double division rounded to fp32; an empty block gets 0.
 *   counts int32 [L][H_kv][T]; importance fp32 [L][M].
 * sg_transfer_budget -- Eq. 2 (host arithmetic, no GPU): K_r = M (L-1) T_p / T_t rounded down, clipped to
 *   [2M, LM].  The global top-K_r blocks are then sg_select_topk on importance viewed as one row of L*M values.
 * sg_proactive_mask -- the KV mask of layer `layer` after the proactive transfer (Section 4.2: 1 = locally
 *   available, 2 = on the remote prefill node): tokens whose block's flat id layer*M + m is in `selected`
 *   (int32 [num_selected], ascending -- sg_select_topk's output) get 1, all others 2.  kv_mask int8 [T].
 *   The mask is what sg_split_index consumes.
 * sg_push_blocks -- the online transfer of one layer (Section 4.1, "Online KV transfer": the layer's cache is
 *   split into M blocks and every block whose position is among the top-K_r is pushed to the decoding node's
 *   KV cache pool): for every token of `layer` whose block's flat id layer*M + m is in `selected` (ascending,
 *   as for sg_proactive_mask), the rows of all KV heads are copied from src_k/src_v to the same positions of
 *   dst_k/dst_v.  Both caches are bf16, device, addressed with the shape's strides; the call covers the
 *   shape->num_layers consecutive layers layer, layer + 1, ... (the pointers address the first of them; 1 =
 *   the paper's layer-by-layer push as each layer is offloaded); rows of other blocks are not written.
 *   kv_mask (int8 [shape->num_layers][T], device, may be NULL): the decode-side KV mask of those layers; the
 *   tokens of every pushed block are set to 1 (Section 4.2: every pushed block is followed by an update of the
 *   decode-side KV mask), all other entries keep their value (2 = remote, 0 = padding).  The same call with the
 *   blocks of a speculative transfer (Section 4.3) completes the mask over the decoding iterations.  The network hop is out of scope: the
 *   destination is another HBM buffer.  src and dst must not overlap.
 * sg_speculative_delivered -- speculative transfer (Section 4.3; host arithmetic, no GPU): after the prefill
 *   stage pushed the top-K_r blocks, every decoding iteration delivers the next blocks in the order of their
 *   Eq. 1 importance, at most `ratio` of all L*M blocks per iteration (rounded down, at least one).  Returns the
 *   number n of blocks on the decode node after `iteration` speculative transfers; the set is the global top-n
 *   (sg_select_topk with budget n) and the layer masks follow from sg_proactive_mask with that set.
 */
sg_status sg_profile_accumulate(const sg_shape* shape, const int32_t* kv_index, const int32_t* cu_k, int32_t total_sel,
                                int32_t* counts, int32_t* dev_status, void* stream);
sg_status sg_block_importance(const sg_shape* shape, const int32_t* counts, int32_t num_blocks, float* importance,
                              void* stream);
int64_t sg_transfer_budget(int32_t num_layers, int32_t num_blocks, double t_prefill, double t_transfer);
sg_status sg_proactive_mask(const sg_shape* shape, int32_t num_blocks, int32_t layer, const int32_t* selected,
                            int32_t num_selected, int8_t* kv_mask, void* stream);
sg_status sg_push_blocks(const sg_shape* shape, int32_t num_blocks, int32_t layer, const int32_t* selected,
                         int32_t num_selected, const void* src_k, const void* src_v, void* dst_k, void* dst_v,
                         int8_t* kv_mask, void* stream);
int64_t sg_speculative_delivered(int32_t num_layers, int32_t num_blocks, int64_t k_r, double ratio, int32_t iteration);

/*
 * sg_select_threshold -- threshold selection under a cap, the rule of the KV selection algorithm the paper
 * deploys (Section 5.1, "Parameters": an alpha value and a maximum KV selection ratio): per (layer, sequence,
 * KV head) every token whose score exceeds the row maximum minus `alpha` is selected, at most
 * cap_b = cu_cap[b+1] - cu_cap[b] of them; if more exceed the threshold the cap_b largest are kept, ties to the
 * lower index.  The comparison is strict.  Scores must not be NaN (sg_score never produces one): a NaN is never
 * selected, but which of the other tokens of its row are is then unspecified (always in range, never a fault).
 *   scores    fp32 [L][H_kv][T], device (any per-token score; sg_score's importance has this layout)
 *   alpha     >= 0, in the units of the scores
 *   cu_cap    int32 [B+1], device: prefix sums of the caps (0 <= cap_b <= N_b), total_cap = cu_cap[B] on the host
 *   sel_idx   int32 [L][H_kv][total_cap], device, written: per row the selected sequence-local positions in
 *             ascending order, then -1 up to cap_b
 *   sel_count int32 [L][B][H_kv], device, written: the number selected per row
 * Runs sg_select_topk with the caps as budgets, then trims each row at the threshold; the counts differ per KV
 * head, so the rows go to sg_pack_kv_counted / sg_sparse_decode_attn_counted (sg_pack_kv takes one budget per
 * sequence).
 * Errors as sg_select_topk.
 */
sg_status sg_select_threshold(const sg_shape* shape, const float* scores, float alpha, const int32_t* cu_cap,
                              int32_t total_cap, int32_t* sel_idx, int32_t* sel_count, int32_t* dev_status, void* stream);

/*
 * sg_pack_kv_counted, sg_sparse_decode_attn_counted -- the gather-pack and the decode attention for a selection
 * that kept a different number of entries per KV head (sg_select_threshold).  The packed buffer keeps the layout
 * of sg_pack_kv with the caps as budgets (row of (b, g, j) = cu_cap[b]*H_kv + g*cap_b + j), so every head owns a
 * slot of cap_b rows, of which only the first count are meaningful:
 *   sg_pack_kv_counted            sel_count int32 [L][B][H_kv], device: entries j >= sel_count[l][b][g] of a row of
 *                                 sel_idx are skipped (not read, their rows of packed_k/packed_v not written);
 *                                 everything else as sg_pack_kv with cu_cap / total_cap in place of cu_k / total_sel.
 *   sg_sparse_decode_attn_counted packed_count int32 [B][H_kv], device (one layer's slice of sel_count): the list of
 *                                 (b, g) is its first packed_count[b][g] packed rows, then its local rows; values
 *                                 are clamped to [0, cap_b].  local_skip int32 [B][H_kv], device: the first
 *                                 local_skip[b][g] entries of the local-index row of (b, g) are not in the list
 *                                 (clamped to the row).  Either array may be NULL (not both).  No workspace.
 *                                 Everything else as sg_sparse_decode_attn.
 * With every count equal to its cap (and no skip) the two calls are sg_pack_kv and sg_sparse_decode_attn.
 * Two-lane fetching (Section 4.2) with these calls: sg_split_index with reorder gives, per head, the KV index with
 * its n_remote[b][g] remote entries first; sg_pack_kv_counted(sel_idx = reordered, sel_count = n_remote) fetches the
 * remote lane from the prefill-side cache; sg_sparse_decode_attn_counted(packed_count = n_remote, local_idx =
 * reordered, cu_nloc = cu_k, local_skip = n_remote) attends the fetched rows and the local rest of every row.
 */
sg_status sg_pack_kv_counted(const sg_shape* shape, const void* k_cache, const void* v_cache, const int32_t* sel_idx,
                             const int32_t* cu_cap, int32_t total_cap, const int32_t* sel_count, void* packed_k,
                             void* packed_v, int32_t* dev_status, void* stream);
sg_status sg_sparse_decode_attn_counted(const sg_shape* shape, const void* q, const void* packed_k, const void* packed_v,
                                        const int32_t* cu_cap, int32_t total_cap, const int32_t* packed_count,
                                        const void* local_k, const void* local_v, const int32_t* local_idx,
                                        const int32_t* cu_nloc, int32_t total_loc, const int32_t* local_skip,
                                        float softmax_scale, void* out, float* lse, int32_t* dev_status, void* stream);

/*
 * sg_score_static -- sg_score without a workspace argument, for callers that cannot allocate.
 *
 * The paper has no counterpart to this call: it computes exactly what sg_score computes.  It exists
 * for hosts of this library that may not call cudaMalloc (or any allocating routine) at the point
 * where they score -- code running under a fixed memory plan, inside a region where allocation is
 * forbidden, or in a process whose allocator belongs to another runtime.  The scratch that pass 1
 * and pass 2 of the scoring kernel exchange lives in a fixed array inside the library image,
 * SG_SCORE_STATIC_SCRATCH_BYTES long; every GPU that loads the library holds that much memory until
 * the process exits.
 *
 *   - Shapes whose sg_workspace_bytes(SG_OP_SCORE, ...) exceeds SG_SCORE_STATIC_SCRATCH_BYTES are
 *     rejected with SG_ERR_WORKSPACE before anything is launched; use sg_score for those.
 *   - The call allocates nothing and frees nothing.  The first call on each device looks up the
 *     array's device address (one cudaGetSymbolAddress with that device current); make that first
 *     call before starting any stream capture on the device.
 *   - All calls on a device share the one array, which keeps the previous call's contents.  The
 *     call itself clears the few counters in it that must start at zero (a memset on `stream`);
 *     everything else is written before it is read within a call.  But two calls
 *     that overlap on the GPU -- different streams, or one stream's call still running when another
 *     starts -- race on it and give undefined importance.  Serialise them, or use sg_score with
 *     separate workspaces.
 *   - Inputs, outputs, status word and error behaviour are those of sg_score.
 */
#define SG_SCORE_STATIC_SCRATCH_BYTES (8u << 20)
sg_status sg_score_static(const sg_shape* shape, const void* q_win, const void* k_cache, float* importance,
                          int32_t* dev_status, void* stream);

/* Static description of a status code. */
const char* sg_strerror(sg_status status);

/* cudaError_t (or CUresult for driver calls) of the last failed CUDA call on this host thread. */
int sg_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SMARTGEN_H_ */
