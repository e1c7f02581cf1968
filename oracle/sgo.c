/*
 * CPU oracle for the selective-KV hot path (TEST INFRASTRUCTURE, not a product path).
 *
 * Plain, slow, scalar C written from the paper's definitions.  It shares no code with the
 * CUDA library and must never be called from it: only the tests, the smoke check and the
 * benchmark's cpu-baseline leg load this file.
 *
 * Arithmetic: bf16 inputs are widened exactly; every dot product, exponential and sum is in
 * double; results are rounded once to float.  The only parallelism is an OpenMP loop over
 * independent (layer, sequence, KV head) units.
 *
 * Notation (paper, Section 2.1 / 2.3): H x N x d tensors per layer, attention
 * softmax(Q K^T / sqrt(d)) V per head; the "KV index" is a BH x k matrix whose rows hold the k
 * selected entries of one head of one request; the "selected KV" has shape BH x k x d.
 * Here the batch is ragged: sequence b owns tokens cu[b] .. cu[b+1]-1 of a token-major cache.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_double(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int sgo_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void sgo_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/*
 * Importance of every prompt token for every (layer, KV head).
 *
 * Section 4.1 defines a KV entry's importance through how often the selection algorithm picks
 * it, and notes that all such algorithms rank entries by attention-score magnitude; S(e) in
 * Eq. 1 is a plain count (a sum over occurrences).  The prefill side cannot see decode queries,
 * so the last W prompt queries stand in for them: importance[t] is the attention mass
 * (Section 2.1: softmax(q K^T / sqrt(d)), each query attending to itself and all previous
 * tokens) that those W queries of the G query heads sharing KV head g put on token t, summed
 * over the G*W rows without normalisation.
 *
 * q_win      bf16 [L][B][W][Hq][d]; row i of sequence b is the query at position N_b - W_eff + i,
 *            W_eff = min(W, N_b); rows i >= W_eff are ignored.
 * k_cache    bf16, element (l, token, g, c) at l*ls + token*ts + g*hs + c.
 * importance float [L][Hkv][T].
 */
int sgo_score(int L, int B, int Hq, int Hkv, int d, int W, const int32_t *cu,
              const uint16_t *q_win, const uint16_t *k_cache, int64_t ls, int64_t ts, int64_t hs,
              float *importance) {
    if (Hkv <= 0 || Hq % Hkv != 0 || d <= 0 || W <= 0) return 1;
    const int G = Hq / Hkv;
    const int64_t T = cu[B];
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    int fail = 0;
#pragma omp parallel for collapse(3) schedule(dynamic, 1)
    for (int l = 0; l < L; ++l)
        for (int b = 0; b < B; ++b)
            for (int g = 0; g < Hkv; ++g) {
                const int64_t c0 = cu[b];
                const int N = cu[b + 1] - cu[b];
                float *imp = importance + ((int64_t)l * Hkv + g) * T + c0;
                if (N <= 0) continue;
                const int Weff = W < N ? W : N;
                double *acc = (double *)calloc((size_t)N, sizeof(double));
                double *s = (double *)malloc((size_t)N * sizeof(double));
                double *qd = (double *)malloc((size_t)d * sizeof(double));
                if (!acc || !s || !qd) { fail = 1; free(acc); free(s); free(qd); continue; }
                for (int hh = 0; hh < G; ++hh)
                    for (int i = 0; i < Weff; ++i) {
                        const int h = g * G + hh;
                        const int pos = N - Weff + i;            /* position of this query in the prompt */
                        const uint16_t *q = q_win + ((((int64_t)l * B + b) * W + i) * Hq + h) * d;
                        for (int c = 0; c < d; ++c) qd[c] = bf16_to_double(q[c]);
                        double mx = -INFINITY;
                        for (int t = 0; t <= pos; ++t) {         /* causal: keys 0..pos are visible */
                            const uint16_t *k = k_cache + l * ls + (c0 + t) * ts + g * hs;
                            double dot = 0.0;
                            for (int c = 0; c < d; ++c) dot += qd[c] * bf16_to_double(k[c]);
                            s[t] = dot * inv_sqrt_d;
                            if (s[t] > mx) mx = s[t];
                        }
                        double sum = 0.0;
                        for (int t = 0; t <= pos; ++t) { s[t] = exp(s[t] - mx); sum += s[t]; }
                        for (int t = 0; t <= pos; ++t) acc[t] += s[t] / sum;
                    }
                for (int t = 0; t < N; ++t) imp[t] = (float)acc[t];
                free(acc); free(s); free(qd);
            }
    return fail;
}

/* Order-preserving image of a float's bit pattern: larger float <=> larger unsigned key.
 * (+0 > -0; +inf above every finite value; NaNs ordered by their bit patterns.) */
static uint32_t order_key(float x) {
    uint32_t u;
    memcpy(&u, &x, sizeof u);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

typedef struct { uint32_t key; int32_t t; } sgo_pair;

static int cmp_key_desc_index_asc(const void *a, const void *b) {
    const sgo_pair *x = (const sgo_pair *)a, *y = (const sgo_pair *)b;
    if (x->key != y->key) return x->key > y->key ? -1 : 1;
    return (x->t > y->t) - (x->t < y->t);
}

static int cmp_int_asc(const void *a, const void *b) {
    const int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/*
 * Per-head top-k KV index (Section 2.3: each row of the BH x k KV index holds the top-k entries
 * of one head of one request).  For (l, b, g) the k_b = cu_k[b+1]-cu_k[b] positions with the
 * largest importance are kept; equal values go to the lower position; the row is emitted in
 * ascending position order (entry order does not change attention, Section 4.2).
 *
 * importance float [L][Hkv][T];  sel_idx int32 [L][Hkv][K_tot], sequence-local positions.
 * Returns 2 if some k_b is outside [0, N_b].
 */
int sgo_select_topk(int L, int B, int Hkv, const int32_t *cu, const float *importance,
                    const int32_t *cu_k, int32_t *sel_idx) {
    const int64_t T = cu[B], K_tot = cu_k[B];
    for (int b = 0; b < B; ++b) {
        const int kb = cu_k[b + 1] - cu_k[b];
        if (kb < 0 || kb > cu[b + 1] - cu[b]) return 2;
    }
    int fail = 0;
#pragma omp parallel for collapse(3) schedule(dynamic, 1)
    for (int l = 0; l < L; ++l)
        for (int b = 0; b < B; ++b)
            for (int g = 0; g < Hkv; ++g) {
                const int N = cu[b + 1] - cu[b];
                const int kb = cu_k[b + 1] - cu_k[b];
                if (kb == 0) continue;
                const float *imp = importance + ((int64_t)l * Hkv + g) * T + cu[b];
                int32_t *out = sel_idx + ((int64_t)l * Hkv + g) * K_tot + cu_k[b];
                sgo_pair *p = (sgo_pair *)malloc((size_t)N * sizeof(sgo_pair));
                if (!p) { fail = 1; continue; }
                for (int t = 0; t < N; ++t) { p[t].key = order_key(imp[t]); p[t].t = t; }
                qsort(p, (size_t)N, sizeof(sgo_pair), cmp_key_desc_index_asc);
                for (int j = 0; j < kb; ++j) out[j] = p[j].t;
                qsort(out, (size_t)kb, sizeof(int32_t), cmp_int_asc);
                free(p);
            }
    return fail;
}

/*
 * Gather-pack of the selected K/V rows into a contiguous buffer (Section 4.2: the selected KV
 * has shape BH x k x d, a row being the k entries of one head; the prefill node picks the required
 * entries out of its own cache before sending them).
 *
 * packed_k/v bf16 [L][K_tot*Hkv][d]; row of (b, g, j) is cu_k[b]*Hkv + g*k_b + j.
 * Returns 3 if an index is outside its sequence.
 */
int sgo_pack_kv(int L, int B, int Hkv, int d, const int32_t *cu, const uint16_t *k_cache,
                const uint16_t *v_cache, int64_t ls, int64_t ts, int64_t hs, const int32_t *sel_idx,
                const int32_t *cu_k, uint16_t *packed_k, uint16_t *packed_v, const int32_t *sel_count) {
    /* sel_count (int32 [L][B][Hkv], may be NULL): only the first sel_count[l][b][g] entries of a row of the KV index
     * are selected (threshold selection); the remaining rows of the head's slot in the buffer are left as they are. */
    const int64_t K_tot = cu_k[B];
    int bad = 0;
    for (int l = 0; l < L; ++l)
        for (int b = 0; b < B; ++b)
            for (int g = 0; g < Hkv; ++g) {
                const int N = cu[b + 1] - cu[b];
                const int kb = cu_k[b + 1] - cu_k[b];
                int kbe = kb;
                if (sel_count) {
                    kbe = sel_count[((int64_t)l * B + b) * Hkv + g];
                    if (kbe < 0) kbe = 0;
                    if (kbe > kb) kbe = kb;
                }
                for (int j = 0; j < kbe; ++j) {
                    const int32_t t = sel_idx[((int64_t)l * Hkv + g) * K_tot + cu_k[b] + j];
                    if (t < 0 || t >= N) { bad = 3; continue; }
                    const int64_t src = l * ls + ((int64_t)cu[b] + t) * ts + g * hs;
                    const int64_t dst = (((int64_t)l * K_tot + cu_k[b]) * Hkv + (int64_t)g * kb + j) * d;
                    memcpy(packed_k + dst, k_cache + src, (size_t)d * sizeof(uint16_t));
                    memcpy(packed_v + dst, v_cache + src, (size_t)d * sizeof(uint16_t));
                }
            }
    return bad;
}

/*
 * Decode attention of one new query per (sequence, query head) over a two-source KV list
 * (Section 4.2, two-lane fetching: the entries of a head arrive partly as contiguous rows at
 * the start of its row of the selected KV, partly by gathering with a local index).  Since the
 * order of KV entries along the sequence axis does not change softmax(q K^T / sqrt(d)) V, the
 * result is plain attention over the concatenated list
 *     [packed rows 0..k_b-1 of (b, g)] ++ [local rows cu[b] + local_idx[g][cu_nloc[b] + j]],
 * computed here in one pass.  The list is a multiset: nothing is de-duplicated.
 *
 * q bf16 [B][Hq][d]; packed_k/v bf16 [K_tot*Hkv][d] (one layer, layout of sgo_pack_kv);
 * local_k/v bf16, element (token, g, c) at token*ts + g*hs + c; local_idx int32 [Hkv][NL_tot].
 * out float [B][Hq][d] (not rounded to bf16); lse float [B][Hq] = max + ln(sum).
 * An empty list gives out = 0 and lse = -inf.  Returns 3 on an out-of-range local index.
 * packed_count (int32 [B][Hkv], may be NULL): when the selection kept a different number of entries per KV head
 * (threshold selection), only the first packed_count[b][g] of the k_b packed rows of (b, g) are in the list.
 * local_skip (int32 [B][Hkv], may be NULL): the first local_skip[b][g] entries of the local-index row of (b, g) are
 * not in the list.  With Algorithm 1's reordered KV index as local_idx (remote entries first) and both arrays set
 * to the remote counts, the list is [remote rows, fetched and packed] ++ [local rows, by index]: two-lane fetching.
 */
int sgo_sparse_decode_attn(int B, int Hq, int Hkv, int d, const int32_t *cu, const uint16_t *q,
                           const uint16_t *packed_k, const uint16_t *packed_v, const int32_t *cu_k,
                           const uint16_t *local_k, const uint16_t *local_v, int64_t ts, int64_t hs,
                           const int32_t *local_idx, const int32_t *cu_nloc, double softmax_scale,
                           float *out, float *lse, const int32_t *packed_count, const int32_t *local_skip) {
    if (Hkv <= 0 || Hq % Hkv != 0) return 1;
    const int G = Hq / Hkv;
    const int64_t NL_tot = cu_nloc[B];
    const double scale = softmax_scale > 0.0 ? softmax_scale : 1.0 / sqrt((double)d);
    int bad = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < Hq; ++h) {
            const int g = h / G;
            const int N = cu[b + 1] - cu[b];
            const int kb = cu_k[b + 1] - cu_k[b];
            int kbe = kb;                                        /* packed rows actually in the list */
            if (packed_count) {
                kbe = packed_count[(int64_t)b * Hkv + g];
                if (kbe < 0) kbe = 0;
                if (kbe > kb) kbe = kb;
            }
            const int nl = cu_nloc[b + 1] - cu_nloc[b];
            int skip = 0;
            if (local_skip) {
                skip = local_skip[(int64_t)b * Hkv + g];
                if (skip < 0) skip = 0;
                if (skip > nl) skip = nl;
            }
            const int n = kbe + nl - skip;
            float *o = out + ((int64_t)b * Hq + h) * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0f;
            if (lse) lse[(int64_t)b * Hq + h] = -INFINITY;
            if (n == 0) continue;
            const uint16_t **kr = (const uint16_t **)malloc((size_t)n * sizeof(*kr));
            const uint16_t **vr = (const uint16_t **)malloc((size_t)n * sizeof(*vr));
            double *s = (double *)malloc((size_t)n * sizeof(double));
            double *acc = (double *)calloc((size_t)d, sizeof(double));
            int m = 0;
            for (int j = 0; j < kbe; ++j, ++m) {
                const int64_t row = ((int64_t)cu_k[b] * Hkv + (int64_t)g * kb + j) * d;
                kr[m] = packed_k + row;
                vr[m] = packed_v + row;
            }
            for (int j = skip; j < nl; ++j) {
                const int32_t t = local_idx[(int64_t)g * NL_tot + cu_nloc[b] + j];
                if (t < 0 || t >= N) { bad = 3; continue; }
                const int64_t off = ((int64_t)cu[b] + t) * ts + g * hs;
                kr[m] = local_k + off;
                vr[m] = local_v + off;
                ++m;
            }
            const uint16_t *qq = q + ((int64_t)b * Hq + h) * d;
            double mx = -INFINITY;
            for (int j = 0; j < m; ++j) {
                double dot = 0.0;
                for (int c = 0; c < d; ++c) dot += bf16_to_double(qq[c]) * bf16_to_double(kr[j][c]);
                s[j] = dot * scale;
                if (s[j] > mx) mx = s[j];
            }
            double sum = 0.0;
            for (int j = 0; j < m; ++j) { s[j] = exp(s[j] - mx); sum += s[j]; }
            for (int j = 0; j < m; ++j)
                for (int c = 0; c < d; ++c) acc[c] += s[j] * bf16_to_double(vr[j][c]);
            if (m > 0) {
                for (int c = 0; c < d; ++c) o[c] = (float)(acc[c] / sum);
                if (lse) lse[(int64_t)b * Hq + h] = (float)(mx + log(sum));
            }
            free(kr); free(vr); free(s); free(acc);
        }
    return bad;
}

/*
 * KV index splitting and reordering (Algorithm 1, Section 4.2), per row of the KV index.
 *
 * Definition used here: the KV mask holds one int8 per token, shared by all heads, that names the
 * token's class (2 = its entries are on the remote prefill node, 1 = locally available,
 * 0 = padding).  A row of the KV index is split by the class of each of its entries: the local list
 * is the row's entries of class 1, the remote list those of class 2, each in the row's own order.
 * With `reorder` the row itself is also returned as a stable partition by class, remote entries
 * first, then local, then padding (a stable descending sort by class), so that the remote entries
 * are contiguous at the start of the row.
 *
 * kv_index int32 [Hkv][K_tot] with prefix sums cu_k (sequence-local positions, row segment of
 * (b, g) at g*K_tot + cu_k[b]); kv_mask int8 [T] ragged by cu.
 * Outputs: reordered int32 [Hkv][K_tot] (the partitioned row, or a copy when reorder == 0);
 * local_index / remote_index int32 [Hkv][K_tot], each row segment filled from its start;
 * n_local / n_remote int32 [B][Hkv].  Entries with mask 0 are dropped from both lists.
 */
int sgo_split_index(int B, int Hkv, const int32_t *cu, const int32_t *cu_k, const int32_t *kv_index,
                    const int8_t *kv_mask, int reorder, int32_t *reordered, int32_t *local_index,
                    int32_t *remote_index, int32_t *n_local, int32_t *n_remote) {
    const int64_t K_tot = cu_k[B];
    int bad = 0;
    for (int b = 0; b < B; ++b)
        for (int g = 0; g < Hkv; ++g) {
            const int N = cu[b + 1] - cu[b];
            const int kb = cu_k[b + 1] - cu_k[b];
            const int64_t base = (int64_t)g * K_tot + cu_k[b];
            int8_t *mask = (int8_t *)malloc((size_t)(kb > 0 ? kb : 1));
            int32_t *row = (int32_t *)malloc((size_t)(kb > 0 ? kb : 1) * sizeof(int32_t));
            for (int j = 0; j < kb; ++j) {
                const int32_t t = kv_index[base + j];
                row[j] = t;
                if (t < 0 || t >= N) { bad = 3; mask[j] = 0; } else mask[j] = kv_mask[cu[b] + t];
            }
            if (reorder) {           /* stable descending sort of (mask, index) by mask: insertion sort */
                for (int j = 1; j < kb; ++j) {
                    const int8_t mj = mask[j];
                    const int32_t rj = row[j];
                    int i = j - 1;
                    while (i >= 0 && mask[i] < mj) { mask[i + 1] = mask[i]; row[i + 1] = row[i]; --i; }
                    mask[i + 1] = mj; row[i + 1] = rj;
                }
            }
            int nl = 0, nr = 0;
            for (int j = 0; j < kb; ++j) {
                reordered[base + j] = row[j];
                if (mask[j] == 1) local_index[base + nl++] = row[j];
                else if (mask[j] == 2) remote_index[base + nr++] = row[j];
            }
            n_local[b * Hkv + g] = nl;
            n_remote[b * Hkv + g] = nr;
            free(mask); free(row);
        }
    return bad;
}

/* ------------------------------------------------------------------------------------------------
 * Profile-based proactive selection (Section 4.1).
 *
 * Block of a token: every layer's cache is partitioned along the sequence into M blocks; token t of
 * a sequence of length N belongs to block floor(t * M / N), so block sizes differ by at most one.
 */
static int64_t block_of(int64_t t, int64_t N, int64_t M) { return t * M / N; }

/* S(e) of Eq. 1 (Section 4.1): how often a KV entry was selected over the profiled decode steps.
 * Adds one to counts[g][cu[b] + t] for every entry t of the KV index (one layer, one decode step).
 * kv_index int32 [Hkv][K_tot] with prefix sums cu_k; counts int32 [Hkv][T]. */
int sgo_profile_accumulate(int B, int Hkv, const int32_t *cu, const int32_t *cu_k, const int32_t *kv_index,
                           int32_t *counts) {
    const int64_t T = cu[B], K_tot = cu_k[B];
    int bad = 0;
    for (int g = 0; g < Hkv; ++g)
        for (int b = 0; b < B; ++b)
            for (int j = cu_k[b]; j < cu_k[b + 1]; ++j) {
                const int32_t t = kv_index[(int64_t)g * K_tot + j];
                if (t < 0 || t >= cu[b + 1] - cu[b]) { bad = 3; continue; }
                counts[(int64_t)g * T + cu[b] + t] += 1;
            }
    return bad;
}

/* Eq. 1: I[l][m] = +inf for l = 0, 1; otherwise the mean of S(e) over the entries of block B_{l,m}
 * (all tokens of the block, all KV heads, all profiled sequences).  An empty block gets 0.
 * counts int32 [L][Hkv][T]; importance float [L][M].  The mean is a double division rounded to float. */
int sgo_block_importance(int L, int B, int Hkv, int M, const int32_t *cu, const int32_t *counts, float *importance) {
    const int64_t T = cu[B];
    for (int l = 0; l < L; ++l)
        for (int m = 0; m < M; ++m) {
            if (l < 2) { importance[(int64_t)l * M + m] = INFINITY; continue; }
            int64_t sum = 0, entries = 0;
            for (int b = 0; b < B; ++b) {
                const int64_t N = cu[b + 1] - cu[b];
                for (int64_t t = 0; t < N; ++t) {
                    if (block_of(t, N, M) != m) continue;
                    entries += Hkv;
                    for (int g = 0; g < Hkv; ++g) sum += counts[((int64_t)l * Hkv + g) * T + cu[b] + t];
                }
            }
            importance[(int64_t)l * M + m] = entries ? (float)((double)sum / (double)entries) : 0.0f;
        }
    return 0;
}

/* Eq. 2: K_r = M (L-1) T_p / T_t, the number of blocks whose transfer overlaps the prefill of all but the first
 * transformer block; clipped to [2M, LM] so that the first two layers always go.  Rounded down. */
int64_t sgo_transfer_budget(int L, int M, double T_p, double T_t) {
    double k = (double)M * (double)(L - 1) * T_p / T_t;
    const double lo = 2.0 * M, hi = (double)L * M;
    if (!(k >= lo)) k = lo;          /* also catches NaN */
    if (k > hi) k = hi;
    if (L < 2) k = hi;
    return (int64_t)floor(k);
}

/* KV mask of one layer after the proactive transfer (Section 4.2: 1 = locally available, 2 = on the remote
 * prefill node): tokens of the blocks of layer l that are in the global top-K_r set are local, the rest remote.
 * selected int32 [K_r]: flat block ids l*M + m in ascending order.  mask int8 [T]. */
int sgo_proactive_mask(int B, int M, const int32_t *cu, int layer, const int32_t *selected, int K_r, int8_t *mask) {
    for (int b = 0; b < B; ++b) {
        const int64_t N = cu[b + 1] - cu[b];
        for (int64_t t = 0; t < N; ++t) {
            const int32_t id = (int32_t)((int64_t)layer * M + block_of(t, N, M));
            int8_t v = 2;
            for (int j = 0; j < K_r; ++j)
                if (selected[j] == id) { v = 1; break; }
            mask[cu[b] + t] = v;
        }
    }
    return 0;
}

/* Speculative transfer (Section 4.3): after the prefill stage has pushed the top-K_r blocks, every decoding
 * iteration delivers the next blocks in descending order of their Eq. 1 importance, at most a fixed
 * fraction (the speculative ratio) of ALL L*M blocks per iteration.  Number of blocks on the decode node after
 * `iteration` speculative transfers; the per-iteration quota is ratio * L * M rounded down, at least one block. */
int64_t sgo_speculative_delivered(int L, int M, int64_t K_r, double ratio, int iteration) {
    const int64_t total = (int64_t)L * M;
    int64_t quota = (int64_t)floor(ratio * (double)total);
    if (quota < 1) quota = 1;
    int64_t n = K_r + (int64_t)iteration * quota;
    if (n > total) n = total;
    if (n < 0) n = 0;
    return n;
}

/* Online proactive transfer of one layer (Section 4.1, "Online KV transfer"): the layer's cache is split into
 * M blocks; every block whose position is among the top-K_r (flat id layer*M + m in `selected`) is written,
 * all KV heads, K and V, to the same token positions of the decode-side cache; nothing else is written.
 * Caches of this layer: uint16 [T][Hkv][d] (dense).  selected int32 [K_r], any order.
 * kv_mask (int8 [T], may be NULL): "each time a KV block is pushed to the decoding node, the prefill node also
 * updates the corresponding values in the decoding-side KV mask" (Section 4.2): the tokens of a pushed block get
 * 1 (locally available); other entries keep their value. */
int sgo_push_blocks(int B, int Hkv, int d, int M, const int32_t *cu, int layer, const int32_t *selected, int K_r,
                    const uint16_t *src_k, const uint16_t *src_v, uint16_t *dst_k, uint16_t *dst_v, int8_t *kv_mask) {
    for (int b = 0; b < B; ++b) {
        const int64_t N = cu[b + 1] - cu[b];
        for (int m = 0; m < M; ++m) {
            const int32_t id = (int32_t)((int64_t)layer * M + m);
            int pushed = 0;
            for (int j = 0; j < K_r; ++j)
                if (selected[j] == id) { pushed = 1; break; }
            if (!pushed) continue;
            for (int64_t t = 0; t < N; ++t) {
                if (block_of(t, N, M) != m) continue;      /* E(B_{l,m}): the tokens of the block */
                const int64_t row = (cu[b] + t) * Hkv * (int64_t)d;
                for (int64_t e = 0; e < (int64_t)Hkv * d; ++e) {
                    dst_k[row + e] = src_k[row + e];
                    dst_v[row + e] = src_v[row + e];
                }
                if (kv_mask) kv_mask[cu[b] + t] = 1;
            }
        }
    }
    return 0;
}

/* Threshold selection (the selection rule of the KV selection algorithm the paper deploys, Section 5.1
 * "Parameters": an alpha value and a maximum KV selection ratio): per (layer, sequence, KV head) every token
 * whose score exceeds the row maximum minus alpha is selected, at most cap_b = cu_cap[b+1] - cu_cap[b] of them;
 * if more exceed the threshold, the cap_b largest are kept (ties to the lower index).
 * scores float [L][Hkv][T]; sel_idx int32 [L][Hkv][cap_tot]: the selected positions in ascending order, then -1;
 * sel_count int32 [L][B][Hkv].  NaN scores are never selected.  Returns 2 for a cap outside [0, N_b]. */
int sgo_select_threshold(int L, int B, int Hkv, const int32_t *cu, const float *scores, float alpha,
                         const int32_t *cu_cap, int32_t *sel_idx, int32_t *sel_count) {
    const int64_t T = cu[B], cap_tot = cu_cap[B];
    for (int b = 0; b < B; ++b) {
        const int cap = cu_cap[b + 1] - cu_cap[b];
        if (cap < 0 || cap > cu[b + 1] - cu[b]) return 2;
    }
    for (int l = 0; l < L; ++l)
        for (int b = 0; b < B; ++b)
            for (int g = 0; g < Hkv; ++g) {
                const int N = cu[b + 1] - cu[b];
                const int cap = cu_cap[b + 1] - cu_cap[b];
                const float *x = scores + ((int64_t)l * Hkv + g) * T + cu[b];
                int32_t *out = sel_idx + ((int64_t)l * Hkv + g) * cap_tot + cu_cap[b];
                int have_max = 0;
                float m = 0.0f;
                for (int t = 0; t < N; ++t)
                    if (x[t] == x[t] && (!have_max || x[t] > m)) { m = x[t]; have_max = 1; }
                const float thr = m - alpha;                         /* single precision, as the scores are */
                sgo_pair *p = (sgo_pair *)malloc((size_t)(N > 0 ? N : 1) * sizeof(sgo_pair));
                if (!p) return 1;
                int n = 0;
                if (have_max)
                    for (int t = 0; t < N; ++t)
                        if (x[t] > thr) { p[n].key = order_key(x[t]); p[n].t = t; ++n; }
                if (n > cap) {
                    qsort(p, (size_t)n, sizeof(sgo_pair), cmp_key_desc_index_asc);
                    n = cap;
                }
                for (int j = 0; j < n; ++j) out[j] = p[j].t;
                qsort(out, (size_t)n, sizeof(int32_t), cmp_int_asc);
                for (int j = n; j < cap; ++j) out[j] = -1;
                sel_count[((int64_t)l * B + b) * Hkv + g] = n;
                free(p);
            }
    return 0;
}
