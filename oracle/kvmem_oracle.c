/* KVMem hot path, CPU oracle.  TEST INFRASTRUCTURE, NOT PRODUCT.
 *
 * A plain, slow, loop-nest statement of what one recall step computes: Mean-K index,
 * query-conditioned block scores, selection under the active budget, execution-view
 * assembly and GQA attention over the view.  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it.  It shares no code with the CUDA library.
 *
 * Precision: bf16 inputs are widened exactly; every reduction accumulates in fp64
 * (closer to the real-number result than either implementation), with one exception
 * that is part of the contract: the Mean-K sum is fp32 in ascending token order followed
 * by a single round-to-nearest-even to bf16, because the stored index is a quantised
 * code and both sides must take that rounding decision in the same precision.
 *
 * Readings taken where the paper is silent:
 * candidate set C = every block of the session, reserved blocks included; the selector
 * alone applies sink/recent reservation; g(h) = h / (H/G); sum over query tokens, mean
 * over layers and heads; ties broken by lower block id; partial blocks never indexed.
 *
 * OpenMP pragmas parallelise independent outer iterations only; no blocking, fusion or
 * reordering inside a reduction.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef uint16_t bf16_t;

static inline float bf16_to_f32(bf16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static inline bf16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (bf16_t)((u >> 16) | 0x40u); /* NaN */
    u += 0x7fffu + ((u >> 16) & 1u);
    return (bf16_t)(u >> 16);
}

/* ---------------------------------------------------------------------------------------
 * Mean-K index (Eq. "mean_k_index", Sec. 4.3):  kbar[l][b][g] = (1/|b|) sum_{i in b} k[l][i][g].
 * K is token-major [n_blocks*B][L][G][d]; idx is [L][G][idx_stride][d], written at rows
 * [b_first, b_first + n_blocks).  Only whole blocks exist, so |b| = B.
 */
void kvo_mean_k_index(const bf16_t* K, int64_t n_blocks, int B, int L, int G, int d,
                      bf16_t* idx, int64_t idx_stride, int64_t b_first) {
    const float inv = 1.0f / (float)B;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t b = 0; b < n_blocks; ++b)
        for (int l = 0; l < L; ++l)
            for (int g = 0; g < G; ++g)
                for (int c = 0; c < d; ++c) {
                    float acc = 0.0f;
                    for (int t = 0; t < B; ++t)
                        acc += bf16_to_f32(K[(((b * B + t) * L + l) * G + g) * (int64_t)d + c]);
                    float mean = acc * inv;
                    idx[((l * (int64_t)G + g) * idx_stride + b_first + b) * d + c] = f32_to_bf16_rne(mean);
                }
}

/* ---------------------------------------------------------------------------------------
 * Block relevance (Eq. "kvmem-block-score", Sec. 4.3):
 *   R_b = sum_m mean_{l,h} softmax_{b' in C}( q[l][m][h] . kbar[l][b'][g(h)] / sqrt(d) )_b
 * q is [M][L][H][d]; idx is [L][G][idx_stride][d] of which the first NB rows are the
 * candidate set C.  R is [NB].  R_g (may be NULL) is [G][NB]: the same sum restricted to
 * the query heads of KV head g and averaged over them and over layers, so that
 * R_b = (1/G) sum_g R_g[g][b].
 * Returns 0, or -1 if the logit buffer cannot be allocated.
 */
int kvo_block_scores(const bf16_t* q, const bf16_t* idx, int64_t NB, int64_t idx_stride,
                     int M, int L, int H, int G, int d, float* R, float* R_g) {
    const int r = H / G;
    const int64_t rows = (int64_t)L * M * H;
    double* s = (double*)malloc(sizeof(double) * (size_t)rows * (size_t)NB);
    double* mx = (double*)malloc(sizeof(double) * (size_t)rows);
    double* Z = (double*)malloc(sizeof(double) * (size_t)rows);
    if (!s || !mx || !Z) { free(s); free(mx); free(Z); return -1; }
    const double inv_sqrt_d = 1.0 / sqrt((double)d);

    /* scaled dot products, then the softmax statistics of each fixed (l, m, h) */
#pragma omp parallel for schedule(static)
    for (int64_t row = 0; row < rows; ++row) {
        const int h = (int)(row % H);
        const int m = (int)((row / H) % M);
        const int l = (int)(row / ((int64_t)H * M));
        const int g = h / r;
        const bf16_t* qv = q + (((int64_t)m * L + l) * H + h) * d;
        double* srow = s + row * NB;
        double best = -INFINITY;
        for (int64_t b = 0; b < NB; ++b) {
            const bf16_t* kv = idx + ((l * (int64_t)G + g) * idx_stride + b) * d;
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += (double)bf16_to_f32(qv[c]) * (double)bf16_to_f32(kv[c]);
            srow[b] = acc * inv_sqrt_d;
            if (srow[b] > best) best = srow[b];
        }
        double sum = 0.0;
        for (int64_t b = 0; b < NB; ++b) sum += exp(srow[b] - best);
        mx[row] = best;
        Z[row] = sum;
    }

    /* sum over query tokens, mean over (layer, head) pairs */
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < NB; ++b) {
        double total = 0.0;
        for (int g = 0; g < G; ++g) {
            double part = 0.0;
            for (int l = 0; l < L; ++l)
                for (int m = 0; m < M; ++m)
                    for (int h = g * r; h < (g + 1) * r; ++h) {
                        const int64_t row = ((int64_t)l * M + m) * H + h;
                        part += exp(s[row * NB + b] - mx[row]) / Z[row];
                    }
            if (R_g) R_g[(int64_t)g * NB + b] = (float)(part / ((double)L * r));
            total += part;
        }
        R[b] = (float)(total / ((double)L * H));
    }
    free(s); free(mx); free(Z);
    return 0;
}

/* ---------------------------------------------------------------------------------------
 * Budget (Eq. "active_budget" and Eq. "active_capacity", Sec. 3.1):
 *   N(Q) + B * |R| <= B_a  =>  k = min(budget_blocks, floor((B_a - N(Q)) / B), NB), never below 0.
 */
int64_t kvo_budget_blocks(int64_t NB, int B, int64_t budget_blocks, int64_t max_view_tokens,
                          int64_t mandatory_tokens) {
    int64_t room = max_view_tokens - mandatory_tokens;
    int64_t k = room > 0 ? room / B : 0;
    if (budget_blocks < k) k = budget_blocks;
    if (NB < k) k = NB;
    if (k < 0) k = 0;
    return k;
}

typedef struct { float score; int32_t id; } kvo_cand_t;

static int kvo_cand_cmp(const void* a, const void* b) {
    const kvo_cand_t* x = (const kvo_cand_t*)a;
    const kvo_cand_t* y = (const kvo_cand_t*)b;
    if (x->score > y->score) return -1;
    if (x->score < y->score) return 1;
    return (x->id > y->id) - (x->id < y->id);           /* equal score: lower id first */
}

static int kvo_i32_cmp(const void* a, const void* b) {
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
    return (x > y) - (x < y);
}

/* ---------------------------------------------------------------------------------------
 * Selector (Sec. 4.3, last paragraph of "Query-Conditioned Block Scoring"; Sec. 5.2):
 * reserve the sink (oldest) and recent (newest) blocks, fill the rest of the budget with
 * the largest R_b, restore chronological order.  Writes k ascending ids; returns k.
 */
int64_t kvo_select(const float* R, int64_t NB, int B, int64_t budget_blocks, int64_t max_view_tokens,
                   int64_t mandatory_tokens, int64_t n_sink, int64_t n_recent, int32_t* sel) {
    const int64_t k = kvo_budget_blocks(NB, B, budget_blocks, max_view_tokens, mandatory_tokens);
    if (k == 0) return 0;
    char* taken = (char*)calloc((size_t)NB, 1);
    kvo_cand_t* cand = (kvo_cand_t*)malloc(sizeof(kvo_cand_t) * (size_t)NB);
    int64_t n = 0;
    if (n_sink < 0) n_sink = 0;
    if (n_recent < 0) n_recent = 0;
    for (int64_t b = 0; b < NB && b < n_sink && n < k; ++b)            /* sinks, oldest first   */
        if (!taken[b]) { taken[b] = 1; sel[n++] = (int32_t)b; }
    for (int64_t j = 0; j < n_recent && j < NB && n < k; ++j) {         /* recents, newest first */
        int64_t b = NB - 1 - j;
        if (!taken[b]) { taken[b] = 1; sel[n++] = (int32_t)b; }
    }
    int64_t nc = 0;
    for (int64_t b = 0; b < NB; ++b)
        if (!taken[b]) { cand[nc].score = R[b]; cand[nc].id = (int32_t)b; ++nc; }
    qsort(cand, (size_t)nc, sizeof(kvo_cand_t), kvo_cand_cmp);          /* total order: no ties left */
    for (int64_t i = 0; i < nc && n < k; ++i) sel[n++] = cand[i].id;
    qsort(sel, (size_t)n, sizeof(int32_t), kvo_i32_cmp);                /* chronological order   */
    free(taken); free(cand);
    return n;
}

/* ---------------------------------------------------------------------------------------
 * Repository: physical pages hold B tokens each, token-major inside the page
 * ([n_pages][B][L][G][d]); logical block b of a session lives in page table[b].
 */
void kvo_place_blocks(const bf16_t* K, const bf16_t* V, int64_t n_blocks, int B, int L, int G, int d,
                      const int32_t* table, bf16_t* pagesK, bf16_t* pagesV) {
    const size_t page = (size_t)B * L * G * d;
    for (int64_t b = 0; b < n_blocks; ++b) {
        memcpy(pagesK + (size_t)table[b] * page, K + (size_t)b * page, page * sizeof(bf16_t));
        memcpy(pagesV + (size_t)table[b] * page, V + (size_t)b * page, page * sizeof(bf16_t));
    }
}

/* ---------------------------------------------------------------------------------------
 * Execution view (Sec. 4.4, "execution view"; Sec. 5.2): the selected blocks, in
 * chronological order, at contiguous compact positions: view token j*B + t is token t of
 * block sel[j], read through the block table.  View layout [L][G][cap_tokens][d].
 * K is copied unchanged (keys are position-independent on this path).
 */
void kvo_gather(const bf16_t* pagesK, const bf16_t* pagesV, const int32_t* table,
                const int32_t* sel, int64_t n_sel, int B, int L, int G, int d,
                bf16_t* viewK, bf16_t* viewV, int64_t cap_tokens) {
    const size_t page = (size_t)B * L * G * d;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n_sel; ++j) {
        const size_t src = (size_t)table[sel[j]] * page;
        for (int t = 0; t < B; ++t)
            for (int l = 0; l < L; ++l)
                for (int g = 0; g < G; ++g) {
                    const size_t s = src + (((size_t)t * L + l) * G + g) * d;
                    const size_t o = (((size_t)l * G + g) * cap_tokens + (size_t)j * B + t) * d;
                    memcpy(viewK + o, pagesK + s, (size_t)d * sizeof(bf16_t));
                    memcpy(viewV + o, pagesV + s, (size_t)d * sizeof(bf16_t));
                }
    }
}

/* ---------------------------------------------------------------------------------------
 * GQA attention over the first T view tokens, no mask (every query token of the step sees
 * the whole recalled history):  o = softmax(q K^T * scale) V,  lse = ln sum_t exp(s_t).
 * q [M][L][H][d]; view [L][G][cap_tokens][d]; out [M][L][H][d] fp32; lse [M][L][H] fp32.
 * T = 0 gives o = 0 and lse = -inf.
 */
void kvo_attend(const bf16_t* q, const bf16_t* viewK, const bf16_t* viewV, int64_t T, int64_t cap_tokens,
                int M, int L, int H, int G, int d, double scale, float* out, float* lse) {
    const int r = H / G;
    const int64_t rows = (int64_t)M * L * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t row = 0; row < rows; ++row) {
        const int h = (int)(row % H);
        const int l = (int)((row / H) % L);
        const int g = h / r;
        const bf16_t* qv = q + row * d;
        const bf16_t* Kg = viewK + ((size_t)l * G + g) * (size_t)cap_tokens * d;
        const bf16_t* Vg = viewV + ((size_t)l * G + g) * (size_t)cap_tokens * d;
        double* s = (double*)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1));
        double* o = (double*)calloc((size_t)d, sizeof(double));
        double best = -INFINITY;
        for (int64_t t = 0; t < T; ++t) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c)
                acc += (double)bf16_to_f32(qv[c]) * (double)bf16_to_f32(Kg[(size_t)t * d + c]);
            s[t] = acc * scale;
            if (s[t] > best) best = s[t];
        }
        double sum = 0.0;
        for (int64_t t = 0; t < T; ++t) sum += exp(s[t] - best);
        for (int64_t t = 0; t < T; ++t) {
            const double p = exp(s[t] - best) / sum;
            for (int c = 0; c < d; ++c) o[c] += p * (double)bf16_to_f32(Vg[(size_t)t * d + c]);
        }
        for (int c = 0; c < d; ++c) out[row * d + c] = (float)o[c];
        lse[row] = T > 0 ? (float)(best + log(sum)) : -INFINITY;
        free(s); free(o);
    }
}

/* Threads the parallel loops above will use (reported next to the timed baseline). */
int kvo_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}

/* =======================================================================================
 * Position-consistent materialisation (Sec. 4.3 "Mean-K Retrieval-Index Construction":
 * positional encoding is removed before indexing and from the query; Sec. 4.4: RoPE is
 * applied to raw K at the block's assigned compact position, V is copied unchanged, with
 * precomputed sine/cosine tables).
 *
 * Readings (the paper names RoPE but prints no formula): rotate-half pairing (i, i + d/2),
 * frequency of pair i = theta^(-2i/d), angle = position * frequency.  The table holds
 * cos and sin of the fp64 angle rounded once to fp32.  A rotated bf16 element is a
 * quantised code, so its arithmetic is fixed: four fp32 products and two fp32 sums (no fused
 * multiply-add), one round-to-nearest-even to bf16; the CUDA kernels do the same.
 */

/* tab[p][i] = (cos, sin) of p * theta^(-2i/d) as fp32 pairs; tab is [n_pos][d/2][2] */
void kvo_rope_table(int64_t n_pos, int d, double theta, float* tab) {
    const int half = d / 2;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < n_pos; ++p)
        for (int i = 0; i < half; ++i) {
            const double freq = pow(theta, -2.0 * (double)i / (double)d);
            const double ang = (double)p * freq;
            tab[(p * half + i) * 2 + 0] = (float)cos(ang);
            tab[(p * half + i) * 2 + 1] = (float)sin(ang);
        }
}

/* one vector of d elements at position p; inverse != 0 rotates by -p (removes the encoding) */
static void kvo_rotate_vec(const bf16_t* x, bf16_t* y, int d, const float* tab_row, int inverse) {
    const int half = d / 2;
    for (int i = 0; i < half; ++i) {
        const float a = bf16_to_f32(x[i]), b = bf16_to_f32(x[i + half]);
        const float c = tab_row[2 * i], s = inverse ? -tab_row[2 * i + 1] : tab_row[2 * i + 1];
        const float ac = a * c, bs = b * s, bc = b * c, as = a * s;
        const float lo = ac - bs, hi = bc + as;
        y[i] = f32_to_bf16_rne(lo);
        y[i + half] = f32_to_bf16_rne(hi);
    }
}

/* x, y: [n_rows][n_vec][d] bf16; every vector of row r is rotated by pos[r] (or by -pos[r]).
 * Returns -1 if a position is outside the table. */
int kvo_rope_rotate(const bf16_t* x, bf16_t* y, int64_t n_rows, int n_vec, int d, const int32_t* pos,
                    const float* tab, int64_t n_pos, int inverse) {
    for (int64_t r = 0; r < n_rows; ++r)
        if (pos[r] < 0 || pos[r] >= n_pos) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n_rows; ++r)
        for (int v = 0; v < n_vec; ++v)
            kvo_rotate_vec(x + (r * n_vec + v) * d, y + (r * n_vec + v) * d, d, tab + (size_t)pos[r] * (d / 2) * 2, inverse);
    return 0;
}

/* Execution view with position-consistent keys: as kvo_gather, but the raw key of view token
 * j*B + t is rotated to compact position first_pos + j*B + t; values are copied unchanged.
 * in_block != 0: the pages hold keys that already carry the rotation of their offset t inside
 * their block (a position-independent encoding too: t never changes); the view key is then the
 * stored key rotated by the block's compact position first_pos + j*B alone, which is the same
 * rotation R(first_pos + j*B + t) of the raw key up to the rounding of the stored key. */
int kvo_gather_rope(const bf16_t* pagesK, const bf16_t* pagesV, const int32_t* table, const int32_t* sel,
                    int64_t n_sel, int B, int L, int G, int d, bf16_t* viewK, bf16_t* viewV, int64_t cap_tokens,
                    int64_t first_pos, const float* tab, int64_t n_pos, int in_block) {
    if (first_pos < 0 || first_pos + n_sel * B > n_pos) return -1;
    const size_t page = (size_t)B * L * G * d;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n_sel; ++j) {
        const size_t src = (size_t)table[sel[j]] * page;
        for (int t = 0; t < B; ++t)
            for (int l = 0; l < L; ++l)
                for (int g = 0; g < G; ++g) {
                    const size_t s = src + (((size_t)t * L + l) * G + g) * d;
                    const size_t o = (((size_t)l * G + g) * cap_tokens + (size_t)j * B + t) * d;
                    kvo_rotate_vec(pagesK + s, viewK + o, d, tab + (size_t)(first_pos + j * B + (in_block ? 0 : t)) * (d / 2) * 2, 0);
                    memcpy(viewV + o, pagesV + s, (size_t)d * sizeof(bf16_t));
                }
    }
    return 0;
}

/* =======================================================================================
 * Working-set delta (Eq. "kvmem-working-set-delta", Sec. 4.4): with W_prev and W_next the block
 * sets of two consecutive steps,
 *     R = W_next n W_prev (retained),  L = W_next \ W_prev (incoming),  E = W_prev \ W_next (outgoing).
 * Inputs are the chronological (ascending) id lists; a block's slot is its index in its list, i.e. its
 * compact position divided by B.  Outputs, all in ascending id order:
 *   retained [nR][3] = (id, slot in prev, slot in next); incoming [nL][2] = (id, slot in next);
 *   outgoing [nE] = id.  counts = (nR, nL, nE).
 */
void kvo_working_set_delta(const int32_t* prev, int64_t n_prev, const int32_t* next, int64_t n_next,
                           int32_t* retained, int32_t* incoming, int32_t* outgoing, int32_t* counts) {
    int64_t nR = 0, nL = 0, nE = 0;
    for (int64_t j = 0; j < n_next; ++j) {
        int64_t found = -1;
        for (int64_t i = 0; i < n_prev; ++i)
            if (prev[i] == next[j]) { found = i; break; }
        if (found >= 0) {
            retained[3 * nR] = next[j]; retained[3 * nR + 1] = (int32_t)found; retained[3 * nR + 2] = (int32_t)j; ++nR;
        } else {
            incoming[2 * nL] = next[j]; incoming[2 * nL + 1] = (int32_t)j; ++nL;
        }
    }
    for (int64_t i = 0; i < n_prev; ++i) {
        int found = 0;
        for (int64_t j = 0; j < n_next; ++j)
            if (next[j] == prev[i]) { found = 1; break; }
        if (!found) outgoing[nE++] = prev[i];
    }
    counts[0] = (int32_t)nR; counts[1] = (int32_t)nL; counts[2] = (int32_t)nE;
}

/* =======================================================================================
 * Execution cache with working-set reuse and bounded delta re-RoPE (Sec. 4.4, "Retrieval-Aware
 * Hierarchical Reuse" and the paragraph on the two views).
 *
 * The cache is `cap` slots (the paper's active GPU pages); a slot holds one block: K encoded for the
 * block's current compact position and an unchanged copy of V.  State per slot: slot_block (block id,
 * -1 = empty), slot_pos (compact block index the keys are encoded for), slot_cnt (delta re-RoPE
 * operations since the keys were last built from raw K).  One update takes the cache from the
 * previous working set to `sel` (ascending ids, n_sel <= cap), in the paper's order:
 *   1. delta (Eq. "kvmem-working-set-delta"): a resident block that is selected again is retained
 *      and keeps its slot; every other slot is reclaimed;
 *   2. incoming blocks, in ascending id order, take the free slots in ascending slot order; their
 *      keys are built from raw K with RoPE at the new compact position, their values are copied;
 *   3. a retained block whose compact position changed is re-encoded: by a delta rotation of its
 *      current keys by (new - old) positions while slot_cnt < max_delta (slot_cnt += 1), otherwise
 *      rebuilt from raw K at the new position (slot_cnt = 0).  A retained block that did not move is
 *      left alone.
 * view_slots[j] = slot of the j-th selected block (the execution view's page table).
 * stats = (retained and unmoved, delta re-RoPEd, rebuilt, incoming).
 * Readings: the slot policy (lowest free slot, ascending ids) and the counter semantics (a limit on
 * operations between reconstructions, reset by a reconstruction) are ours; the paper fixes neither.
 * cacheK / cacheV: [cap][B][L][G][d] (token-major, like the repository pages of this file).
 * in_block: as in kvo_gather_rope (keys stored with the rotation of their in-block offset; loads and rebuilds
 * rotate by the block's position alone).  d <= 1024.  Returns -1 if n_sel > cap or positions leave the table.
 */
int kvo_view_cache_update(const bf16_t* pagesK, const bf16_t* pagesV, const int32_t* table, const int32_t* sel,
                          int64_t n_sel, int B, int L, int G, int d, int64_t cap, int64_t max_delta,
                          int64_t first_pos, const float* tab, int64_t n_pos, bf16_t* cacheK, bf16_t* cacheV,
                          int32_t* slot_block, int32_t* slot_pos, int32_t* slot_cnt, int32_t* view_slots,
                          int32_t* stats, int in_block) {
    if (n_sel > cap || first_pos < 0 || first_pos + n_sel * B > n_pos) return -1;
    const size_t page = (size_t)B * L * G * d;
    const int n_vec = L * G;
    stats[0] = stats[1] = stats[2] = stats[3] = 0;
    for (int64_t j = 0; j < n_sel; ++j) view_slots[j] = -1;
    /* 1. retained blocks keep their slot, all other slots are reclaimed */
    for (int64_t s = 0; s < cap; ++s) {
        int64_t found = -1;
        if (slot_block[s] >= 0)
            for (int64_t j = 0; j < n_sel; ++j)
                if (sel[j] == slot_block[s]) { found = j; break; }
        if (found >= 0) view_slots[found] = (int32_t)s;
        else slot_block[s] = -1;
    }
    /* 2. incoming blocks take the lowest free slots */
    int64_t next_free = 0;
    for (int64_t j = 0; j < n_sel; ++j) {
        if (view_slots[j] >= 0) continue;
        while (slot_block[next_free] >= 0) ++next_free;
        const int64_t s = next_free;
        const size_t src = (size_t)table[sel[j]] * page, dst = (size_t)s * page;
        for (int t = 0; t < B; ++t)
            for (int v = 0; v < n_vec; ++v) {
                const size_t o = ((size_t)t * n_vec + v) * d;
                kvo_rotate_vec(pagesK + src + o, cacheK + dst + o, d, tab + (size_t)(first_pos + j * B + (in_block ? 0 : t)) * (d / 2) * 2, 0);
            }
        memcpy(cacheV + dst, pagesV + src, page * sizeof(bf16_t));
        slot_block[s] = sel[j]; slot_pos[s] = (int32_t)j; slot_cnt[s] = 0;
        view_slots[j] = (int32_t)s;
        stats[3] += 1;
    }
    /* 3. retained blocks that moved */
    for (int64_t j = 0; j < n_sel; ++j) {
        const int64_t s = view_slots[j];
        if (slot_pos[s] == j) continue;                            /* unmoved, or loaded in step 2 */
        const size_t dst = (size_t)s * page;
        if (slot_cnt[s] < max_delta) {
            const int64_t delta = (j - slot_pos[s]) * B;           /* positions; the same for every token of the block */
            const int64_t mag = delta < 0 ? -delta : delta;
            for (int t = 0; t < B; ++t)
                for (int v = 0; v < n_vec; ++v) {
                    const size_t o = ((size_t)t * n_vec + v) * d;
                    bf16_t tmp[1024];
                    memcpy(tmp, cacheK + dst + o, (size_t)d * sizeof(bf16_t));
                    kvo_rotate_vec(tmp, cacheK + dst + o, d, tab + (size_t)mag * (d / 2) * 2, delta < 0);
                }
            slot_cnt[s] += 1;
            stats[1] += 1;
        } else {
            const size_t src = (size_t)table[sel[j]] * page;
            for (int t = 0; t < B; ++t)
                for (int v = 0; v < n_vec; ++v) {
                    const size_t o = ((size_t)t * n_vec + v) * d;
                    kvo_rotate_vec(pagesK + src + o, cacheK + dst + o, d, tab + (size_t)(first_pos + j * B + (in_block ? 0 : t)) * (d / 2) * 2, 0);
                }
            slot_cnt[s] = 0;
            stats[2] += 1;
        }
        slot_pos[s] = (int32_t)j;
    }
    stats[0] = (int32_t)n_sel - stats[1] - stats[2] - stats[3];
    return 0;
}

/* The execution view as attention sees it: slot view_slots[j] supplies view tokens [j*B, (j+1)*B).
 * viewK / viewV: [L][G][cap_tokens][d]. */
void kvo_view_cache_view(const bf16_t* cacheK, const bf16_t* cacheV, const int32_t* view_slots, int64_t n_sel,
                         int B, int L, int G, int d, bf16_t* viewK, bf16_t* viewV, int64_t cap_tokens) {
    const size_t page = (size_t)B * L * G * d;
    for (int64_t j = 0; j < n_sel; ++j)
        for (int t = 0; t < B; ++t)
            for (int l = 0; l < L; ++l)
                for (int g = 0; g < G; ++g) {
                    const size_t s = (size_t)view_slots[j] * page + (((size_t)t * L + l) * G + g) * d;
                    const size_t o = (((size_t)l * G + g) * cap_tokens + (size_t)j * B + t) * d;
                    memcpy(viewK + o, cacheK + s, (size_t)d * sizeof(bf16_t));
                    memcpy(viewV + o, cacheV + s, (size_t)d * sizeof(bf16_t));
                }
}

/* =======================================================================================
 * FP8 execution view (the paper's evaluation keeps the KV cache in FP8, Sec. 6.1).
 *
 * Format: E4M3 in its finite-only form (1 sign, 4 exponent, 3 mantissa bits, bias 7, no
 * infinities, largest finite value 448, codes 0x7f / 0xff are NaN).  A stored element is the
 * code of x * inv_scale (one fp32 product), rounded to nearest with ties to the even code and
 * saturated to +-448: a quantised code, so both implementations take that decision on the same
 * fp32 value.  Readings: one static scale per tensor (keys, values), given by the caller, as FP8
 * KV caches are commonly run; the paper states no scaling rule.
 * View layout: keys [L][G][cap_tokens][d] bytes; values transposed inside every 64-token tile,
 * [L][G][cap_tokens/64][d][64] bytes (so that both operands of the attention contractions are read
 * along their contraction index).
 */
static float e4m3_to_f32(uint8_t c) {
    const int e = (c >> 3) & 15, m = c & 7;
    float v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexpf((float)m, -9);                       /* subnormal: m * 2^-9 */
    else v = ldexpf(1.0f + (float)m / 8.0f, e - 7);
    return (c & 0x80) ? -v : v;
}

static uint8_t f32_to_e4m3(float x) {
    const uint8_t sign = signbit(x) ? 0x80 : 0x00;
    const float a = fabsf(x);
    if (isnan(x)) return 0x7f;
    if (a >= 448.0f) return sign | 0x7e;                        /* saturate */
    /* nearest of the 127 non-negative finite values; on a tie the even code */
    int lo = 0, hi = 0x7e;                                      /* value(lo) <= a <= value(hi) */
    while (hi - lo > 1) {
        const int mid = (lo + hi) / 2;
        if (e4m3_to_f32((uint8_t)mid) <= a) lo = mid; else hi = mid;
    }
    const float vl = e4m3_to_f32((uint8_t)lo), vh = e4m3_to_f32((uint8_t)hi);
    const double dl = (double)a - (double)vl, dh = (double)vh - (double)a;
    int code;
    if (dl < dh) code = lo;
    else if (dh < dl) code = hi;
    else code = (lo & 1) ? hi : lo;
    return sign | (uint8_t)code;
}

void kvo_quantize_e4m3(const bf16_t* x, uint8_t* y, int64_t n, float inv_scale) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) y[i] = f32_to_e4m3(bf16_to_f32(x[i]) * inv_scale);
}

void kvo_dequantize_e4m3(const uint8_t* y, float* x, int64_t n, float scale) {
    for (int64_t i = 0; i < n; ++i) x[i] = e4m3_to_f32(y[i]) * scale;
}

/* as kvo_gather, quantising on the way; cap_tokens is a multiple of 64 */
void kvo_gather_fp8(const bf16_t* pagesK, const bf16_t* pagesV, const int32_t* table, const int32_t* sel,
                    int64_t n_sel, int B, int L, int G, int d, float k_inv_scale, float v_inv_scale,
                    uint8_t* viewK8, uint8_t* viewV8T, int64_t cap_tokens) {
    const size_t page = (size_t)B * L * G * d;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n_sel; ++j) {
        const size_t src = (size_t)table[sel[j]] * page;
        for (int t = 0; t < B; ++t) {
            const int64_t tok = j * B + t, tile = tok / 64, tt = tok % 64;
            for (int l = 0; l < L; ++l)
                for (int g = 0; g < G; ++g) {
                    const size_t s = src + (((size_t)t * L + l) * G + g) * d;
                    const size_t head = (size_t)l * G + g;
                    for (int c = 0; c < d; ++c) {
                        viewK8[(head * cap_tokens + (size_t)tok) * d + c] = f32_to_e4m3(bf16_to_f32(pagesK[s + c]) * k_inv_scale);
                        viewV8T[((head * (size_t)(cap_tokens / 64) + (size_t)tile) * d + c) * 64 + (size_t)tt] =
                            f32_to_e4m3(bf16_to_f32(pagesV[s + c]) * v_inv_scale);
                    }
                }
        }
    }
}

/* kvo_attend over an FP8 view: keys are code * k_scale, values code * v_scale */
void kvo_attend_fp8(const bf16_t* q, const uint8_t* viewK8, const uint8_t* viewV8T, int64_t T, int64_t cap_tokens,
                    int M, int L, int H, int G, int d, double scale, double k_scale, double v_scale, float* out, float* lse) {
    const int r = H / G;
    const int64_t rows = (int64_t)M * L * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t row = 0; row < rows; ++row) {
        const int h = (int)(row % H);
        const int l = (int)((row / H) % L);
        const size_t head = (size_t)l * G + (size_t)(h / r);
        const bf16_t* qv = q + row * d;
        double* s = (double*)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1));
        double* o = (double*)calloc((size_t)d, sizeof(double));
        double best = -INFINITY;
        for (int64_t t = 0; t < T; ++t) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c)
                acc += (double)bf16_to_f32(qv[c]) * ((double)e4m3_to_f32(viewK8[(head * cap_tokens + (size_t)t) * d + c]) * k_scale);
            s[t] = acc * scale;
            if (s[t] > best) best = s[t];
        }
        double sum = 0.0;
        for (int64_t t = 0; t < T; ++t) sum += exp(s[t] - best);
        for (int64_t t = 0; t < T; ++t) {
            const double p = exp(s[t] - best) / sum;
            const size_t vbase = (head * (size_t)(cap_tokens / 64) + (size_t)(t / 64)) * d;
            for (int c = 0; c < d; ++c) o[c] += p * ((double)e4m3_to_f32(viewV8T[(vbase + c) * 64 + (size_t)(t % 64)]) * v_scale);
        }
        for (int c = 0; c < d; ++c) out[row * d + c] = (float)o[c];
        lse[row] = T > 0 ? (float)(best + log(sum)) : -INFINITY;
        free(s); free(o);
    }
}

/* =======================================================================================
 * Attention with position-consistent keys when the pages hold in-block-rotated keys k' = R(t) k
 * (kvo_gather_rope with in_block): the logit q . R(p0 + t) k equals (R(-p0) q) . k', so the
 * query is rotated back by the compact position p0 = first_pos + tile*B of each tile of B tokens
 * instead of the keys forward.  The rotated query is a bf16 vector (the arithmetic of
 * kvo_rope_rotate, inverse), which is what the tensor cores are fed; everything after it is
 * kvo_attend.  viewK: plain gather (kvo_gather) of the stored keys k'.  B = tokens per tile.
 */
void kvo_attend_qrot(const bf16_t* q, const bf16_t* viewK, const bf16_t* viewV, int64_t T, int64_t cap_tokens,
                     int M, int L, int H, int G, int d, int B, int64_t first_pos, const float* tab, double scale,
                     float* out, float* lse) {
    const int r = H / G;
    const int64_t rows = (int64_t)M * L * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t row = 0; row < rows; ++row) {
        const int h = (int)(row % H);
        const int l = (int)((row / H) % L);
        const int g = h / r;
        const bf16_t* qv = q + row * d;
        const bf16_t* Kg = viewK + ((size_t)l * G + g) * (size_t)cap_tokens * d;
        const bf16_t* Vg = viewV + ((size_t)l * G + g) * (size_t)cap_tokens * d;
        double* s = (double*)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1));
        double* o = (double*)calloc((size_t)d, sizeof(double));
        bf16_t qr[1024];
        double best = -INFINITY;
        for (int64_t t = 0; t < T; ++t) {
            if (t % B == 0) kvo_rotate_vec(qv, qr, d, tab + (size_t)(first_pos + t) * (d / 2) * 2, 1);
            double acc = 0.0;
            for (int c = 0; c < d; ++c)
                acc += (double)bf16_to_f32(qr[c]) * (double)bf16_to_f32(Kg[(size_t)t * d + c]);
            s[t] = acc * scale;
            if (s[t] > best) best = s[t];
        }
        double sum = 0.0;
        for (int64_t t = 0; t < T; ++t) sum += exp(s[t] - best);
        for (int64_t t = 0; t < T; ++t) {
            const double p = exp(s[t] - best) / sum;
            for (int c = 0; c < d; ++c) o[c] += p * (double)bf16_to_f32(Vg[(size_t)t * d + c]);
        }
        for (int c = 0; c < d; ++c) out[row * d + c] = (float)o[c];
        lse[row] = T > 0 ? (float)(best + log(sum)) : -INFINITY;
        free(s); free(o);
    }
}
