/*
 * DASC oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 CPU statement of what the DASC hot path computes
 * (plan, pack, restore + zero-fill, suffix refresh), written from the paper's
 * definitions.  It shares no code with the CUDA library and must never be
 * imported, linked or executed by the product path: only the tests, the smoke
 * check and the benchmark's CPU-baseline leg may use it.
 *
 * Orientation.  The paper writes the recurrent state as S in R^{d_v x d_k}
 * with o = S q (Section 3.1).  Everything here stores the TRANSPOSE,
 * S[d_k][d_v] row-major, so that one KDA key channel S_{h,:,k} (Section 4.1)
 * is one contiguous row of d_v values.  Transposing Eq. 1 gives
 *     S_t = (I - beta_t k_t k_t^T) Diag(alpha_t) S_{t-1} + beta_t k_t v_t^T,
 *     o_t = S_t^T q_t.
 *
 * Pins.  Every function below is pinned by the CPU tests against closed
 * forms, brute force or an independent formulation.  Two things cannot be
 * pinned without the trained weights the paper used, and are therefore
 * "parity unpinned": the paper's compression figures (2.63x ...) and its
 * weight-only decay statistics; and the accuracy of the zero-fill and
 * suffix-refresh approximations on real models.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_KDA = 0, ORACLE_GDN = 1 };
enum { ORACLE_SEL_THRESHOLD = 0, ORACLE_SEL_TOP_RATIO = 1, ORACLE_SEL_EXPLICIT = 2 };
enum { ORACLE_SCOPE_HEAD = 0, ORACLE_SCOPE_LAYER = 1, ORACLE_SCOPE_MODEL = 2 };
enum { ORACLE_MODE_CONTINUE = 0, ORACLE_MODE_SCRATCH_MERGE_LOCAL = 1 };

/* ------------------------------------------------------------------ */
/* Section 3.3, Eq. 2 and Eq. 3: static log-decay and retention horizon */
/* ------------------------------------------------------------------ */

/* softplus(x) = ln(1 + e^x), written to stay finite for large |x|. */
static double softplus64(double x)
{
    if (x > 0.0) return x + log1p(exp(-x));
    return log1p(exp(x));
}

/* Eq. 2: g = -exp(A_log) * softplus(a + dt_bias), with the gate logit fixed
 * at `a` (the paper uses a = -0.3).  Eq. 3: H_s = ln(eps) / g. */
void oracle_horizon(int64_t n_units, const float *A_log, const float *dt_bias,
                    double a, double eps, double *g_out, double *Hs_out)
{
    for (int64_t u = 0; u < n_units; ++u) {
        double g = -exp((double)A_log[u]) * softplus64(a + (double)dt_bias[u]);
        if (g_out) g_out[u] = g;
        if (Hs_out) Hs_out[u] = log(eps) / g;
    }
}

/* Eq. 7: "rounded up to a power of two": the smallest 2^m >= H (an exact
 * power of two maps to itself), then clamped to [4, w_max]. */
double oracle_replay_window_unit(double Hs, double w_max)
{
    double p;
    if (!(Hs > 0.0)) {
        p = 0.0;
    } else if (isinf(Hs)) {
        p = Hs;
    } else {
        int e;
        double f = frexp(Hs, &e); /* Hs = f * 2^e, f in [0.5, 1) */
        p = (f == 0.5) ? ldexp(1.0, e - 1) : ldexp(1.0, e);
    }
    if (p < 4.0) p = 4.0;
    if (p > w_max) p = w_max;
    return p;
}

/* Smallest power of two >= H, no clamp (used to derive a window cap when the
 * selection rule is not the paper's threshold rule). */
static double next_pow2_64(double Hs)
{
    if (!(Hs > 0.0)) return 0.0;
    if (isinf(Hs)) return Hs;
    int e;
    double f = frexp(Hs, &e);
    return (f == 0.5) ? ldexp(1.0, e - 1) : ldexp(1.0, e);
}

/* splitmix64: the counter-based generator behind count-matched random
 * selection.  The library implements the same published function on its own. */
static uint64_t splitmix64(uint64_t x)
{
    x += 0x9E3779B97F4A7C15ULL;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ULL;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBULL;
    return x ^ (x >> 31);
}

/* The same function, exported so that a test can hold it against the generator's
 * published outputs (the n-th output of a generator seeded s is splitmix64 of
 * s + (n-1) * 0x9E3779B97F4A7C15). */
uint64_t oracle_splitmix64(uint64_t x) { return splitmix64(x); }

/* Keep the r units of a group with the largest score; ties go to the lower
 * index.  Deliberately O(n^2): rank by counting, no sort to get wrong. */
static void keep_top(const double *score, int64_t n, int64_t r, uint8_t *mask)
{
    for (int64_t i = 0; i < n; ++i) {
        int64_t ahead = 0; /* units that outrank unit i */
        for (int64_t j = 0; j < n; ++j) {
            if (score[j] > score[i] || (score[j] == score[i] && j < i)) ++ahead;
        }
        mask[i] = (ahead < r) ? 1 : 0;
    }
}

/* Same, but "smallest 64-bit key first" for the random selector. */
static void keep_smallest_key(const uint64_t *key, int64_t n, int64_t r, uint8_t *mask)
{
    for (int64_t i = 0; i < n; ++i) {
        int64_t ahead = 0;
        for (int64_t j = 0; j < n; ++j) {
            if (key[j] < key[i] || (key[j] == key[i] && j < i)) ++ahead;
        }
        mask[i] = (ahead < r) ? 1 : 0;
    }
}

/* Retained count of a top-ratio group: the smallest integer >= ratio*n,
 * where a product within 1e-9 above an integer counts as that integer. */
static int64_t ratio_count(double ratio, int64_t n)
{
    double x = ratio * (double)n - 1e-9;
    int64_t r = (int64_t)ceil(x);
    if (r < 0) r = 0;
    if (r > n) r = n;
    return r;
}

/*
 * The static selection plan (Section 4.1, Eq. 6, Eq. 7, Appendix B).
 *
 * Units: GDN -> one per value head (units_per_head = 1); KDA -> one per
 * (head, key channel) (units_per_head = d_k).  Unit u of layer l has index
 * l*n_l + u with u = head*units_per_head + channel.
 *
 * sel = THRESHOLD: retained iff H_s > w_max, strictly (Section 4.1).
 * sel = TOP_RATIO: within each scope group keep the ratio_count() units of
 *       largest H_s (a benchmark rule; the paper only has the threshold).
 * sel = EXPLICIT: mask supplied by the caller.
 * randomize != 0: afterwards replace each layer's selection by a uniform
 *       draw of the SAME count r_l (the count-matched random control of
 *       Appendix C.3), keyed by splitmix64(seed + (layer << 32) + unit).
 *
 * Outputs (any may be NULL): Hs[L*n_l], mask[L*n_l] (1 = retained),
 * r_l[L], o_l[L+1] with o_0 = 0, o_{l+1} = o_l + r_l (Appendix B, ragged),
 * W_u[L*n_l], and stats[8] = { sum n_l, sum r_l, R_max, C_temp_rag,
 * C_temp_pad, C_ckpt_rag, W_replay, w_max actually used }.
 * unit_bytes and conv_bytes enter C_ckpt only.
 */
int oracle_plan(int kind, int32_t n_layers, int32_t n_heads, int32_t units_per_head,
                const float *A_log, const float *dt_bias, double a, double eps,
                int sel, double w_max, double keep_ratio, int scope,
                int randomize, uint64_t seed, const uint8_t *explicit_mask,
                int64_t unit_bytes, int64_t conv_bytes,
                double *Hs_out, uint8_t *mask_out, int64_t *r_l, int64_t *o_l,
                double *W_u, double *stats)
{
    (void)kind;
    const int64_t n_l = (int64_t)n_heads * units_per_head;
    const int64_t n_all = n_l * n_layers;
    double *Hs = (double *)malloc(sizeof(double) * (size_t)(n_all ? n_all : 1));
    uint8_t *mask = (uint8_t *)malloc((size_t)(n_all ? n_all : 1));
    if (!Hs || !mask) { free(Hs); free(mask); return 1; }

    oracle_horizon(n_all, A_log, dt_bias, a, eps, NULL, Hs);

    if (sel == ORACLE_SEL_THRESHOLD) {
        for (int64_t u = 0; u < n_all; ++u) mask[u] = (Hs[u] > w_max) ? 1 : 0;
    } else if (sel == ORACLE_SEL_TOP_RATIO) {
        int64_t group = (scope == ORACLE_SCOPE_HEAD) ? units_per_head
                      : (scope == ORACLE_SCOPE_LAYER) ? n_l : n_all;
        for (int64_t base = 0; base < n_all; base += group) {
            keep_top(Hs + base, group, ratio_count(keep_ratio, group), mask + base);
        }
    } else if (sel == ORACLE_SEL_EXPLICIT) {
        for (int64_t u = 0; u < n_all; ++u) mask[u] = explicit_mask[u] ? 1 : 0;
    } else {
        free(Hs); free(mask); return 2;
    }

    if (randomize) {
        uint64_t *key = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)(n_l ? n_l : 1));
        if (!key) { free(Hs); free(mask); return 1; }
        for (int32_t l = 0; l < n_layers; ++l) {
            int64_t r = 0;
            for (int64_t u = 0; u < n_l; ++u) r += mask[l * n_l + u];
            for (int64_t u = 0; u < n_l; ++u)
                key[u] = splitmix64(seed + (((uint64_t)l) << 32) + (uint64_t)u);
            keep_smallest_key(key, n_l, r, mask + l * n_l);
        }
        free(key);
    }

    /* per-layer counts and ragged offsets */
    int64_t sum_r = 0, R_max = 0;
    for (int32_t l = 0; l < n_layers; ++l) {
        int64_t r = 0;
        for (int64_t u = 0; u < n_l; ++u) r += mask[l * n_l + u];
        if (r_l) r_l[l] = r;
        if (o_l) { if (l == 0) o_l[0] = 0; o_l[l + 1] = o_l[l] + r; }
        sum_r += r;
        if (r > R_max) R_max = r;
    }
    if (o_l && n_layers == 0) o_l[0] = 0;

    /* replay windows, Eq. 7 */
    double w_cap = w_max;
    if (sel != ORACLE_SEL_THRESHOLD && !(w_max > 0.0)) {
        double hmax = 0.0;
        for (int64_t u = 0; u < n_all; ++u) if (!mask[u] && Hs[u] > hmax) hmax = Hs[u];
        w_cap = next_pow2_64(hmax);
        if (w_cap < 4.0 && hmax > 0.0) w_cap = 4.0;
    }
    double w_replay = 0.0;
    for (int64_t u = 0; u < n_all; ++u) {
        double w = oracle_replay_window_unit(Hs[u], w_cap);
        if (W_u) W_u[u] = w;
        if (!mask[u] && w > w_replay) w_replay = w;
    }

    if (stats) {
        double sum_n = (double)n_all;
        stats[0] = sum_n;
        stats[1] = (double)sum_r;
        stats[2] = (double)R_max;
        stats[3] = sum_r ? sum_n / (double)sum_r : INFINITY;               /* Eq. 6 */
        stats[4] = R_max ? sum_n / ((double)n_layers * (double)R_max) : INFINITY;
        double b_dense = sum_n * (double)unit_bytes, b_rag = (double)sum_r * (double)unit_bytes;
        stats[5] = (b_rag + (double)conv_bytes) > 0.0
                 ? (b_dense + (double)conv_bytes) / (b_rag + (double)conv_bytes) : INFINITY;
        stats[6] = w_replay;
        stats[7] = w_cap;
    }
    if (Hs_out) memcpy(Hs_out, Hs, sizeof(double) * (size_t)n_all);
    if (mask_out) memcpy(mask_out, mask, (size_t)n_all);
    free(Hs); free(mask);
    return 0;
}

/* Appendix C.1 slot budget: N = floor(B / max_r[b_r^temporal + b^conv]) - 1
 * (allocator slot 0 is reserved). */
int64_t oracle_slot_budget(int64_t budget_bytes, const int64_t *temporal_bytes_per_rank,
                           int32_t n_ranks, int64_t conv_bytes)
{
    int64_t worst = 0;
    for (int32_t r = 0; r < n_ranks; ++r) {
        int64_t b = temporal_bytes_per_rank[r] + conv_bytes;
        if (b > worst) worst = b;
    }
    if (worst <= 0) return -1;
    return budget_bytes / worst - 1;
}

/* Section 4.3, second stage: the TP group as one storage pool.  With U_r packed
 * units on rank r and T ranks, the per-rank slot width is C = ceil(sum_r U_r / T).
 * The paper fixes C and that only remotely owned units move; which unit goes where
 * is this build's reading: the packed units of all ranks, in rank order, form one
 * sequence, and the unit at global position p is stored on rank p / C.
 * send[r*T + s] = number of rank r's units stored on rank s (the diagonal stays put).
 * Done unit by unit. */
int64_t oracle_tp_balance(const int64_t *U, int32_t T, int64_t *send)
{
    int64_t total = 0;
    for (int32_t r = 0; r < T; ++r) total += U[r];
    int64_t C = (total + T - 1) / T;
    for (int32_t i = 0; i < T * T; ++i) send[i] = 0;
    int64_t p = 0; /* global position */
    for (int32_t r = 0; r < T; ++r)
        for (int64_t u = 0; u < U[r]; ++u, ++p) send[r * T + (int32_t)(p / C)] += 1;
    return C;
}

/* Section 4.3, second stage, the placement itself: rank `rank` holds `U[rank]`
 * packed units in `packed` (one checkpoint slot, the output of oracle_pack).
 * Its j-th unit has global position p = U[0] + ... + U[rank-1] + j and is stored
 * on rank p / C at local unit index p % C, C = ceil(sum U / T).  pools[s] is the
 * slot of rank s (C units).  Walks the units one by one. */
void oracle_tp_place(const uint32_t *packed, const int64_t *U, int32_t T, int32_t rank,
                     int64_t unit_words, uint32_t *const *pools)
{
    int64_t total = 0, begin = 0;
    for (int32_t r = 0; r < T; ++r) { total += U[r]; if (r < rank) begin += U[r]; }
    if (total == 0) return;
    int64_t C = (total + T - 1) / T;
    for (int64_t j = 0; j < U[rank]; ++j) {
        int64_t p = begin + j;
        uint32_t *dst = pools[p / C] + (p % C) * unit_words;
        for (int64_t w = 0; w < unit_words; ++w) dst[w] = packed[j * unit_words + w];
    }
}

/* Section 4.3, first stage.  The paper says only that head bundles are
 * redistributed across TP ranks at model-load time; the reading implemented:
 * every rank keeps n_bundles / T bundles of every layer; layers are visited in
 * ascending order and, within a layer, the not yet placed bundle with the most
 * retained units (ties: lower index) goes to the rank whose payload so far is
 * smallest among the ranks that still have room in this layer (ties: lower
 * rank).  weight[l*n_bundles + b] = retained units of bundle b in layer l.
 * perm[l*n_bundles + i] = bundle at position i; rank r owns positions
 * [r*per, (r+1)*per) with its bundles in ascending index.  Selection by
 * repeated scanning, no sort. */
void oracle_tp_head_permutation(const int64_t *weight, int32_t n_layers, int32_t n_bundles,
                                int32_t T, int32_t *perm, int64_t *load)
{
    int32_t per = n_bundles / T;
    int32_t *owner = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_bundles ? n_bundles : 1));
    int32_t *room = (int32_t *)malloc(sizeof(int32_t) * (size_t)T);
    for (int32_t r = 0; r < T; ++r) load[r] = 0;
    for (int32_t l = 0; l < n_layers; ++l) {
        const int64_t *w = weight + (int64_t)l * n_bundles;
        for (int32_t b = 0; b < n_bundles; ++b) owner[b] = -1;
        for (int32_t r = 0; r < T; ++r) room[r] = per;
        for (int32_t placed = 0; placed < n_bundles; ++placed) {
            int32_t pick = -1;
            for (int32_t b = 0; b < n_bundles; ++b)
                if (owner[b] < 0 && (pick < 0 || w[b] > w[pick])) pick = b;
            int32_t to = -1;
            for (int32_t r = 0; r < T; ++r)
                if (room[r] > 0 && (to < 0 || load[r] < load[to])) to = r;
            owner[pick] = to;
            room[to] -= 1;
            load[to] += w[pick];
        }
        for (int32_t r = 0; r < T; ++r) {
            int32_t i = 0;
            for (int32_t b = 0; b < n_bundles; ++b)
                if (owner[b] == r) perm[(int64_t)l * n_bundles + r * per + i++] = b;
        }
    }
    free(owner); free(room);
}

/* The convolution state travels with a checkpoint as an opaque blob (Section
 * 4.1): dst[dst_idx[i]] = src[src_idx[i]], blob_bytes each, strides in bytes. */
void oracle_copy_blobs(const uint8_t *src, int64_t src_stride, const int32_t *src_idx,
                       uint8_t *dst, int64_t dst_stride, const int32_t *dst_idx,
                       int64_t blob_bytes, int32_t n_pairs)
{
    for (int32_t i = 0; i < n_pairs; ++i)
        for (int64_t b = 0; b < blob_bytes; ++b)
            dst[(int64_t)dst_idx[i] * dst_stride + b] = src[(int64_t)src_idx[i] * src_stride + b];
}

/* ------------------------------------------------------------------ */
/* Store path (Section 4.1, Appendix B ragged layout): pack             */
/* ------------------------------------------------------------------ */

/*
 * For every pair i and layer l, the retained units of the dense state, in
 * ascending unit index, are copied to pool[dst_slot[i]][o_l + j].  A unit is
 * unit_words 32-bit words (d_v for a KDA row, d_k*d_v for a GDN head) and
 * unit u of layer l of request q starts at word
 *     q*req_stride + l*layer_stride + u*unit_words.
 * Bits are copied, never interpreted.
 */
void oracle_pack(const uint8_t *mask, int32_t n_layers, int64_t n_l, int64_t unit_words,
                 const uint32_t *state, int64_t layer_stride, int64_t req_stride,
                 const int32_t *src_req, uint32_t *pool, int64_t slot_stride,
                 const int32_t *dst_slot, int32_t n_pairs)
{
    for (int32_t i = 0; i < n_pairs; ++i) {
        int64_t j = 0; /* running packed position = o_l + (rank within layer) */
        for (int32_t l = 0; l < n_layers; ++l) {
            for (int64_t u = 0; u < n_l; ++u) {
                if (!mask[l * n_l + u]) continue;
                const uint32_t *src = state + (int64_t)src_req[i] * req_stride + l * layer_stride + u * unit_words;
                uint32_t *dst = pool + (int64_t)dst_slot[i] * slot_stride + j * unit_words;
                for (int64_t w = 0; w < unit_words; ++w) dst[w] = src[w];
                ++j;
            }
        }
    }
}

/* ------------------------------------------------------------------ */
/* Load path, zero-fill policy (Section 4.2): restore                   */
/* ------------------------------------------------------------------ */

/* The destination dense state is first cleared to all-zero bits, then the
 * retained units are copied back to their architectural positions. */
void oracle_restore(const uint8_t *mask, int32_t n_layers, int64_t n_l, int64_t unit_words,
                    const uint32_t *pool, int64_t slot_stride, const int32_t *src_slot,
                    uint32_t *state, int64_t layer_stride, int64_t req_stride,
                    const int32_t *dst_req, int32_t n_pairs)
{
    for (int32_t i = 0; i < n_pairs; ++i) {
        for (int32_t l = 0; l < n_layers; ++l) {
            uint32_t *dense = state + (int64_t)dst_req[i] * req_stride + l * layer_stride;
            for (int64_t w = 0; w < n_l * unit_words; ++w) dense[w] = 0u;
        }
        int64_t j = 0;
        for (int32_t l = 0; l < n_layers; ++l) {
            for (int64_t u = 0; u < n_l; ++u) {
                if (!mask[l * n_l + u]) continue;
                const uint32_t *src = pool + (int64_t)src_slot[i] * slot_stride + j * unit_words;
                uint32_t *dst = state + (int64_t)dst_req[i] * req_stride + l * layer_stride + u * unit_words;
                for (int64_t w = 0; w < unit_words; ++w) dst[w] = src[w];
                ++j;
            }
        }
    }
}

/* ------------------------------------------------------------------ */
/* Appendix B, padded layout (Scheme 1): pool [L][slots][R_max][unit]   */
/* ------------------------------------------------------------------ */

/* Entry (l, slot, j) of the padded pool, j < R_max, starts at word
 *     ((l*n_slots + slot)*R_max + j)*unit_words.
 * Layer l's j-th retained unit (ascending unit index) goes to entry j; entries
 * r_l .. R_max-1 are padding and are neither written (pack) nor read (restore). */
void oracle_pack_padded(const uint8_t *mask, int32_t n_layers, int64_t n_l, int64_t unit_words,
                        const uint32_t *state, int64_t layer_stride, int64_t req_stride,
                        const int32_t *src_req, uint32_t *pool, int64_t n_slots, int64_t R_max,
                        const int32_t *dst_slot, int32_t n_pairs)
{
    for (int32_t i = 0; i < n_pairs; ++i) {
        for (int32_t l = 0; l < n_layers; ++l) {
            int64_t j = 0; /* rank of the unit among the layer's retained units */
            for (int64_t u = 0; u < n_l; ++u) {
                if (!mask[l * n_l + u]) continue;
                const uint32_t *src = state + (int64_t)src_req[i] * req_stride + l * layer_stride + u * unit_words;
                uint32_t *dst = pool + (((int64_t)l * n_slots + dst_slot[i]) * R_max + j) * unit_words;
                for (int64_t w = 0; w < unit_words; ++w) dst[w] = src[w];
                ++j;
            }
        }
    }
}

/* Zero-fill load from the padded pool: clear, then copy the valid entries back. */
void oracle_restore_padded(const uint8_t *mask, int32_t n_layers, int64_t n_l, int64_t unit_words,
                           const uint32_t *pool, int64_t n_slots, int64_t R_max, const int32_t *src_slot,
                           uint32_t *state, int64_t layer_stride, int64_t req_stride,
                           const int32_t *dst_req, int32_t n_pairs)
{
    for (int32_t i = 0; i < n_pairs; ++i) {
        for (int32_t l = 0; l < n_layers; ++l) {
            uint32_t *dense = state + (int64_t)dst_req[i] * req_stride + l * layer_stride;
            for (int64_t w = 0; w < n_l * unit_words; ++w) dense[w] = 0u;
            int64_t j = 0;
            for (int64_t u = 0; u < n_l; ++u) {
                if (!mask[l * n_l + u]) continue;
                const uint32_t *src = pool + (((int64_t)l * n_slots + src_slot[i]) * R_max + j) * unit_words;
                uint32_t *dst = dense + u * unit_words;
                for (int64_t w = 0; w < unit_words; ++w) dst[w] = src[w];
                ++j;
            }
        }
    }
}

/* ------------------------------------------------------------------ */
/* Suffix refresh (Section 3.1 Eq. 1; Section 4.2): token-by-token replay */
/* ------------------------------------------------------------------ */

static double bf16_to_double(uint16_t h)
{
    uint32_t w = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

static double load_io(const void *p, int is_bf16, int64_t idx)
{
    return is_bf16 ? bf16_to_double(((const uint16_t *)p)[idx]) : (double)((const float *)p)[idx];
}

/*
 * One (request, layer, value head) unit of Eq. 1, transposed orientation.
 * S is d_k x d_v fp64 in/out.  Token streams are addressed through the
 * element strides given; g_chan_stride = 0 broadcasts one decay over the key
 * channels (GDN, scalar per-head alpha), 1 reads a channel-wise decay (KDA).
 */
static void replay_unit(double *S, int32_t d_k, int32_t d_v, int64_t n_tok,
                        const void *q, const void *k, int64_t qk_tok_stride,
                        const void *v, int64_t v_tok_stride, int io_bf16,
                        const float *g, int64_t g_tok_stride, int64_t g_chan_stride,
                        const float *beta, int64_t beta_tok_stride, double q_scale,
                        double *o, int64_t o_tok_stride, double *r_tmp)
{
    for (int64_t t = 0; t < n_tok; ++t) {
        /* attenuate the old state: Diag(alpha_t) acts on the key-channel index */
        for (int32_t c = 0; c < d_k; ++c) {
            double alpha = exp((double)g[t * g_tok_stride + c * g_chan_stride]);
            for (int32_t j = 0; j < d_v; ++j) S[c * d_v + j] *= alpha;
        }
        /* r = (decayed S)^T k_t : what the state currently returns for key k_t */
        for (int32_t j = 0; j < d_v; ++j) r_tmp[j] = 0.0;
        for (int32_t c = 0; c < d_k; ++c) {
            double kc = load_io(k, io_bf16, t * qk_tok_stride + c);
            for (int32_t j = 0; j < d_v; ++j) r_tmp[j] += kc * S[c * d_v + j];
        }
        /* remove the content aligned with k_t and write the new association */
        double b = (double)beta[t * beta_tok_stride];
        for (int32_t j = 0; j < d_v; ++j) /* u_t = beta_t (v_t - r) */
            r_tmp[j] = b * (load_io(v, io_bf16, t * v_tok_stride + j) - r_tmp[j]);
        for (int32_t c = 0; c < d_k; ++c) {
            double kc = load_io(k, io_bf16, t * qk_tok_stride + c);
            for (int32_t j = 0; j < d_v; ++j) S[c * d_v + j] += kc * r_tmp[j];
        }
        /* read-out from the post-update state: o_t = S_t^T q_t */
        if (o) {
            for (int32_t j = 0; j < d_v; ++j) {
                double acc = 0.0;
                for (int32_t c = 0; c < d_k; ++c)
                    acc += load_io(q, io_bf16, t * qk_tok_stride + c) * S[c * d_v + j];
                o[t * o_tok_stride + j] = q_scale * acc;
            }
        }
    }
}

/*
 * Batched refresh over requests x layers x value heads.
 *
 * Streams (token-major, T = cu_seqlens[n_req] tokens per layer):
 *   q, k : [n_layers][T][H_k][d_k]   bf16 (uint16 bit patterns) or fp32
 *   v    : [n_layers][T][H_v][d_v]   same dtype
 *   g    : [n_layers][T][H_v][d_k]   fp32 log-decay (KDA)
 *          [n_layers][T][H_v]        fp32 log-decay (GDN)
 *   beta : [n_layers][T][H_v]        fp32
 *   o    : [n_layers][T][H_v][d_v]   fp64 out (may be NULL)
 * Value head h reads key head h / (H_v / H_k).
 * State: fp32, unit (req, l, h) at state + req_idx[r]*req_stride +
 *   l*layer_stride + h*d_k*d_v, updated in place.  final_state64 (may be
 *   NULL) additionally receives every unit's fp64 final state,
 *   [n_req][n_layers][H_v][d_k][d_v], before rounding to fp32.
 *
 * mode CONTINUE: start from the stored state, write every row back.
 * mode SCRATCH_MERGE_LOCAL (the paper's suffix-refresh load policy): start
 *   from a zero scratch state, then copy only the OMITTED units of the plan
 *   (mask == 0: KDA rows, GDN whole heads) into the stored state; retained
 *   units keep their stored values.  final_state64 then holds the merged state.
 */
int oracle_refresh(int kind, int32_t n_layers, int32_t H_v, int32_t H_k, int32_t d_k, int32_t d_v,
                   float *state, int64_t layer_stride, int64_t req_stride, const int32_t *req_idx,
                   const void *q, const void *k, const void *v, int io_bf16,
                   const float *g, const float *beta, const int32_t *cu_seqlens, int32_t n_req,
                   double q_scale, double *o, int mode, const uint8_t *mask,
                   double *final_state64, int32_t n_threads)
{
    if (H_k <= 0 || H_v % H_k != 0) return 2;
    const int64_t T = cu_seqlens[n_req];
    const int32_t group = H_v / H_k;
    const int64_t n_units = (int64_t)n_req * n_layers * H_v;
    const int64_t sd = (int64_t)d_k * d_v;
    const int64_t g_width = (kind == ORACLE_KDA) ? d_k : 1;
    const size_t esz = io_bf16 ? 2 : 4;
    int failed = 0;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#else
    (void)n_threads;
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t w = 0; w < n_units; ++w) {
        const int32_t h = (int32_t)(w % H_v);
        const int32_t l = (int32_t)((w / H_v) % n_layers);
        const int32_t r = (int32_t)(w / ((int64_t)H_v * n_layers));
        const int32_t hk = h / group;
        const int64_t t0 = cu_seqlens[r], n_tok = cu_seqlens[r + 1] - t0;
        double *S = (double *)malloc(sizeof(double) * (size_t)(sd + d_v));
        if (!S) { failed = 1; continue; }
        double *r_tmp = S + sd;
        float *st = state + (int64_t)req_idx[r] * req_stride + (int64_t)l * layer_stride + (int64_t)h * sd;
        if (mode == ORACLE_MODE_CONTINUE) for (int64_t i = 0; i < sd; ++i) S[i] = (double)st[i];
        else for (int64_t i = 0; i < sd; ++i) S[i] = 0.0;

        const int64_t tok = (int64_t)l * T + t0;
        replay_unit(S, d_k, d_v, n_tok,
                    (const char *)q + esz * (size_t)((tok * H_k + hk) * d_k),
                    (const char *)k + esz * (size_t)((tok * H_k + hk) * d_k), (int64_t)H_k * d_k,
                    (const char *)v + esz * (size_t)((tok * H_v + h) * d_v), (int64_t)H_v * d_v, io_bf16,
                    g + (tok * H_v + h) * g_width, (int64_t)H_v * g_width, (kind == ORACLE_KDA) ? 1 : 0,
                    beta + tok * H_v + h, (int64_t)H_v, q_scale,
                    o ? o + (tok * H_v + h) * d_v : NULL, (int64_t)H_v * d_v, r_tmp);

        double *f64 = final_state64 ? final_state64 + w * sd : NULL;
        if (mode == ORACLE_MODE_CONTINUE) {
            for (int64_t i = 0; i < sd; ++i) { st[i] = (float)S[i]; if (f64) f64[i] = S[i]; }
        } else {
            for (int32_t c = 0; c < d_k; ++c) {
                int64_t unit = (kind == ORACLE_KDA) ? ((int64_t)h * d_k + c) : h;
                int64_t n_l = (kind == ORACLE_KDA) ? (int64_t)H_v * d_k : H_v;
                int retained = mask[(int64_t)l * n_l + unit];
                for (int32_t j = 0; j < d_v; ++j) {
                    int64_t i = (int64_t)c * d_v + j;
                    if (!retained) st[i] = (float)S[i];
                    if (f64) f64[i] = retained ? (double)st[i] : S[i];
                }
            }
        }
        free(S);
    }
    return failed;
}

int32_t oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ */
/* Appendix D: symmetric INT8 checkpoint quantiser                      */
/* ------------------------------------------------------------------ */

/*
 * One scale per row of `width` values (a (layer, head, key channel) tuple,
 * shared over d_v):  a = max|S|, s = max(a, 1e-8)/127,
 * q = clip(round(S/s), -127, 127), with max, division and rounding done in
 * fp32 as the paper states; round = to nearest, ties to even.
 */
void oracle_int8_quantize(const float *rows, int64_t n_rows, int64_t width, int8_t *q, float *scale)
{
    for (int64_t r = 0; r < n_rows; ++r) {
        float a = 0.0f;
        for (int64_t j = 0; j < width; ++j) {
            float x = fabsf(rows[r * width + j]);
            if (x > a) a = x;
        }
        float s = (a > 1e-8f ? a : 1e-8f) / 127.0f;
        scale[r] = s;
        for (int64_t j = 0; j < width; ++j) {
            float y = nearbyintf(rows[r * width + j] / s); /* default rounding mode: ties to even */
            if (y > 127.0f) y = 127.0f;
            if (y < -127.0f) y = -127.0f;
            q[r * width + j] = (int8_t)y;
        }
    }
}

/* Dequantise once on a hit: S_hat = q * s (fp32). */
void oracle_int8_dequantize(const int8_t *q, const float *scale, int64_t n_rows, int64_t width, float *rows)
{
    for (int64_t r = 0; r < n_rows; ++r)
        for (int64_t j = 0; j < width; ++j)
            rows[r * width + j] = (float)q[r * width + j] * scale[r];
}
