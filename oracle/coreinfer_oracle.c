/*
 * CPU oracle for the CoreInfer hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain statement of what the path computes.  It is
 * used by the tests, by the smoke check and by the benchmark's CPU-baseline
 * leg; the product (the CUDA library) never calls, links or imports it, and
 * it shares no code with the CUDA path.
 *
 * What it follows:
 *   - token-wise core neurons      : Definition 1 / Eq. 1
 *   - per-neuron membership count  : Eq. 3
 *   - sentence-wise core neurons   : Definition 2 / Eq. 2
 *   - decode over the fixed set    : Section 4.2 (the set found at pre-fill is
 *                                    used unchanged for every decoded token)
 *   - precision                    : Section 5 "Models" (stored values fp32,
 *                                    intermediate activations fp32)
 *
 * Readings taken where the paper leaves a choice (each is also what the CUDA
 * path is required to do):
 *   - "top alpha" keeps the LARGEST alpha-fraction of the positive entries;
 *     the number kept is ceil(alpha * P), P = number of positive entries.
 *   - exactly that many are kept; equal values are ordered by lower index.
 *   - the sentence set has exactly ceil(beta * N) members out of all N
 *     neurons; equal counts are ordered by lower index (so neurons with
 *     count 0 fill the set in ascending index if too few were ever counted).
 *   - "positive" is decided on the IEEE-754 bit pattern: sign clear, not
 *     zero, not NaN.  Subnormals and +Inf are positive.
 *   - the set is emitted in ascending neuron index.
 *
 * Floating point: tensors are stored as fp32 (bf16 inputs are widened exactly
 * by the caller); every running sum is a double and is rounded to fp32 once.
 * Compiled with -DORACLE_F32_ACC the running sums of oracle_ffn are fp32 instead
 * (plain sequential fp32 sums): that variant is not the oracle, it only serves
 * to report how far a pure fp32 accumulation is from the double one.
 *
 * Every function here is pinned by tests that do not call it to produce their
 * expected values (hand-worked example, brute-force ranking, library sort and
 * matmul, closed forms, invariants).  Nothing here is "parity unpinned".
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

#ifdef ORACLE_F32_ACC
typedef float acc_t;
#else
typedef double acc_t;
#endif
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ceil(frac * n), clamped to [0, n].  The 1e-6 guard makes products that are
 * exact integers in decimal (0.2 * 20480, 0.25 * 11008) immune to the binary
 * representation error of frac.  (Reading of Definitions 1 and 2: the size of
 * a "top fraction" is the ceiling of fraction times population.) */
int32_t oracle_count(double frac, int32_t n)
{
    if (n <= 0) return 0;
    double c = ceil(frac * (double)n - 1e-6);
    if (c < 0.0) c = 0.0;
    if (c > (double)n) c = (double)n;
    return (int32_t)c;
}

static inline uint32_t f32_bits(float v)
{
    uint32_t u;
    memcpy(&u, &v, sizeof u);
    return u;
}

/* a_n > 0 of Definition 1, decided on the bit pattern. */
static inline int is_positive(float v)
{
    uint32_t u = f32_bits(v);
    return u > 0u && u <= 0x7F800000u;
}

typedef struct { uint32_t key; int32_t idx; } entry_t;

/* larger key first; equal keys: lower index first */
static int cmp_entry_desc(const void *pa, const void *pb)
{
    const entry_t *a = (const entry_t *)pa, *b = (const entry_t *)pb;
    if (a->key != b->key) return (a->key > b->key) ? -1 : 1;
    if (a->idx != b->idx) return (a->idx < b->idx) ? -1 : 1;
    return 0;
}

static int cmp_i32_asc(const void *pa, const void *pb)
{
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

/* Token-wise core neurons of one row (Definition 1 / Eq. 1).
 * Writes the member indices (in rank order) to `members` (capacity N) and
 * returns how many there are.  Positive floats order like their bit patterns,
 * so the sort key is the pattern itself. */
int32_t oracle_token_core(const float *a, int32_t N, double alpha,
                          int32_t *members)
{
    entry_t *pos = (entry_t *)malloc(sizeof(entry_t) * (size_t)(N > 0 ? N : 1));
    int32_t P = 0;
    for (int32_t n = 0; n < N; ++n)
        if (is_positive(a[n])) { pos[P].key = f32_bits(a[n]); pos[P].idx = n; ++P; }
    int32_t k = oracle_count(alpha, P);
    qsort(pos, (size_t)P, sizeof(entry_t), cmp_entry_desc);   /* full sort */
    for (int32_t i = 0; i < k; ++i) members[i] = pos[i].idx;
    free(pos);
    return k;
}

/* Sentence-wise core neurons (Definition 2 / Eq. 2 with the counts of Eq. 3).
 * A: [T][ld] fp32, first N entries of each row used.
 * S: out, K = oracle_count(beta, N) ascending indices.
 * f: out, [N] membership counts.  Returns K. */
int32_t oracle_select(const float *A, int32_t T, int32_t N, int64_t ld,
                      double alpha, double beta, int32_t *S, int32_t *f)
{
    for (int32_t n = 0; n < N; ++n) f[n] = 0;
#ifdef _OPENMP
#pragma omp parallel
#endif
    {
        int32_t *members = (int32_t *)malloc(sizeof(int32_t) * (size_t)(N > 0 ? N : 1));
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
        for (int32_t t = 0; t < T; ++t) {
            int32_t k = oracle_token_core(A + (int64_t)t * ld, N, alpha, members);
            for (int32_t i = 0; i < k; ++i) {
#ifdef _OPENMP
#pragma omp atomic
#endif
                f[members[i]] += 1;                  /* Eq. 3: the indicator sum */
            }
        }
        free(members);
    }
    int32_t K = oracle_count(beta, N);
    entry_t *ord = (entry_t *)malloc(sizeof(entry_t) * (size_t)(N > 0 ? N : 1));
    for (int32_t n = 0; n < N; ++n) { ord[n].key = (uint32_t)f[n]; ord[n].idx = n; }
    qsort(ord, (size_t)N, sizeof(entry_t), cmp_entry_desc);   /* full sort */
    for (int32_t i = 0; i < K; ++i) S[i] = ord[i].idx;
    qsort(S, (size_t)K, sizeof(int32_t), cmp_i32_asc);
    free(ord);
    return K;
}

/* Compaction: "deploy only the necessary neurons" (Section 5.3) written as
 * element copies.  Sources are row-major W_up [N][d], W_gate [N][d] (or NULL),
 * W_down [d][N], b_up [N] (or NULL), elements of `esize` bytes.  Outputs are
 * [K][d] row-major (the W_down one is the transpose of its selected columns)
 * and [K]. */
void oracle_compact(const void *w_up, const void *w_gate, const void *w_down,
                    const void *b_up, int32_t esize, int32_t d, int32_t N,
                    const int32_t *S, int32_t K,
                    void *w_up_c, void *w_gate_c, void *w_downT_c, void *b_up_c)
{
    const char *up = (const char *)w_up, *gate = (const char *)w_gate;
    const char *down = (const char *)w_down, *bu = (const char *)b_up;
    char *upc = (char *)w_up_c, *gatec = (char *)w_gate_c;
    char *downc = (char *)w_downT_c, *buc = (char *)b_up_c;
    size_t e = (size_t)esize;
    for (int32_t k = 0; k < K; ++k) {
        size_t n = (size_t)S[k];
        for (int32_t i = 0; i < d; ++i) {
            memcpy(upc + ((size_t)k * d + i) * e, up + (n * d + i) * e, e);
            if (gate)
                memcpy(gatec + ((size_t)k * d + i) * e, gate + (n * d + i) * e, e);
            memcpy(downc + ((size_t)k * d + i) * e, down + ((size_t)i * N + n) * e, e);
        }
        if (bu) memcpy(buc + (size_t)k * e, bu + n * e, e);
    }
}

/* Gate nonlinearity of the gated kinds.  kind 1: ReLU.  kind 2: SiLU, g / (1 + exp(-g)),
 * the activation of the LLaMA models for which Section 5.1 ("Verification and Analysis") and
 * the appendix "Generalization to LLaMA3.1-8b" report the same core-neuron behaviour; the
 * paper gives no separate score for them, so Definition 1 is applied unchanged to the
 * intermediate h = silu(w_gate.x) * (w_up.x) (entries that are not positive are never core
 * neurons, as for the ReLU-gated kind).  Evaluated in double, rounded to fp32. */
static float gate_act(float g, int32_t kind)
{
    if (kind == 2) return (float)((double)g / (1.0 + exp(-(double)g)));
    return g > 0.0f ? g : 0.0f;
}

/* Decode FFN over compacted weights (Section 4.2: inference through the fixed
 * core neurons only).  kind 0: h = max(w_up.x + b_up, 0); kind 1 (ReLU-gated):
 * h = max(w_gate.x, 0) * (w_up.x); kind 2 (SiLU-gated): h = silu(w_gate.x) * (w_up.x).
 * y = sum_k h_k * w_downT_c[k] + b_down.
 * x: [B][d]; w_*_c: [K][d]; b_up_c: [K] or NULL; b_down: [d] or NULL;
 * y: [B][d]; h_out: [B][K] or NULL. */
void oracle_ffn(const float *x, int32_t B, int32_t kind, int32_t d, int32_t K,
                const float *w_up_c, const float *w_gate_c, const float *w_downT_c,
                const float *b_up_c, const float *b_down, float *y, float *h_out)
{
    float *h = (float *)malloc(sizeof(float) * (size_t)(K > 0 ? K : 1));
    acc_t *acc = (acc_t *)malloc(sizeof(acc_t) * (size_t)(d > 0 ? d : 1));
    for (int32_t b = 0; b < B; ++b) {
        const float *xb = x + (size_t)b * d;
#ifdef _OPENMP
#pragma omp parallel for schedule(static)
#endif
        for (int32_t k = 0; k < K; ++k) {
            acc_t su = 0;
            for (int32_t i = 0; i < d; ++i)
                su += (acc_t)w_up_c[(size_t)k * d + i] * (acc_t)xb[i];
            if (kind == 0 && b_up_c) su += (acc_t)b_up_c[k];
            float u = (float)su;
            if (kind >= 1) {
                acc_t sg = 0;
                for (int32_t i = 0; i < d; ++i)
                    sg += (acc_t)w_gate_c[(size_t)k * d + i] * (acc_t)xb[i];
                float g = (float)sg;
                h[k] = gate_act(g, kind) * u;
            } else {
                h[k] = u > 0.0f ? u : 0.0f;
            }
        }
        /* y_j = sum over k in ascending order.  Columns are handed to the threads in
         * blocks; within a block the k loop is outermost only so that memory is walked
         * row by row: each y_j still adds k = 0, 1, ... in that order, whatever the
         * number of threads. */
#ifdef _OPENMP
#pragma omp parallel for schedule(static)
#endif
        for (int32_t j0 = 0; j0 < d; j0 += 64) {
            const int32_t j1 = j0 + 64 < d ? j0 + 64 : d;
            for (int32_t j = j0; j < j1; ++j) acc[j] = 0;
            for (int32_t k = 0; k < K; ++k) {
                acc_t hk = (acc_t)h[k];
                const float *row = w_downT_c + (size_t)k * d;
                for (int32_t j = j0; j < j1; ++j) acc[j] += hk * (acc_t)row[j];
            }
            for (int32_t j = j0; j < j1; ++j)
                y[(size_t)b * d + j] = (float)(acc[j] + (b_down ? (acc_t)b_down[j] : (acc_t)0));
        }
        if (h_out) memcpy(h_out + (size_t)b * K, h, sizeof(float) * (size_t)K);
    }
    free(h);
    free(acc);
}

/* Dense FFN on the uncompacted weights: the same arithmetic with k over all N
 * neurons and W_down read in its own [d][N] layout.  H: [T][N] intermediate
 * activations (the tensor Definition 1 is applied to) or NULL; Y: [T][d] or
 * NULL. */
void oracle_ffn_dense(const float *x, int32_t T, int32_t kind, int32_t d, int32_t N,
                      const float *w_up, const float *w_gate, const float *w_down,
                      const float *b_up, const float *b_down, float *H, float *Y)
{
#ifdef _OPENMP
#pragma omp parallel
#endif
    {
        float *h = (float *)malloc(sizeof(float) * (size_t)(N > 0 ? N : 1));
#ifdef _OPENMP
#pragma omp for schedule(static)
#endif
        for (int32_t t = 0; t < T; ++t) {
            const float *xt = x + (size_t)t * d;
            for (int32_t n = 0; n < N; ++n) {
                double su = 0.0;
                for (int32_t i = 0; i < d; ++i)
                    su += (double)w_up[(size_t)n * d + i] * (double)xt[i];
                if (kind == 0 && b_up) su += (double)b_up[n];
                float u = (float)su;
                if (kind >= 1) {
                    double sg = 0.0;
                    for (int32_t i = 0; i < d; ++i)
                        sg += (double)w_gate[(size_t)n * d + i] * (double)xt[i];
                    float g = (float)sg;
                    h[n] = gate_act(g, kind) * u;
                } else {
                    h[n] = u > 0.0f ? u : 0.0f;
                }
            }
            if (H) memcpy(H + (size_t)t * N, h, sizeof(float) * (size_t)N);
            if (Y) {
                for (int32_t j = 0; j < d; ++j) {
                    double s = 0.0;
                    for (int32_t n = 0; n < N; ++n)
                        s += (double)h[n] * (double)w_down[(size_t)j * N + n];
                    Y[(size_t)t * d + j] = (float)(s + (b_down ? (double)b_down[j] : 0.0));
                }
            }
        }
        free(h);
    }
}

/* Layer-to-layer glue of the decode stack.  The paper does not describe the
 * rest of the transformer; the stack used for measurement chains FFN layers
 * with a parameter-free residual + RMS normalisation so that each layer
 * depends on the previous one:  out = (x + y) / sqrt(mean((x + y)^2)).
 * Computed in double, returned as fp32 (the caller rounds to the layer
 * input type). */
void oracle_glue(const float *x, const float *y, int32_t d, float *out)
{
    double ss = 0.0;
    for (int32_t i = 0; i < d; ++i) {
        double v = (double)x[i] + (double)y[i];
        ss += v * v;
    }
    double r = sqrt(ss / (double)d);
    for (int32_t i = 0; i < d; ++i)
        out[i] = (float)(((double)x[i] + (double)y[i]) / r);
}

/* ---- core sets over several sentences (Section 3.2 Insight-1/2, Section 4.1) -------------
 *
 * The neurons "that appear most frequently": the `K` entries of counts[0..N) with the largest
 * count, equal counts ordered by lower index, written in ascending index (the same rule as
 * Definition 2 / Eq. 2 applies to the counts of Eq. 3).  It serves two purposes:
 *   - the sentence-wise set of a prompt that arrives in pieces: Eq. 3 is a sum over tokens, so
 *     the counts of the pieces add up and the set of the whole prompt follows from the sum;
 *   - similarity-guided prediction (Section 4.1): counts[n] = number of sentences of a semantic
 *     group whose core set holds n, K = ceil(gamma * N). */
void oracle_top_by_count(const int32_t *counts, int32_t N, int32_t K, int32_t *S)
{
    entry_t *ord = (entry_t *)malloc(sizeof(entry_t) * (size_t)(N > 0 ? N : 1));
    for (int32_t n = 0; n < N; ++n) { ord[n].key = (uint32_t)counts[n]; ord[n].idx = n; }
    qsort(ord, (size_t)N, sizeof(entry_t), cmp_entry_desc);   /* full sort */
    for (int32_t i = 0; i < K; ++i) S[i] = ord[i].idx;
    qsort(S, (size_t)K, sizeof(int32_t), cmp_i32_asc);
    free(ord);
}

/* counts[n] += 1 for every member of a core set (one sentence of a semantic group). */
void oracle_counts_add_set(int32_t *counts, const int32_t *S, int32_t K)
{
    for (int32_t i = 0; i < K; ++i) counts[S[i]] += 1;
}

/* Core-neuron similarity of two sets (Insight-2: "the ratio of identical neurons to the total
 * number of neurons involved"): out[0] = |A and B|, out[1] = |A or B|.  Quadratic on purpose. */
void oracle_core_similarity(const int32_t *A, int32_t KA, const int32_t *B, int32_t KB, int32_t *out)
{
    int32_t shared = 0;
    for (int32_t i = 0; i < KA; ++i)
        for (int32_t j = 0; j < KB; ++j)
            if (A[i] == B[j]) { ++shared; break; }
    out[0] = shared;
    out[1] = KA + KB - shared;
}

/* Nearest centroid (similarity-guided prediction: the group of an input is the cluster its
 * feature vector falls into; K-Means assigns a point to the centroid at the smallest Euclidean
 * distance).  centroids: [G][D]; equal distances go to the lower group.  Squared distances in
 * double; dist2 (may be NULL) receives them. */
int32_t oracle_nearest_centroid(const float *centroids, int32_t G, int32_t D, const float *v, double *dist2)
{
    int32_t best = 0;
    double best_d = 0.0;
    for (int32_t g = 0; g < G; ++g) {
        double s = 0.0;
        for (int32_t i = 0; i < D; ++i) {
            double t = (double)v[i] - (double)centroids[(size_t)g * D + i];
            s += t * t;
        }
        if (dist2) dist2[g] = s;
        if (g == 0 || s < best_d) { best = g; best_d = s; }
    }
    return best;
}

/* Updating a deployed set in place (Fig. 1: the set may be updated after the stability
 * estimate; the paper gives no rule, this is the mechanism).  slot_neuron[K] says which neuron
 * each row of the compacted buffers holds (any order).  Rows whose neuron is not in S_new
 * (ascending) are reassigned, in ascending slot order, to the members of S_new not held yet, in
 * ascending neuron order.  Writes the changed (slot, neuron) pairs and updates slot_neuron;
 * returns their number. */
int32_t oracle_set_delta(int32_t *slot_neuron, int32_t K, const int32_t *S_new, int32_t *slots, int32_t *neurons)
{
    int32_t n_leave = 0, n_enter = 0;
    for (int32_t p = 0; p < K; ++p) {
        int keep = 0;
        for (int32_t j = 0; j < K; ++j) if (S_new[j] == slot_neuron[p]) { keep = 1; break; }
        if (!keep) slots[n_leave++] = p;
    }
    for (int32_t j = 0; j < K; ++j) {
        int held = 0;
        for (int32_t p = 0; p < K; ++p) if (slot_neuron[p] == S_new[j]) { held = 1; break; }
        if (!held) neurons[n_enter++] = S_new[j];
    }
    /* both lists have the same length because both sets have K distinct members */
    for (int32_t i = 0; i < n_leave; ++i) slot_neuron[slots[i]] = neurons[i];
    return n_leave;
}
