/*
 * DaSS reference oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, fp64 CPU statement of what the DaSS hot path computes
 * (Dependency-aware Semi-structured Sparsity, arXiv 2405.01943).  It exists so
 * that tests and the benchmark's CPU-baseline leg have something obviously
 * correct to compare the CUDA library against.  It shares no code with the CUDA
 * library and the CUDA library never calls it.
 *
 * Every function is the definition written out: no blocking, no fusion, no
 * reordering, no SIMD, no BLAS.  OpenMP is used only to run independent
 * neurons / rows / columns on several cores; every output element is still
 * produced by one thread in the textbook order.
 *
 * Inputs are passed as `float` arrays: both bf16 and fp32 stored values are
 * exactly representable in a float, so the Python wrapper widens bf16 tensors
 * without rounding.  All arithmetic on them is done in double.
 *
 * Notation (paper, Section 2.2 and Section 3): T tokens, d = d_hidden,
 * I = d_int.  X is [T x d]; Wg, Wu are the transposed gate / up projections
 * W(1)^T, W(2)^T of shape [I x d]; Wd is W(3)^T of shape [d x I]; all row-major.
 *
 * Pins (what each function is checked against, see tests/test_oracle_*.py):
 *   activations      closed forms, odd-part identities, torch fp64 functional
 *   feature_sumsq    numpy sum of squares, linearity, known vectors
 *   calib_sumsq      numpy matmul special case, one-hot closed forms,
 *                    batching / linearity / power-of-two scaling invariants
 *   scale, score_nm  exact-rational brute force over all N:M subsets,
 *                    hand-worked fixtures, Wanda (Eq. 1) reduction for Eq. 5,
 *                    magnitude-only reduction for alpha = 0 / equal norms
 *   select_unstructured   monotonicity invariants of the dependency metric
 *   compress_nm      round trip to the pruned matrix, metadata well-formedness
 *   round_bf16       torch's float32 -> bfloat16 conversion, hand-picked ties
 *   mlp_forward      hand-worked fixture, numpy float64 matmul composition,
 *                    identity / one-hot down projections, linearity in Wd
 *   pack_mask        bit-by-bit re-derivation in the tests
 * The absolute layout of mask words / metadata and the tie-break are readings
 * of this library (the paper is silent): those are "parity unpinned" in the
 * sense that only this project's documents fix them.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_ACT_SILU = 0, ORACLE_ACT_GELU_TANH = 1, ORACLE_ACT_RELU = 2 };
enum { ORACLE_AXIS_ROWS = 0, ORACLE_AXIS_COLS = 1 };

/* ---- activation, Eq. 2 (sigma) and Section 2.2 (Swish / GeLU / ReLU) ------ */

double dass_oracle_act(int act, double g)
{
    if (act == ORACLE_ACT_SILU) {
        /* Swish with beta = 1: g * sigmoid(g) */
        return g / (1.0 + exp(-g));
    }
    if (act == ORACLE_ACT_GELU_TANH) {
        /* tanh form of GeLU: 0.5 g (1 + tanh( sqrt(2/pi) (g + 0.044715 g^3) )) */
        const double c = sqrt(2.0 / M_PI);
        return 0.5 * g * (1.0 + tanh(c * (g + 0.044715 * g * g * g)));
    }
    if (act == ORACLE_ACT_RELU) {
        return g > 0.0 ? g : 0.0;
    }
    return NAN;
}

/* ---- stage (a): Eq. 2 followed by the per-neuron sum of squares -----------
 * sumsq[i] += sum_t ( act(x_t . Wg[i,:]) * (x_t . Wu[i,:]) )^2
 * (the squared l2 norm of intermediate neuron i over all tokens; Section 3,
 * "Incorporating Dependency into Weight Importance"; the norm runs over all
 * tokens as for Eq. 1).  Accumulates, so that batches can be fed one by one. */
void dass_oracle_calib_sumsq(const float *X, int64_t T, int64_t ldx,
                             const float *Wg, const float *Wu,
                             int64_t I, int64_t d, int64_t ldw,
                             int act, double *sumsq)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < I; ++i) {
        double s = 0.0;
        for (int64_t t = 0; t < T; ++t) {
            double g = 0.0, u = 0.0;
            for (int64_t k = 0; k < d; ++k) {
                double x = (double)X[t * ldx + k];
                g += x * (double)Wg[i * ldw + k];
                u += x * (double)Wu[i * ldw + k];
            }
            double h = dass_oracle_act(act, g) * u;
            s += h * h;
        }
        sumsq[i] += s;
    }
}

/* Eq. 1's input-feature norms (Wanda, used by the paper for the attention projections):
 * sumsq[j] += sum_t X[t,j]^2, the squared l2 norm of feature j over all tokens. */
void dass_oracle_feature_sumsq(const float *X, int64_t T, int64_t d, int64_t ldx, double *sumsq)
{
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < d; ++j) {
        double s = 0.0;
        for (int64_t t = 0; t < T; ++t) {
            double x = (double)X[t * ldx + j];
            s += x * x;
        }
        sumsq[j] += s;
    }
}

/* One row of H = act(X Wg^T) * (X Wu^T) for a single token, all neurons.
 * Only used by tests that need H itself (Wanda reduction of Eq. 5). */
void dass_oracle_glu_row(const float *x, const float *Wg, const float *Wu,
                         int64_t I, int64_t d, int64_t ldw, int act, double *h)
{
    for (int64_t i = 0; i < I; ++i) {
        double g = 0.0, u = 0.0;
        for (int64_t k = 0; k < d; ++k) {
            g += (double)x[k] * (double)Wg[i * ldw + k];
            u += (double)x[k] * (double)Wu[i * ldw + k];
        }
        h[i] = dass_oracle_act(act, g) * u;
    }
}

/* Round a double to the nearest bf16 value (8 significant bits, float's exponent
 * range), ties to even; the result is returned as a double.  Written out from
 * the format's definition: find the binade, scale so that one unit in the last
 * place is 1, round to the nearest integer with ties to even, scale back. */
double dass_oracle_round_bf16(double v)
{
    if (v == 0.0 || isnan(v) || isinf(v)) return v;
    int e;
    (void)frexp(v, &e);            /* |v| = f * 2^e with f in [0.5, 1)  ->  binade exponent e - 1 */
    int ex = e - 1;
    if (ex < -126) ex = -126;      /* subnormal range: fixed spacing 2^-133 */
    const double ulp = ldexp(1.0, ex - 7);
    const double r = nearbyint(v / ulp) * ulp;      /* default rounding mode: to nearest, ties to even */
    if (fabs(r) >= ldexp(1.0, 128)) return v > 0 ? INFINITY : -INFINITY;
    return r;
}

/* ---- the pruned layer's forward pass, Eq. 2 then Eq. 3 ---------------------
 * y_t = act(x_t Wg^T) * (x_t Wu^T),  z_t = y_t Wd^T, for every token t, with whatever
 * (pruned) weights are passed in.  h_round = 1 rounds every y to bf16 before Eq. 3,
 * which is what a model whose activations are stored in bf16 does between the two
 * projections; h_round = 0 keeps y in double.  Z is [T x d] (ld = d); H, when not
 * NULL, receives y as used by Eq. 3, [T x I] (ld = I). */
void dass_oracle_mlp_forward(const float *X, int64_t T, int64_t ldx,
                             const float *Wg, const float *Wu, int64_t I, int64_t d, int64_t ldw,
                             const float *Wd, int64_t ldd, int act, int h_round,
                             double *Z, double *H)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t t = 0; t < T; ++t) {
        double *y = (double *)malloc((size_t)I * sizeof(double));
        for (int64_t i = 0; i < I; ++i) {
            double g = 0.0, u = 0.0;
            for (int64_t k = 0; k < d; ++k) {
                double x = (double)X[t * ldx + k];
                g += x * (double)Wg[i * ldw + k];
                u += x * (double)Wu[i * ldw + k];
            }
            double h = dass_oracle_act(act, g) * u;
            y[i] = h_round ? dass_oracle_round_bf16(h) : h;
            if (H) H[t * I + i] = y[i];
        }
        for (int64_t n = 0; n < d; ++n) {
            double z = 0.0;
            for (int64_t i = 0; i < I; ++i) z += y[i] * (double)Wd[n * ldd + i];
            Z[t * d + n] = z;
        }
        free(y);
    }
}

/* norm[i] = sqrt(sumsq[i]), stored for the scoring stage as a float. */
void dass_oracle_norm(const double *sumsq, int64_t I, float *norm)
{
    for (int64_t i = 0; i < I; ++i) norm[i] = (float)sqrt(sumsq[i]);
}

/* ---- ||y||^alpha of Eq. 4 (alpha = 1 gives the factor of Eq. 5) -----------
 * The value is rounded to float exactly once, by a recipe made only of
 * correctly rounded IEEE operations for alpha in {0, 1/4, 1/2, 3/4, 1}, so any
 * IEEE machine reproduces it bit for bit.  0^0 := 1. */
float dass_oracle_scale(float norm, float alpha)
{
    double n = (double)norm;
    if (alpha == 0.0f) return 1.0f;
    if (alpha == 1.0f) return norm;
    if (alpha == 0.5f) return (float)sqrt(n);
    if (alpha == 0.25f) return (float)sqrt(sqrt(n));
    if (alpha == 0.75f) {
        double r = sqrt(n);
        double q = sqrt(r);
        double p = r * q;
        return (float)p;
    }
    return (float)pow(n, (double)alpha);
}

/* ---- stage (b): Eq. 4 / Eq. 5 score and N:M selection ---------------------
 * score(r,c) = |W[r,c]| * scale(norm[k], alpha), k = r if norm_axis = ROWS,
 * c if norm_axis = COLS, taken as the exact real product (a float times a
 * float fits a double without rounding).
 * Groups are m consecutive elements along group_axis (ROWS: rows r..r+m-1 of
 * one column; COLS: columns c..c+m-1 of one row).  Inside a group the elements
 * are put in the total order "higher score first, then lower index first" and
 * the first n_keep are kept (Section 3, "Pruning Granularity": sort, prune the
 * lowest; "Extension to N:M Sparsity").
 *   gate / up (Eq. 4): W = [I x d], norm_axis = ROWS, group_axis = ROWS
 *   down      (Eq. 5): W = [d x I], norm_axis = COLS, group_axis = COLS, alpha = 1
 * mask is one byte per element (1 = kept), row-major [rows x cols].
 * W_pruned (optional) is [rows x cols] dense, survivors copied, others +0.
 * Returns 0, or -1 on a shape the definition does not cover. */
typedef struct { double score; int idx; } oracle_item;

static int item_before(const oracle_item *a, const oracle_item *b)
{
    if (a->score > b->score) return 1;
    if (a->score < b->score) return 0;
    return a->idx < b->idx;
}

static void sort_items(oracle_item *it, int n)
{
    /* insertion sort into the total order; n is a group size */
    for (int a = 1; a < n; ++a) {
        oracle_item key = it[a];
        int b = a - 1;
        while (b >= 0 && item_before(&key, &it[b])) {
            it[b + 1] = it[b];
            --b;
        }
        it[b + 1] = key;
    }
}

static double score_at(const float *W, int64_t ld, int64_t r, int64_t c,
                       const float *norm, int norm_axis, float alpha)
{
    float nk = norm[norm_axis == ORACLE_AXIS_ROWS ? r : c];
    double scale = (double)dass_oracle_scale(nk, alpha);
    return fabs((double)W[r * ld + c]) * scale;
}

int dass_oracle_score_nm(const float *W, int64_t rows, int64_t cols, int64_t ld,
                         const float *norm, int norm_axis, float alpha,
                         int n_keep, int m, int group_axis,
                         uint8_t *mask, float *W_pruned)
{
    if (m < 2 || m > 64 || n_keep < 1 || n_keep >= m) return -1;
    int64_t extent = (group_axis == ORACLE_AXIS_ROWS) ? rows : cols;
    if (extent % m != 0) return -1;
    memset(mask, 0, (size_t)(rows * cols));

    if (group_axis == ORACLE_AXIS_COLS) {
#pragma omp parallel for schedule(static)
        for (int64_t r = 0; r < rows; ++r) {
            oracle_item it[64];
            for (int64_t c0 = 0; c0 < cols; c0 += m) {
                for (int p = 0; p < m; ++p) {
                    it[p].score = score_at(W, ld, r, c0 + p, norm, norm_axis, alpha);
                    it[p].idx = p;
                }
                sort_items(it, m);
                for (int q = 0; q < n_keep; ++q) mask[r * cols + c0 + it[q].idx] = 1;
            }
        }
    } else {
#pragma omp parallel for schedule(static)
        for (int64_t c = 0; c < cols; ++c) {
            oracle_item it[64];
            for (int64_t r0 = 0; r0 < rows; r0 += m) {
                for (int p = 0; p < m; ++p) {
                    it[p].score = score_at(W, ld, r0 + p, c, norm, norm_axis, alpha);
                    it[p].idx = p;
                }
                sort_items(it, m);
                for (int q = 0; q < n_keep; ++q) mask[(r0 + it[q].idx) * cols + c] = 1;
            }
        }
    }
    if (W_pruned) {
        for (int64_t r = 0; r < rows; ++r)
            for (int64_t c = 0; c < cols; ++c)
                W_pruned[r * cols + c] = mask[r * cols + c] ? W[r * ld + c] : 0.0f;
    }
    return 0;
}

/* ---- unstructured selection at sparsity s (Section 3, "Pruning Granularity")
 * compare_axis = ROWS: the comparison group is a whole column (all rows at one
 * input j: "input-balanced", used for gate / up); COLS: a whole row
 * ("output-balanced", used for down).  The floor(s * size) lowest elements in
 * the total order are pruned. */
int dass_oracle_select_unstructured(const float *W, int64_t rows, int64_t cols, int64_t ld,
                                    const float *norm, int norm_axis, float alpha,
                                    double sparsity, int compare_axis, uint8_t *mask)
{
    if (!(sparsity >= 0.0 && sparsity < 1.0)) return -1;
    int64_t size = (compare_axis == ORACLE_AXIS_ROWS) ? rows : cols;
    int64_t lines = (compare_axis == ORACLE_AXIS_ROWS) ? cols : rows;
    int64_t n_prune = (int64_t)floor(sparsity * (double)size);
    int64_t n_keep = size - n_prune;
    memset(mask, 0, (size_t)(rows * cols));
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t l = 0; l < lines; ++l) {
        oracle_item *it = (oracle_item *)malloc(sizeof(oracle_item) * (size_t)size);
        for (int64_t p = 0; p < size; ++p) {
            int64_t r = (compare_axis == ORACLE_AXIS_ROWS) ? p : l;
            int64_t c = (compare_axis == ORACLE_AXIS_ROWS) ? l : p;
            it[p].score = score_at(W, ld, r, c, norm, norm_axis, alpha);
            it[p].idx = (int)p;
        }
        sort_items(it, (int)size);
        for (int64_t q = 0; q < n_keep; ++q) {
            int64_t p = it[q].idx;
            int64_t r = (compare_axis == ORACLE_AXIS_ROWS) ? p : l;
            int64_t c = (compare_axis == ORACLE_AXIS_ROWS) ? l : p;
            mask[r * cols + c] = 1;
        }
        free(it);
    }
    return 0;
}

/* ---- packed mask: one bit per weight, row-major, rows padded to whole words;
 * bit (c % 32) of word r * ceil(cols/32) + c / 32 is 1 iff (r,c) is kept. */
void dass_oracle_pack_mask(const uint8_t *mask, int64_t rows, int64_t cols, uint32_t *bits)
{
    int64_t wpr = (cols + 31) / 32;
    memset(bits, 0, (size_t)(rows * wpr) * sizeof(uint32_t));
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c)
            if (mask[r * cols + c]) bits[r * wpr + c / 32] |= (uint32_t)1 << (c % 32);
}

/* ---- N:M compressed form: values + metadata -------------------------------
 * values: the n_keep survivors of every group, in index order.
 *   group_axis = COLS: [rows x cols*n_keep/m]; ROWS: [rows*n_keep/m x cols].
 * metadata: a field of `bpg` bits per group.  For 2:4 the field is the nibble
 * pos_lo | pos_hi << 2 (positions 0..3 of the two survivors, pos_lo < pos_hi).
 * For every other n:m it is the m-bit keep mask of the group (bit p = position
 * p kept).  Fields are packed LSB first along the columns; one "line" of
 * fields (COLS: a row, cols/m groups; ROWS: a row group, cols groups) is padded
 * to whole 32-bit words.  m must divide 32 (so a field never straddles words).
 * Returns 0, or -1 if a group does not hold exactly n_keep survivors. */
int dass_oracle_compress_nm(const float *W, const uint8_t *mask,
                            int64_t rows, int64_t cols, int64_t ld,
                            int n_keep, int m, int group_axis,
                            float *values, uint32_t *meta)
{
    if (m < 2 || m > 32 || 32 % m != 0 || n_keep < 1 || n_keep >= m) return -1;
    int two_four = (n_keep == 2 && m == 4);
    int bpg = two_four ? 4 : m;
    int fpw = 32 / bpg; /* fields per word */
    int64_t extent = (group_axis == ORACLE_AXIS_ROWS) ? rows : cols;
    if (extent % m != 0) return -1;
    int64_t lines = (group_axis == ORACLE_AXIS_COLS) ? rows : rows / m;
    int64_t fields_per_line = (group_axis == ORACLE_AXIS_COLS) ? cols / m : cols;
    int64_t wpl = (fields_per_line + fpw - 1) / fpw;
    memset(meta, 0, (size_t)(lines * wpl) * sizeof(uint32_t));
    int64_t vcols = (group_axis == ORACLE_AXIS_COLS) ? cols * n_keep / m : cols;

    for (int64_t l = 0; l < lines; ++l) {
        for (int64_t f = 0; f < fields_per_line; ++f) {
            int pos[32];
            int kept = 0;
            uint32_t keepmask = 0;
            for (int p = 0; p < m; ++p) {
                int64_t r = (group_axis == ORACLE_AXIS_COLS) ? l : l * m + p;
                int64_t c = (group_axis == ORACLE_AXIS_COLS) ? f * m + p : f;
                if (mask[r * cols + c]) {
                    if (kept < 32) pos[kept] = p;
                    ++kept;
                    keepmask |= (uint32_t)1 << p;
                    int64_t vr = (group_axis == ORACLE_AXIS_COLS) ? l : l * n_keep + (kept - 1);
                    int64_t vc = (group_axis == ORACLE_AXIS_COLS) ? f * n_keep + (kept - 1) : f;
                    if (kept <= n_keep) values[vr * vcols + vc] = W[r * ld + c];
                }
            }
            if (kept != n_keep) return -1;
            uint32_t field = two_four ? ((uint32_t)pos[0] | ((uint32_t)pos[1] << 2)) : keepmask;
            meta[l * wpl + f / fpw] |= field << (bpg * (int)(f % fpw));
        }
    }
    return 0;
}
