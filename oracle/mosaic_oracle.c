/*
 * TEST INFRASTRUCTURE - NOT PART OF THE PRODUCT.
 *
 * A plain, slow, scalar CPU statement of what the hot path of Mosaic's
 * composite projection pruning computes.  It exists so that the CUDA library
 * can be checked element by element against something a reader can verify by
 * eye against the paper.  It shares no source, header, table or helper with
 * the CUDA library and must never be called from the product path.
 *
 * Every function is the definition written out: loops in index order, fp64
 * for every accumulation, one fp32 multiply for the score, a full sort for
 * every selection.  OpenMP is used only across independent outputs (columns,
 * rows, units), so threading never changes a result.
 *
 * Notation follows the paper (Section 3.1-3.3):
 *   W      one projection's weights, row-major [rows = out, cols = in]
 *   X      calibration activations feeding that projection, row-major [T, cols]
 *   norm_j l2 norm of column j of X                         (the ||A||_2 of Eq. 5)
 *   w_ij   = norm_j * |W_ij|                                (Eq. 5, Algorithm 1)
 *   C      = rows*cols                                      (Algorithm 1)
 *   O      = #{ w_ij > alpha * mean(w) }                    (Eq. 6, Algorithm 1)
 *   R      = 100 * O / C                                    (Algorithm 1)
 *
 * Parity with the authors' own program is unpinned: the paper prints no
 * worked numeric example and leaves normalize(R_LLM) (Algorithm 1's return)
 * undefined; oracle_allocate_sparsity states the reading taken.  Everything
 * else here is pinned by the CPU tests against brute force in exact rational
 * arithmetic, closed forms and invariants.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };

/* Element idx of a buffer of the given type, widened exactly to fp32. */
static float load_elem(const void *base, int64_t idx, int dtype)
{
    if (dtype == ORACLE_F32)
        return ((const float *)base)[idx];
    uint32_t bits = (uint32_t)((const uint16_t *)base)[idx] << 16; /* bf16 = top half of fp32 */
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

static uint32_t float_bits(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    return u;
}

/* Eq. 5 for one element: a single round-to-nearest fp32 multiply. */
static float weight_metric(float norm_j, float w)
{
    float a = fabsf(w);
    float s = norm_j * a; /* built with -ffp-contract=off: never fused or widened */
    return s;
}

/*
 * Ordering key of a score.  Scores are >= +0, so their fp32 bit patterns
 * order like the values; a NaN score (non-finite input, not covered by the
 * paper) is given the largest key so it is selected last.
 */
static uint32_t score_key(float s)
{
    return (s != s) ? 0xFFFFFFFFu : float_bits(s);
}

/* ------------------------------------------------------------------ */
/* Activation norms: the ||A||_2 term of Eq. 5 (Section 3.3, RC 3-4).  */
/* ------------------------------------------------------------------ */

/*
 * sumsq[j] += sum_t X[t,j]^2: for every column j the squares are added one by
 * one in t order, in fp64 (each square of a bf16/fp32 value is exact in fp64).
 * Columns are independent; they are walked a block at a time only so that
 * memory is read along rows.
 */
void oracle_act_sumsq(const void *X, int64_t tokens, int64_t cols, int64_t ldx,
                      int dtype, double *sumsq)
{
    const int64_t block = 64;
#pragma omp parallel for schedule(static)
    for (int64_t j0 = 0; j0 < cols; j0 += block) {
        int64_t j1 = j0 + block < cols ? j0 + block : cols;
        for (int64_t t = 0; t < tokens; ++t)
            for (int64_t j = j0; j < j1; ++j) {
                double x = (double)load_elem(X, t * ldx + j, dtype);
                sumsq[j] = sumsq[j] + x * x;
            }
    }
}

/* norm[j] = (float) sqrt(sumsq[j]) */
void oracle_norm_finalize(const double *sumsq, int64_t cols, float *norms)
{
    for (int64_t j = 0; j < cols; ++j)
        norms[j] = (float)sqrt(sumsq[j]);
}

/*
 * Certification of the norms of one X against summation order: ok[j] = 1 iff
 * the fp32 norm of column j is the same for the sequential fp64 sum, for an
 * extended-precision (long double) sum, and for that sum perturbed by
 * +-tokens*2^-52 relative - i.e. no admissible fp64 summation order can
 * change the rounded result.  Returns the number of columns NOT certified.
 */
int64_t oracle_norm_certify(const void *X, int64_t tokens, int64_t cols, int64_t ldx,
                            int dtype, uint8_t *ok)
{
    int64_t bad = 0;
    double eps = (double)tokens * ldexp(1.0, -52);
#pragma omp parallel for schedule(static) reduction(+ : bad)
    for (int64_t j = 0; j < cols; ++j) {
        double s = 0.0;
        long double e = 0.0L;
        for (int64_t t = 0; t < tokens; ++t) {
            double x = (double)load_elem(X, t * ldx + j, dtype);
            s = s + x * x;
            e = e + (long double)x * (long double)x;
        }
        float n0 = (float)sqrt(s);
        float n1 = (float)sqrt((double)e);
        float n2 = (float)sqrt((double)e * (1.0 - eps));
        float n3 = (float)sqrt((double)e * (1.0 + eps));
        int good = (float_bits(n0) == float_bits(n1)) && (float_bits(n1) == float_bits(n2)) &&
                   (float_bits(n1) == float_bits(n3));
        if (ok)
            ok[j] = (uint8_t)good;
        bad += good ? 0 : 1;
    }
    return bad;
}

/* ------------------------------------------------------------------ */
/* Weight metric, Eq. 5 / Algorithm 1, materialised.                    */
/* ------------------------------------------------------------------ */
void oracle_score(const void *W, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                  const float *norms, float *score /* [rows, cols] */)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols; ++j)
            score[i * cols + j] = weight_metric(norms[j], load_elem(W, i * ldw + j, dtype));
}

/* ------------------------------------------------------------------ */
/* Projection outlier statistic, Eq. 6 / Algorithm 1.                  */
/* ------------------------------------------------------------------ */
/*
 * sum   = sum_i sum_j (double) w_ij          (row-major order, fp64)
 * tau   = (double)alpha * (sum / C)          (kept in fp64)
 * O     = #{ (double) w_ij > tau }           (strict)
 * certified = 1 iff O is unchanged when tau is moved by +-C*2^-52 relative,
 *             i.e. no admissible fp64 summation order changes the count.
 */
void oracle_outlier_ratio(const void *W, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                          const float *norms, float alpha, int64_t *outlier_count,
                          double *score_sum, double *ratio_percent, int *certified)
{
    double sum = 0.0;
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols; ++j)
            sum = sum + (double)weight_metric(norms[j], load_elem(W, i * ldw + j, dtype));

    double C = (double)(rows * cols);
    double mean = sum / C;
    double tau = (double)alpha * mean;
    double eps = C * ldexp(1.0, -52);
    double tau_lo = tau * (1.0 - eps), tau_hi = tau * (1.0 + eps);

    int64_t O = 0, O_lo = 0, O_hi = 0;
#pragma omp parallel for schedule(static) reduction(+ : O, O_lo, O_hi)
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols; ++j) {
            double s = (double)weight_metric(norms[j], load_elem(W, i * ldw + j, dtype));
            O += (s > tau);
            O_lo += (s > tau_lo);
            O_hi += (s > tau_hi);
        }
    if (outlier_count) *outlier_count = O;
    if (score_sum) *score_sum = sum;
    if (ratio_percent) *ratio_percent = 100.0 * (double)O / C;
    if (certified) *certified = (O == O_lo && O == O_hi);
}

/*
 * Layer outlier distribution (Eq. 3-4, the layer-pruning baseline of Section 4.1.3): the same
 * predicate with ONE threshold for a whole group of matrices (the projections of a layer):
 *   sum   = sum over the matrices, in list order, of their row-major fp64 score sums
 *   tau   = (double)alpha * (sum / C),   C = total number of elements of the group
 *   O_g   = #{ (double) w_ij > tau } in matrix g
 * counts[g] receives O_g (their total is the layer's O).  certified = 1 iff the total count is
 * unchanged when tau is moved by +-C*2^-52 relative.
 */
void oracle_outlier_ratio_group(const void *const *Ws, const int64_t *rows, const int64_t *cols,
                                const int64_t *ldws, int dtype, const float *const *norms, int n_mat,
                                float alpha, int64_t *counts, double *score_sum, double *ratio_percent,
                                int *certified)
{
    double sum = 0.0, C = 0.0;
    for (int g = 0; g < n_mat; ++g) {
        for (int64_t i = 0; i < rows[g]; ++i)
            for (int64_t j = 0; j < cols[g]; ++j)
                sum = sum + (double)weight_metric(norms[g][j], load_elem(Ws[g], i * ldws[g] + j, dtype));
        C += (double)(rows[g] * cols[g]);
    }
    double mean = sum / C;
    double tau = (double)alpha * mean;
    double eps = C * ldexp(1.0, -52);
    double tau_lo = tau * (1.0 - eps), tau_hi = tau * (1.0 + eps);
    int64_t total = 0, total_lo = 0, total_hi = 0;
    for (int g = 0; g < n_mat; ++g) {
        int64_t O = 0, O_lo = 0, O_hi = 0;
#pragma omp parallel for schedule(static) reduction(+ : O, O_lo, O_hi)
        for (int64_t i = 0; i < rows[g]; ++i)
            for (int64_t j = 0; j < cols[g]; ++j) {
                double s = (double)weight_metric(norms[g][j], load_elem(Ws[g], i * ldws[g] + j, dtype));
                O += (s > tau);
                O_lo += (s > tau_lo);
                O_hi += (s > tau_hi);
            }
        if (counts) counts[g] = O;
        total += O;
        total_lo += O_lo;
        total_hi += O_hi;
    }
    if (score_sum) *score_sum = sum;
    if (ratio_percent) *ratio_percent = 100.0 * (double)total / C;
    if (certified) *certified = (total == total_lo && total == total_hi);
}

/* ------------------------------------------------------------------ */
/* normalize(R_LLM) + Projection Planner (Algorithm 1; Section 3.3      */
/* component 8; Eq. 1-2).                                              */
/* ------------------------------------------------------------------ */
/*
 * The paper fixes only the properties: the targets average to p (Eq. 1-2,
 * Projection Planner), and a projection with more outliers is pruned less
 * (Section 3.1).  Reading taken: min-max normalise the ranks R_q = 100*O_q/C_q
 * to r_q in [0,1]; give each projection the deviation d_q = 2*lambda*r_q;
 * s_q = p + mean(d) - d_q.  Then mean(s) = p, s decreases in R, and
 * max(s)-min(s) = 2*lambda.  mode bit 0: 0 normalises over all N*M entries, 1
 * separately over the N entries of each projection category m.  mode bit 1:
 * the mean in "targets average to p" weighs every projection by its number of
 * parameters C_q (mean(d) = sum C_q d_q / sum C_q), so that the pruned share
 * of all parameters of the group is p; without it the mean is the plain one of
 * Eq. 1-2.
 * s is clamped to [0, 1 - 1/cols_q]; k_q = floor(s_q * cols_q) weights are
 * removed from every row.  Returns 0, or 1 if any clamp was applied.
 * mode bit 2 (clamp and redistribute): where a clamp fires, the mean of the
 * targets would leave p; the clamped targets then stay on their bounds and all
 * others are shifted by one common amount t that brings the (plain or
 * weighted) mean of each group back to p - repeated while the shift pushes
 * further targets over a bound (at most one round per target).  With b_q the
 * unclamped target:  t = (p*W - sum_clamped w_q s_q - sum_free w_q b_q) / sum_free w_q.
 * Returns 1 only if p cannot be reached at all (every target of a group on a bound).
 */
int oracle_allocate_sparsity(const int64_t *outlier_counts, const int64_t *numels,
                             const int64_t *cols, int n_layers, int n_proj, double p,
                             double lambda, int mode, double *sparsity, int64_t *k_out)
{
    int total = n_layers * n_proj;
    int clamped = 0;
    double *R = (double *)malloc(sizeof(double) * (size_t)total);
    for (int q = 0; q < total; ++q)
        R[q] = 100.0 * (double)outlier_counts[q] / (double)numels[q];

    int per_category = mode & 1, weighted = (mode >> 1) & 1, redistribute = (mode >> 2) & 1;
    int n_groups = per_category ? n_proj : 1;
    for (int g = 0; g < n_groups; ++g) {
        /* members of this normalisation group, in q order */
        int first = per_category ? g : 0;
        int step = per_category ? n_proj : 1;
        int count = per_category ? n_layers : total;

        double lo = R[first], hi = R[first];
        for (int c = 0, q = first; c < count; ++c, q += step) {
            if (R[q] < lo) lo = R[q];
            if (R[q] > hi) hi = R[q];
        }
        if (hi == lo) {
            for (int c = 0, q = first; c < count; ++c, q += step)
                sparsity[q] = p;
            continue;
        }
        double dsum = 0.0, wsum = 0.0;
        for (int c = 0, q = first; c < count; ++c, q += step) {
            double r = (R[q] - lo) / (hi - lo);
            double d = 2.0 * lambda * r;
            double w = weighted ? (double)numels[q] : 1.0;
            dsum = dsum + w * d;
            wsum = wsum + w;
        }
        double dbar = dsum / wsum;
        for (int c = 0, q = first; c < count; ++c, q += step) {
            double r = (R[q] - lo) / (hi - lo);
            double d = 2.0 * lambda * r;
            sparsity[q] = (p + dbar) - d;
        }
    }
    if (redistribute) {
        uint8_t *fixed = (uint8_t *)malloc((size_t)total);
        double *base = (double *)malloc(sizeof(double) * (size_t)total);
        for (int g = 0; g < n_groups; ++g) {
            int first = per_category ? g : 0;
            int step = per_category ? n_proj : 1;
            int count = per_category ? n_layers : total;
            int any = 0;
            for (int c = 0, q = first; c < count; ++c, q += step) {
                double smax = 1.0 - 1.0 / (double)cols[q];
                base[q] = sparsity[q];
                fixed[q] = 0;
                if (sparsity[q] < 0.0 || sparsity[q] > smax) any = 1;
            }
            if (!any) continue;                       /* nothing to clamp: the targets stand as they are */
            for (int round = 0; round < count; ++round) {
                double wtot = 0.0, wfree = 0.0, sfixed = 0.0, sfree = 0.0;
                for (int c = 0, q = first; c < count; ++c, q += step) {
                    double w = weighted ? (double)numels[q] : 1.0;
                    wtot = wtot + w;
                    if (fixed[q]) sfixed = sfixed + w * sparsity[q];
                    else { wfree = wfree + w; sfree = sfree + w * base[q]; }
                }
                if (wfree == 0.0) { clamped = 1; break; }   /* every target on a bound: p is out of reach */
                double t = (p * wtot - sfixed - sfree) / wfree;
                int newly = 0;
                for (int c = 0, q = first; c < count; ++c, q += step) {
                    if (fixed[q]) continue;
                    double smax = 1.0 - 1.0 / (double)cols[q];
                    double v = base[q] + t;
                    if (v < 0.0) { sparsity[q] = 0.0; fixed[q] = 1; newly = 1; }
                    else if (v > smax) { sparsity[q] = smax; fixed[q] = 1; newly = 1; }
                    else sparsity[q] = v;
                }
                if (!newly) break;
            }
        }
        free(fixed);
        free(base);
        for (int q = 0; q < total; ++q)
            k_out[q] = (int64_t)floor(sparsity[q] * (double)cols[q]);
        free(R);
        return clamped;
    }
    for (int q = 0; q < total; ++q) {
        double smax = 1.0 - 1.0 / (double)cols[q];
        if (sparsity[q] < 0.0) { sparsity[q] = 0.0; clamped = 1; }
        if (sparsity[q] > smax) { sparsity[q] = smax; clamped = 1; }
        k_out[q] = (int64_t)floor(sparsity[q] * (double)cols[q]);
    }
    free(R);
    return clamped;
}

/* ------------------------------------------------------------------ */
/* Unstructured projection pruning (Section 4.1.3: "masked by setting  */
/* their weights to zero"; Section 2.3: the lowest-ranking parameters   */
/* are removed), per output row.                                        */
/* ------------------------------------------------------------------ */
typedef struct { uint32_t key; int64_t idx; } keyed_t;

static int keyed_cmp(const void *a, const void *b)
{
    const keyed_t *x = (const keyed_t *)a, *y = (const keyed_t *)b;
    if (x->key != y->key) return x->key < y->key ? -1 : 1;
    if (x->idx != y->idx) return x->idx < y->idx ? -1 : 1;
    return 0;
}

/*
 * In every row the k entries that come first under (w_ij ascending, j
 * ascending) are set to +0; all others keep their input bits.  mask (optional)
 * is [rows, ceil(cols/32)] words, bit j%32 of word j/32 = 1 for a kept entry,
 * padding bits 0.  W_out may be W_in.
 */
void oracle_prune_unstructured(const void *W_in, void *W_out, int64_t rows, int64_t cols,
                               int64_t ldw, int dtype, const float *norms, int64_t k,
                               uint32_t *mask)
{
    int64_t words = (cols + 31) / 32;
#pragma omp parallel
    {
        keyed_t *order = (keyed_t *)malloc(sizeof(keyed_t) * (size_t)cols);
        uint8_t *pruned = (uint8_t *)malloc((size_t)cols);
#pragma omp for schedule(static)
        for (int64_t i = 0; i < rows; ++i) {
            for (int64_t j = 0; j < cols; ++j) {
                order[j].key = score_key(weight_metric(norms[j], load_elem(W_in, i * ldw + j, dtype)));
                order[j].idx = j;
            }
            qsort(order, (size_t)cols, sizeof(keyed_t), keyed_cmp);
            memset(pruned, 0, (size_t)cols);
            for (int64_t r = 0; r < k; ++r)
                pruned[order[r].idx] = 1;

            if (mask)
                for (int64_t w = 0; w < words; ++w)
                    mask[i * words + w] = 0;
            for (int64_t j = 0; j < cols; ++j) {
                if (dtype == ORACLE_F32) {
                    uint32_t v = ((const uint32_t *)W_in)[i * ldw + j];
                    ((uint32_t *)W_out)[i * ldw + j] = pruned[j] ? 0u : v;
                } else {
                    uint16_t v = ((const uint16_t *)W_in)[i * ldw + j];
                    ((uint16_t *)W_out)[i * ldw + j] = pruned[j] ? (uint16_t)0 : v;
                }
                if (mask && !pruned[j])
                    mask[i * words + j / 32] |= (uint32_t)1 << (j % 32);
            }
        }
        free(order);
        free(pruned);
    }
}

/* ------------------------------------------------------------------ */
/* Structured projection pruning (Section 4.1.3: remove the            */
/* lowest-magnitude heads and channels; Section 2.3: structured         */
/* pruning removes whole data structures, leaving smaller dense         */
/* matrices).                                                           */
/* ------------------------------------------------------------------ */
/*
 * Unit scores.  A row unit u is the row_group consecutive rows
 * [u*row_group, (u+1)*row_group); a column unit likewise.  The score of a
 * unit is the fp64 sum, in row-major order, of w_ij over its elements,
 * rounded once to fp32.  norms == NULL means norm_j = 1 (pure magnitude).
 */
void oracle_unit_scores(const void *W, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                        const float *norms, int64_t row_group, int64_t col_group,
                        float *row_scores /* [rows/row_group] */,
                        float *col_scores /* [cols/col_group] */)
{
    int64_t n_ru = rows / row_group, n_cu = cols / col_group;
#pragma omp parallel for schedule(static)
    for (int64_t u = 0; u < n_ru; ++u) {
        double s = 0.0;
        for (int64_t i = u * row_group; i < (u + 1) * row_group; ++i)
            for (int64_t j = 0; j < cols; ++j)
                s = s + (double)weight_metric(norms ? norms[j] : 1.0f, load_elem(W, i * ldw + j, dtype));
        row_scores[u] = (float)s;
    }
#pragma omp parallel for schedule(static)
    for (int64_t v = 0; v < n_cu; ++v) {
        double s = 0.0;
        for (int64_t i = 0; i < rows; ++i)
            for (int64_t j = v * col_group; j < (v + 1) * col_group; ++j)
                s = s + (double)weight_metric(norms ? norms[j] : 1.0f, load_elem(W, i * ldw + j, dtype));
        col_scores[v] = (float)s;
    }
}

/*
 * Certification of the unit scores against summation order, in the manner of
 * oracle_norm_certify: row_ok[u] / col_ok[v] = 1 iff the fp32 score of the unit
 * is the same for the sequential fp64 sum above, for an extended-precision
 * (long double) sum, and for that sum moved by +-n*2^-52 relative, n being the
 * number of elements of the unit - i.e. no admissible order of the fp64
 * additions can change the rounded score.  Either output may be NULL.  Returns
 * the number of units NOT certified.
 */
static int unit_sum_certified(double s, long double e, double n_elems)
{
    double eps = n_elems * ldexp(1.0, -52);
    float f0 = (float)s;
    float f1 = (float)(double)e;
    float f2 = (float)((double)e * (1.0 - eps));
    float f3 = (float)((double)e * (1.0 + eps));
    return float_bits(f0) == float_bits(f1) && float_bits(f1) == float_bits(f2) &&
           float_bits(f1) == float_bits(f3);
}

int64_t oracle_unit_scores_certify(const void *W, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                                   const float *norms, int64_t row_group, int64_t col_group,
                                   uint8_t *row_ok /* [rows/row_group] or NULL */,
                                   uint8_t *col_ok /* [cols/col_group] or NULL */)
{
    int64_t n_ru = rows / row_group, n_cu = cols / col_group, bad = 0;
#pragma omp parallel for schedule(static) reduction(+ : bad)
    for (int64_t u = 0; u < n_ru; ++u) {
        double s = 0.0;
        long double e = 0.0L;
        for (int64_t i = u * row_group; i < (u + 1) * row_group; ++i)
            for (int64_t j = 0; j < cols; ++j) {
                double x = (double)weight_metric(norms ? norms[j] : 1.0f, load_elem(W, i * ldw + j, dtype));
                s = s + x;
                e = e + (long double)x;
            }
        int good = unit_sum_certified(s, e, (double)(row_group * cols));
        if (row_ok) row_ok[u] = (uint8_t)good;
        bad += good ? 0 : 1;
    }
#pragma omp parallel for schedule(static) reduction(+ : bad)
    for (int64_t v = 0; v < n_cu; ++v) {
        double s = 0.0;
        long double e = 0.0L;
        for (int64_t i = 0; i < rows; ++i)
            for (int64_t j = v * col_group; j < (v + 1) * col_group; ++j) {
                double x = (double)weight_metric(norms ? norms[j] : 1.0f, load_elem(W, i * ldw + j, dtype));
                s = s + x;
                e = e + (long double)x;
            }
        int good = unit_sum_certified(s, e, (double)(rows * col_group));
        if (col_ok) col_ok[v] = (uint8_t)good;
        bad += good ? 0 : 1;
    }
    return bad;
}

/*
 * Of n_units units, the (n_units - keep) that come first under (score
 * ascending, index ascending) are removed; keep_list receives the surviving
 * unit indices in ascending order.
 */
void oracle_rank_units(const float *scores, int64_t n_units, int64_t keep, int32_t *keep_list)
{
    keyed_t *order = (keyed_t *)malloc(sizeof(keyed_t) * (size_t)n_units);
    uint8_t *removed = (uint8_t *)calloc((size_t)n_units, 1);
    for (int64_t u = 0; u < n_units; ++u) {
        order[u].key = score_key(scores[u]);
        order[u].idx = u;
    }
    qsort(order, (size_t)n_units, sizeof(keyed_t), keyed_cmp);
    for (int64_t r = 0; r < n_units - keep; ++r)
        removed[order[r].idx] = 1;
    int64_t out = 0;
    for (int64_t u = 0; u < n_units; ++u)
        if (!removed[u])
            keep_list[out++] = (int32_t)u;
    free(order);
    free(removed);
}

/*
 * Dense compaction: Wc[a, b] = W[row(a), col(b)] bit for bit, where row(a)
 * walks the kept row units in list order (row_group rows each) and col(b) the
 * kept column units.  Wc is [n_rk*row_group, n_ck*col_group], ld = its cols.
 */
void oracle_compact(const void *W, int64_t ldw, int dtype, const int32_t *row_keep, int64_t n_rk,
                    int64_t row_group, const int32_t *col_keep, int64_t n_ck, int64_t col_group,
                    void *Wc)
{
    int64_t out_cols = n_ck * col_group;
    size_t esz = (dtype == ORACLE_F32) ? 4 : 2;
#pragma omp parallel for schedule(static)
    for (int64_t a = 0; a < n_rk * row_group; ++a) {
        int64_t i = (int64_t)row_keep[a / row_group] * row_group + a % row_group;
        for (int64_t b = 0; b < out_cols; ++b) {
            int64_t j = (int64_t)col_keep[b / col_group] * col_group + b % col_group;
            memcpy((char *)Wc + (size_t)(a * out_cols + b) * esz,
                   (const char *)W + (size_t)(i * ldw + j) * esz, esz);
        }
    }
}

/*
 * Calibration-side companion of the path (Section 4.1.3, "Calibration"; Section 4.1.2: the
 * pruning back-end ranks weights with the inverse Hessian): the second-moment matrix of a
 * projection's input activations,
 *     G[j][l] += sum_t X[t][j] * X[t][l],
 * every product and sum in fp64, t in order.  The layer Hessian of that back-end is
 * H = (2 / T) * G over all T calibration tokens (the published definition 2 X X^T averaged over
 * the samples); its diagonal G[j][j] is the squared norm of Eq. 5.  G_abs (optional) receives
 * sum_t |X[t][j]| * |X[t][l]|, the scale an fp32 accumulation's error is bounded against.
 */
void oracle_gram(const void *X, int64_t tokens, int64_t cols, int64_t ldx, int dtype,
                 double *G, double *G_abs)
{
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < cols; ++j) {
        for (int64_t l = 0; l < cols; ++l) {
            double s = 0.0, a = 0.0;
            for (int64_t t = 0; t < tokens; ++t) {
                const double xj = (double)load_elem(X, t * ldx + j, dtype);
                const double xl = (double)load_elem(X, t * ldx + l, dtype);
                s += xj * xl;
                a += fabs(xj) * fabs(xl);
            }
            G[j * cols + l] += s;
            if (G_abs)
                G_abs[j * cols + l] += a;
        }
    }
}

/* The same sums for a list of (j, l) pairs only: out[q] = sum_t X[t][js[q]] * X[t][ls[q]]. */
void oracle_gram_pairs(const void *X, int64_t tokens, int64_t ldx, int dtype, int64_t n_pairs,
                       const int64_t *js, const int64_t *ls, double *out, double *out_abs)
{
#pragma omp parallel for schedule(static)
    for (int64_t q = 0; q < n_pairs; ++q) {
        double s = 0.0, a = 0.0;
        for (int64_t t = 0; t < tokens; ++t) {
            const double xj = (double)load_elem(X, t * ldx + js[q], dtype);
            const double xl = (double)load_elem(X, t * ldx + ls[q], dtype);
            s += xj * xl;
            a += fabs(xj) * fabs(xl);
        }
        out[q] = s;
        if (out_abs)
            out_abs[q] = a;
    }
}

/* Thread count of the parallel loops above (timing only: no result depends on it). */
void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

int oracle_num_threads(void)
{
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
