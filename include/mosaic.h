/*
 * mosaic.h - C ABI of the B200 (sm_100a) library for the data-parallel hot
 * path of Mosaic's composite projection pruning.
 *
 * The path (paper Section 3.1-3.3, Algorithm 1, Section 4.1.3):
 *   activation l2 norms per input channel  ->  weight metric w = norm*|W| (Eq. 5)
 *   ->  projection outlier count (Eq. 6)   ->  non-uniform sparsity targets
 *   (normalize(R_LLM) + Projection Planner, Eq. 1-2)  ->  per-row unstructured
 *   selection + zeroing  ->  structured ranking + dense compaction.
 *
 * Conventions that hold for every call
 *   - Matrices are row-major.  W is [rows = out_features, cols = in_features]
 *     with leading dimension ldw (elements); X is [tokens, cols] with ldx.
 *   - dtype is MOSAIC_F32 or MOSAIC_BF16 (raw IEEE bfloat16 bit patterns).
 *   - "device" pointers are CUDA global memory of the current device; "host"
 *     pointers are ordinary memory.  Matrix base pointers must be 16-byte
 *     aligned and leading dimensions a multiple of 16 bytes (8 bf16 / 4 fp32
 *     elements), otherwise MOSAIC_ERR_MISALIGNED.
 *   - The library allocates no memory and owns none: outputs and workspaces
 *     are the caller's.  A workspace must be 256-byte aligned and at least
 *     the matching *_workspace_bytes() query; its contents are scratch.
 *   - Device calls only enqueue work on `stream` (a cudaStream_t passed as
 *     void*, NULL = default stream) and never synchronise.  Results are
 *     deterministic: the same inputs give the same bytes, run to run.
 *   - Every call returns MOSAIC_OK (0) or a negative mosaic_status; argument
 *     errors are detected before anything is enqueued.  No C++ exception
 *     crosses the boundary.
 *   - norms[] must be >= +0 (they are l2 norms); scores are then >= +0 and
 *     ordered by their fp32 bit patterns.  A NaN score orders above +inf.
 */
#ifndef MOSAIC_H_
#define MOSAIC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MOSAIC_VERSION 100

typedef enum mosaic_status {
    MOSAIC_OK = 0,
    MOSAIC_ERR_INVALID_ARG = -1,
    MOSAIC_ERR_NULL_PTR = -2,
    MOSAIC_ERR_BAD_DTYPE = -3,
    MOSAIC_ERR_MISALIGNED = -4,
    MOSAIC_ERR_WORKSPACE_TOO_SMALL = -5,
    MOSAIC_ERR_ALIASING = -6,
    MOSAIC_ERR_CUDA = -7,
    MOSAIC_ERR_NONFINITE = -8,   /* reserved */
    MOSAIC_ERR_INFEASIBLE = -9,  /* allocation had to clamp a target; outputs are still written */
    MOSAIC_ERR_TIMEOUT = -10     /* a bounded device-side wait ran out (reported through a status word) */
} mosaic_status;

typedef enum mosaic_dtype { MOSAIC_F32 = 0, MOSAIC_BF16 = 1 } mosaic_dtype;

/* flags of mosaic_act_norms */
#define MOSAIC_RESET_ACCUM 1 /* treat sumsq_accum as zero on entry */

/* mode of mosaic_allocate_sparsity */
#define MOSAIC_GLOBAL_NORM 0       /* normalise ranks over all N*M projections            */
#define MOSAIC_PER_CATEGORY_NORM 1 /* normalise separately over the N entries of each m   */
#define MOSAIC_WEIGHTED_MEAN 2     /* flag, or-ed in: the targets average to p weighted by
                                      each projection's parameter count, so the pruned share
                                      of all parameters is p (Eq. 1-2 use the plain mean)   */
#define MOSAIC_REDISTRIBUTE 4      /* flag, or-ed in: clamp and redistribute - a target that
                                      leaves [0, 1 - 1/cols] stays on the bound and the others
                                      of its group shift by one common amount so that the mean
                                      stays p (without it a clamp moves the mean off p)      */

/* flags of mosaic_prune_structured_compact */
#define MOSAIC_ROWS_GIVEN 1    /* row_keep_units is an input (ascending unit indices)      */
#define MOSAIC_COLS_GIVEN 2    /* col_keep_units is an input                               */
#define MOSAIC_RANK_ONLY 4     /* compute scores / keep lists, do not write W_out          */
#define MOSAIC_SCORES_ONLY 8   /* compute unit_scores_out only: no ranking, no compaction  */
#define MOSAIC_SCORES_ACCUM 16 /* add the unit scores to unit_scores_out (fp32) instead of
                                  overwriting it: lets a caller sum the scores of coupled
                                  projections before ranking them once                     */

int mosaic_version(void);
const char *mosaic_status_string(int status);

/* ---------------------------------------------------------------------------
 * mosaic_act_norms - the ||A||_2 term of Eq. 5 (Section 3.3, Activation
 * Processor / Rank Pre-Processor): per input channel j,
 *     sumsq_accum[j] += sum_t X[t,j]^2        (fp64, exact squares)
 * and, if norms_out != NULL,  norms_out[j] = (float) sqrt(sumsq_accum[j]).
 * Accumulating: call once per chunk of calibration tokens; tokens == 0 is
 * legal (only the reset / finalise parts run).
 *   X            device, [tokens, cols], ld ldx, dtype; read only
 *   sumsq_accum  device, [cols] fp64, in-out, caller-owned accumulator
 *   norms_out    device, [cols] fp32, or NULL
 *   flags        0 or MOSAIC_RESET_ACCUM
 *   ws           device scratch, >= mosaic_act_norms_workspace_bytes(tokens, cols)
 * ------------------------------------------------------------------------- */
size_t mosaic_act_norms_workspace_bytes(int64_t tokens, int64_t cols);
int mosaic_act_norms(const void *X, int64_t tokens, int64_t cols, int64_t ldx, int dtype,
                     double *sumsq_accum, float *norms_out, int flags, void *ws, size_t ws_bytes,
                     void *stream);

/* ---------------------------------------------------------------------------
 * mosaic_score - Eq. 5 / the weight-metric step of Algorithm 1, materialised:
 *     score_out[i, j] = fl32( norms[j] * |W[i, j]| )      (one fp32 multiply)
 * For tests and small use; the pruning calls recompute scores on the fly.
 *   W          device, [rows, cols], ld ldw, dtype; read only
 *   norms      device, [cols] fp32
 *   score_out  device, [rows, cols] fp32, ld = cols, 16-byte aligned
 * ------------------------------------------------------------------------- */
int mosaic_score(const void *W, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                 const float *norms, float *score_out, void *stream);

/* ---------------------------------------------------------------------------
 * mosaic_outlier_ratio - Eq. 6 / the outlier-count step of Algorithm 1 for one projection:
 *     S = sum_ij (double) w_ij,  tau = (double)alpha * (S / (rows*cols)),   (fp64, in this order)
 *     O = #{ (i,j) : (double) w_ij > tau }                  (strict)
 *   outlier_count_out  device, 1 x int64
 *   score_sum_out      device, 1 x fp64, or NULL
 *   ws                 device scratch, >= mosaic_outlier_ratio_workspace_bytes()
 * The rank R = 100*O/C (the projection-rank step of Algorithm 1) is formed on the host:
 * mosaic_ratio_from_count.
 * ------------------------------------------------------------------------- */
size_t mosaic_outlier_ratio_workspace_bytes(int64_t rows, int64_t cols);
int mosaic_outlier_ratio(const void *W, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                         const float *norms, float alpha, int64_t *outlier_count_out,
                         double *score_sum_out, void *ws, size_t ws_bytes, void *stream);
double mosaic_ratio_from_count(int64_t outlier_count, int64_t numel);

/* ---------------------------------------------------------------------------
 * mosaic_outlier_ratio_batch - mosaic_outlier_ratio for a list of projections
 * (Algorithm 1 loops over all N*M of them) in a handful of launches instead of
 * two per projection.  Results are bit for bit those of the single call.
 * bf16 matrices with cols % 8 == 0 are read ONCE: an estimate of the threshold
 * from a sample of rows fixes, per column, a ladder of 32 bf16 magnitude patterns
 * around the pattern the threshold will fall on; the sweep that sums the scores
 * counts the weights above the ladder and, per pattern, those on it, and the
 * exact count follows when the sum is known.  A matrix whose threshold falls off
 * a ladder (rows unlike the sampled ones) is counted by a second sweep after
 * all.  The workspace holds the ladders (128 bytes per column and matrix).
 *   jobs   HOST array of n_jobs descriptors (read during the call only); the
 *          pointers inside are device pointers with the meaning of the
 *          single call's arguments (score_sum_out may be NULL)
 *   ws     device scratch, >= mosaic_outlier_ratio_batch_workspace_bytes for
 *          the same list
 * ------------------------------------------------------------------------- */
typedef struct mosaic_outlier_job {
    const void *W;
    int64_t rows, cols, ldw;
    const float *norms;
    int64_t *outlier_count_out;
    double *score_sum_out;
} mosaic_outlier_job;
size_t mosaic_outlier_ratio_batch_workspace_bytes(const mosaic_outlier_job *jobs, int64_t n_jobs);
int mosaic_outlier_ratio_batch(const mosaic_outlier_job *jobs, int64_t n_jobs, int dtype, float alpha,
                               void *ws, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------
 * mosaic_outlier_ratio_grouped - the layer outlier distribution (Eq. 3-4, the
 * layer-pruning baseline of Section 4.1.3): as mosaic_outlier_ratio_batch, but
 * the matrices of a group (the projections of a layer) are counted against ONE
 * threshold,  tau_g = (double)alpha * (S_g / C_g),  S_g the sum over the group's
 * matrices (in list order) of their fp64 score sums, C_g their number of
 * elements.  Every job's outlier_count_out receives that matrix's count against
 * its group's tau (their sum is the layer's O); score_sum_out, if given, the
 * matrix's own S.
 *   group_of   HOST array, n_jobs entries: jobs of one group are adjacent and
 *              carry the same value; a group has at most 256 jobs
 * ------------------------------------------------------------------------- */
int mosaic_outlier_ratio_grouped(const mosaic_outlier_job *jobs, const int32_t *group_of, int64_t n_jobs,
                                 int dtype, float alpha, void *ws, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------
 * mosaic_outlier_ratio_static - mosaic_outlier_ratio without a workspace
 * argument.  (The paper has no counterpart: this is a packaging variant of the
 * call above, not another operation.)
 * Who it is for: code that may not allocate device memory when it calls in -
 * a plug-in running inside a host application that owns the allocator, a
 * callback on a latency-critical path where cudaMalloc's implicit
 * synchronisation is not acceptable, a process whose memory pool is already
 * committed.  Such a caller has nowhere to take the scratch buffer from, so
 * the library carries one itself: a fixed array of
 * MOSAIC_OUTLIER_STATIC_SCRATCH_BYTES in device memory, present on every GPU
 * that loads the library for as long as the process lives.  The call
 * allocates and frees nothing.
 *   - Inputs and outputs are the caller's, exactly as for mosaic_outlier_ratio,
 *     and the results are bit-identical to it.
 *   - A matrix whose scratch need (mosaic_outlier_ratio_workspace_bytes)
 *     exceeds the built-in array is refused with
 *     MOSAIC_ERR_WORKSPACE_TOO_SMALL before anything is enqueued; use the
 *     regular call with your own buffer then.
 *   - The first call on each device looks up the array's device address (a
 *     host-side runtime query, with that device current).  Make that first
 *     call during start-up, outside any stream capture.  The address belongs
 *     to the device's context: after cudaDeviceReset() on a device this entry
 *     point must not be used on it again in the same process.
 *   - All calls on one device share the one array.  Every call overwrites
 *     what it reads from it, so whatever an earlier call left there does no
 *     harm and back-to-back calls on one stream are fine; two calls that can overlap
 *     on the GPU (different streams, different host threads) race on it and
 *     give wrong counts.  Serialise them, or give the overlapping ones their
 *     own workspace through mosaic_outlier_ratio.
 * ------------------------------------------------------------------------- */
#define MOSAIC_OUTLIER_STATIC_SCRATCH_BYTES 65536
size_t mosaic_outlier_ratio_static_max_workspace_bytes(void);
int mosaic_outlier_ratio_static(const void *W, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                                const float *norms, float alpha, int64_t *outlier_count_out,
                                double *score_sum_out, void *stream);

/* ---------------------------------------------------------------------------
 * mosaic_allocate_sparsity - normalize(R_LLM) (the return of Algorithm 1) and the
 * Projection Planner (Section 3.3 component 8; Eq. 1-2).  HOST function, all
 * pointers are host memory, q = n*n_proj + m.
 * The paper states only the properties (targets average to p; more outliers
 * => pruned less).  Definition used, fp64, loops in q order:
 *     R_q = 100*O_q/C_q;  lo = min R, hi = max R;  hi == lo -> s_q = p
 *     r_q = (R_q-lo)/(hi-lo);  d_q = 2*lambda*r_q;  dbar = (sum_q w_q d_q)/(sum_q w_q)
 *     (w_q = 1, or C_q with MOSAIC_WEIGHTED_MEAN)
 *     s_q = (p + dbar) - d_q, clamped to [0, 1 - 1/cols_q]
 *     k_q = floor(s_q * cols_q)       (weights removed from every row)
 * MOSAIC_PER_CATEGORY_NORM applies the same over the n_layers entries of each
 * projection index m separately.  Returns MOSAIC_ERR_INFEASIBLE if a clamp
 * fired (outputs are still complete).  With MOSAIC_REDISTRIBUTE, b_q being the
 * unclamped target: clamped targets keep their bound and every other target of
 * the group becomes b_q + t,  t = (p*W - sum_clamped w_q s_q - sum_free w_q b_q)
 * / sum_free w_q, repeated while t pushes further targets over a bound;
 * MOSAIC_ERR_INFEASIBLE is then returned only if every target of a group sits
 * on a bound (p out of reach).
 * For the layer-pruning baseline (Eq. 3-4, one target per layer) pass the
 * layers' outlier counts with n_proj = 1 and give every projection of layer n
 * k = floor(s_n * cols).
 * ------------------------------------------------------------------------- */
int mosaic_allocate_sparsity(const int64_t *outlier_counts, const int64_t *numels,
                             const int64_t *cols, int n_layers, int n_proj, double p,
                             double lambda, int mode, double *sparsity_out, int64_t *k_out);

/* ---------------------------------------------------------------------------
 * mosaic_prune_unstructured - unstructured projection pruning (Section 4.1.3:
 * pruned parameters are set to zero; Section 2.3: the lowest-ranking
 * parameters are removed), selection per output row.  In every row the k
 * entries that come first under (w_ij ascending, j ascending) become +0; all
 * other entries keep their bits.
 *   W_in      device, [rows, cols]; W_out device, same shape/ld; W_out may be
 *             W_in exactly (in place); any other overlap -> MOSAIC_ERR_ALIASING.
 *             W_out == NULL: mask-only mode, the keep bitmask is the only
 *             output (mask_out is then required) and W_in is left untouched
 *   k         0 <= k <= cols
 *   mask_out  device, [rows, ceil(cols/32)] uint32 or NULL; bit j%32 of word
 *             j/32 is 1 for a kept entry; padding bits are 0
 *   cols      at most 65536
 *   ws        unused (the call needs no scratch); may be NULL
 * ------------------------------------------------------------------------- */
size_t mosaic_prune_unstructured_workspace_bytes(int64_t rows, int64_t cols);
int mosaic_prune_unstructured(const void *W_in, void *W_out, int64_t rows, int64_t cols,
                              int64_t ldw, int dtype, const float *norms, int64_t k,
                              uint32_t *mask_out, void *ws, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------
 * mosaic_prune_unstructured_batch - mosaic_prune_unstructured for a list of
 * projections in as few launches as possible (a model has N*M projections,
 * Section 3.1; each is a few tens of microseconds of work, so one launch per
 * projection is dominated by launch and ramp-up time).  Results are bit for
 * bit those of calling mosaic_prune_unstructured once per job.
 *   jobs     HOST array of n_jobs descriptors (read during the call only);
 *            every pointer inside a descriptor is a device pointer with the
 *            meaning and alignment rules of mosaic_prune_unstructured
 *   dtype    one dtype for the whole list
 *   ws       unused (the call needs no scratch; the query returns a token
 *            256 bytes); may be NULL
 * Jobs must not overlap each other's outputs.  With W_out == W_in (in place)
 * the result is the same bits, but rows already pruned by one part of the
 * launch can be sampled by another when it estimates a matrix's threshold,
 * which only costs speed.
 * ------------------------------------------------------------------------- */
typedef struct mosaic_prune_job {
    const void *W_in;
    void *W_out;
    int64_t rows, cols, ldw;
    const float *norms;
    int64_t k;
    uint32_t *mask_out;
} mosaic_prune_job;
size_t mosaic_prune_unstructured_batch_workspace_bytes(const mosaic_prune_job *jobs, int64_t n_jobs, int dtype);
int mosaic_prune_unstructured_batch(const mosaic_prune_job *jobs, int64_t n_jobs, int dtype, void *ws,
                                    size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------
 * mosaic_prune_structured_compact - structured projection pruning (Section
 * 4.1.3: remove the lowest-magnitude heads and channels; Section 2.3:
 * structured pruning removes whole data structures and leaves smaller dense
 * matrices).  A row unit is row_group consecutive rows, a column unit
 * col_group consecutive columns (rows % row_group == 0, cols % col_group == 0).
 *   1. unit scores: fp64 sum of w_ij over the unit, rounded once to fp32
 *      (norms == NULL means norm = 1, i.e. sum of |W|);
 *   2. per dimension, the (n_units - keep) units first under (score asc,
 *      index asc) are removed; the keep list is the surviving unit indices
 *      in ascending order;
 *   3. W_out[a, b] = W_in[row(a), col(b)] bit for bit, dense,
 *      [row_units_keep*row_group, col_units_keep*col_group], ld = its cols.
 *   row_keep_units / col_keep_units  device int32 [row_units_keep] / [col_units_keep];
 *        outputs, or inputs when the matching *_GIVEN flag is set (ascending
 *        unit indices chosen elsewhere, e.g. shared by coupled projections;
 *        an out-of-range given index is clamped into range)
 *   unit_scores_out  device fp32 [rows/row_group + cols/col_group] (row units
 *        first) or NULL
 *   W_out   device; must not overlap W_in; ignored for RANK_ONLY / SCORES_ONLY
 *   ws      device scratch, >= mosaic_prune_structured_compact_workspace_bytes()
 * ------------------------------------------------------------------------- */
size_t mosaic_prune_structured_compact_workspace_bytes(int64_t rows, int64_t cols);
int mosaic_prune_structured_compact(const void *W_in, int64_t rows, int64_t cols, int64_t ldw,
                                    int dtype, const float *norms, int64_t row_group,
                                    int64_t col_group, int64_t row_units_keep,
                                    int64_t col_units_keep, int32_t *row_keep_units,
                                    int32_t *col_keep_units, int flags, void *W_out,
                                    float *unit_scores_out, void *ws, size_t ws_bytes,
                                    void *stream);

/* ---------------------------------------------------------------------------
 * mosaic_rank_units - step 2 above on its own, for scores a caller combined
 * itself (coupled projections share one keep list: Fig. "composite", nodes
 * between projections are pruned as a group).
 *   scores     device fp32 [n_units], >= +0
 *   keep_out   device int32 [keep], ascending surviving unit indices
 * ------------------------------------------------------------------------- */
int mosaic_rank_units(const float *scores, int64_t n_units, int64_t keep, int32_t *keep_out,
                      void *stream);

/* ---------------------------------------------------------------------------
 * mosaic_sum_unit_scores - dst[u] = fl32(dst[u] + src[u]) for u < n_units: adds
 * the unit scores of a coupled projection to a running total before one
 * ranking (same Fig. "composite" grouping; e.g. MLP channel c = row c of
 * gate and up plus column c of down).  dst, src: device fp32, may not overlap
 * partially.
 * ------------------------------------------------------------------------- */
int mosaic_sum_unit_scores(float *dst, const float *src, int64_t n_units, void *stream);

/* ---------------------------------------------------------------------------
 * Batched forms of the structured steps (Section 4.1.3 structured; Section 2.3):
 * the same arithmetic as steps 1-3 of mosaic_prune_structured_compact, bit for
 * bit, for a HOST list of matrices in one launch per step - a model has N*M
 * projections (Section 3.1) and each is only microseconds of work.  Every
 * pointer inside a descriptor is a device pointer; the lists are read during
 * the call only.  Coupled projections (Fig. "composite": nodes between
 * projections are pruned as a group) are handled by the caller: score all
 * matrices, add the scores of the coupled units, rank once, compact each matrix
 * with the shared keep list.
 * ------------------------------------------------------------------------- */

/* Step 1, unit scores.  row_scores_out [rows/row_group] and col_scores_out
 * [cols/col_group] are fp32 outputs (overwritten); either may be NULL.
 * norms == NULL means norm = 1.  ws: device scratch, 256-byte aligned, >= the
 * query for the same list. */
typedef struct mosaic_unit_score_job {
    const void *W;
    int64_t rows, cols, ldw;
    const float *norms;
    int64_t row_group, col_group;
    float *row_scores_out;
    float *col_scores_out;
} mosaic_unit_score_job;
size_t mosaic_unit_scores_batch_workspace_bytes(const mosaic_unit_score_job *jobs, int64_t n_jobs);
int mosaic_unit_scores_batch(const mosaic_unit_score_job *jobs, int64_t n_jobs, int dtype, void *ws,
                             size_t ws_bytes, void *stream);

/* dst[u] = fl32(a[u] + b[u]), u < n, for every item: the running total of the
 * scores of coupled units.  dst may be a or b exactly; the items of one call
 * must not write what another item reads. */
typedef struct mosaic_add_job {
    float *dst;
    const float *a;
    const float *b;
    int64_t n;
} mosaic_add_job;
int mosaic_add_unit_scores_batch(const mosaic_add_job *jobs, int64_t n_jobs, void *stream);

/* Step 2, mosaic_rank_units for a list of score arrays. */
typedef struct mosaic_rank_job {
    const float *scores;
    int64_t n_units, keep;
    int32_t *keep_out;
} mosaic_rank_job;
int mosaic_rank_units_batch(const mosaic_rank_job *jobs, int64_t n_jobs, void *stream);

/* Step 3, dense compaction with given keep lists (ascending unit indices; an
 * out-of-range index is clamped).  W_out is dense
 * [row_units_keep*row_group, col_units_keep*col_group] and must not overlap W_in. */
typedef struct mosaic_compact_job {
    const void *W_in;
    int64_t rows, cols, ldw;
    const int32_t *row_keep_units;
    int64_t row_units_keep, row_group;
    const int32_t *col_keep_units;
    int64_t col_units_keep, col_group;
    void *W_out;
} mosaic_compact_job;
int mosaic_compact_batch(const mosaic_compact_job *jobs, int64_t n_jobs, int dtype, void *stream);

/* ---------------------------------------------------------------------------
 * mosaic_gram_accumulate - second moments of a projection's input activations,
 * the calibration-side companion of mosaic_act_norms (Section 4.1.3: the same
 * calibration samples also give the pruning back-end its Hessian; Section 4.1.2:
 * that back-end ranks and updates weights with the inverse Hessian):
 *     G[j,l] += sum_t X[t,j] * X[t,l]        for all 0 <= j, l < cols.
 * The layer Hessian of the back-end is a constant multiple of G (2 X X^T over
 * the calibration tokens, divided by whatever the back-end averages by: (2/T) G
 * per token; the constant changes none of its rankings); diag(G) is the squared
 * norm of Eq. 5.  Call once per chunk of tokens.
 *
 *   X          device, [tokens, cols] row-major, ld = ldx, MOSAIC_BF16 only
 *              (bf16 products are exact in fp32; MOSAIC_F32 -> MOSAIC_ERR_BAD_DTYPE).
 *              cols % 8 == 0, tokens < 2^31 - 64.  tokens = 0 is legal.
 *   G          device, fp32 [cols, cols] row-major, ld = ldg (ldg % 4 == 0,
 *              16-byte aligned), in-out, caller-owned; both triangles are written.
 *              Must not overlap X (MOSAIC_ERR_ALIASING).
 *   flags      0 or MOSAIC_RESET_ACCUM (treat G as zero on entry)
 *   status_dev device, one int, or NULL.  Set to 0 when the call is enqueued and to
 *              1 by the kernel if one of its bounded waits ran out (G is then
 *              undefined); read it after synchronising the stream.
 *
 * Arithmetic: products exact, sums in fp32 on the tensor cores in token order
 * within a chunk, one fp32 add per chunk into G.  The result is deterministic
 * (independent of the grid).  The tensor cores truncate when they add 16 tokens'
 * products to the running sum, so the result of a call differs from the exact
 * sum by at most (tokens/4 + 2) * 2^-24 * sum_t |X[t,j]| |X[t,l]| (measured: about
 * tokens/16 * 2^-24 of the sum, low, on sums of one sign such as the diagonal;
 * shorter calls lose proportionally less).
 * ------------------------------------------------------------------------- */
int mosaic_gram_accumulate(const void *X, int64_t tokens, int64_t cols, int64_t ldx, int dtype, float *G,
                           int64_t ldg, int flags, int *status_dev, void *stream);

/* ---------------------------------------------------------------------------
 * mosaic_bounded_wait_selftest - a diagnostic with no counterpart in the paper.
 * The tensor-core kernel of mosaic_gram_accumulate synchronises its roles
 * through mbarriers, and every such wait carries a cycle budget so that a
 * fault in the pipeline ends as a status word instead of a hung GPU.  This
 * call runs that wait alone: one thread waits on a barrier that nothing will
 * complete, for at most budget_cycles (1 .. 2e9, i.e. up to about a second),
 * and writes how the wait ended to status_dev (device, one int):
 *   1  the wait gave up after the budget and raised the error word (expected)
 *   2  the barrier completed (must not happen)   3  inconsistent
 * ------------------------------------------------------------------------- */
int mosaic_bounded_wait_selftest(int64_t budget_cycles, int *status_dev, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* MOSAIC_H_ */
