/*
 * dass.h -- C ABI of the B200 (sm_100a) hot path of DaSS, Dependency-aware
 * Semi-structured Sparsity for GLU-based MLPs (arXiv 2405.01943).
 *
 * Two stages:
 *   (a) calibration: for every intermediate neuron i accumulate, over the
 *       calibration tokens, the squared l2 norm of the GLU intermediate
 *       activation  y = sigma(x W1) (*) x W2  (Eq. 2; norm as group importance,
 *       Section 3 "Incorporating Dependency into Weight Importance").
 *   (b) pruning: score every weight with |W| * ||y||^alpha (Eq. 4, gate / up)
 *       or |W| * ||y|| (Eq. 5, down), keep the best n of every m consecutive
 *       weights of a comparison line (Section 3, "Extension to N:M Sparsity"),
 *       emit mask, pruned weights and a compressed values + metadata form.
 *
 * Conventions for every call
 *   - Matrices are row-major with a leading dimension `ld` counted in elements.
 *     The paper's transposed projections are used as stored by common
 *     checkpoints: Wg = W(1)^T and Wu = W(2)^T are [I x d], Wd = W(3)^T is
 *     [d x I]  (I = d_int, d = d_hidden), X is [T x d] (T tokens).
 *   - Unless a parameter is documented as HOST, every pointer is DEVICE memory of
 *     the current CUDA device, owned by the caller before, during and after the
 *     call.  The library allocates no device memory and frees nothing.
 *   - Calls only enqueue work on `cuda_stream` (a cudaStream_t passed as void*,
 *     NULL = the default stream) and return without waiting for it.
 *   - Base pointers of matrices must be 16-byte aligned and `ld` a multiple of
 *     8 elements (bf16) or 4 elements (f32), else DASS_ERR_ALIGN.  A matrix
 *     buffer must span rows * ld elements (vector loads may touch the padding
 *     between `cols` and `ld`; it is never written).
 *   - Errors are reported by the return code only: nothing aborts, throws or
 *     prints.  Arguments are validated before anything is enqueued: on
 *     DASS_ERR_NULL / SHAPE / ALIGN / DTYPE / UNSUPPORTED / WORKSPACE no output
 *     has been touched.  DASS_ERR_CUDA means a CUDA runtime or driver call
 *     failed part-way (a launch, a tensor-map encode, a copy): work enqueued
 *     before it may still run, and the call's outputs are then unspecified.
 *   - Non-finite inputs are not diagnosed; results for them are unspecified.
 *   - Host threads: the entry points keep no state besides per-device caches that
 *     are atomic, so they may be called from several host threads (each with its
 *     own current device and stream).  Calls that share a workspace, an output
 *     buffer or the static scratch of dass_calib_accumulate_static must be
 *     ordered by the caller, on the host and on the device.
 */
#ifndef DASS_H
#define DASS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DASS_OK = 0,
    DASS_ERR_NULL = 1,         /* a required pointer is NULL */
    DASS_ERR_SHAPE = 2,        /* non-positive size, extent not divisible by m, bad n_keep */
    DASS_ERR_ALIGN = 3,        /* pointer or leading dimension not aligned as required */
    DASS_ERR_DTYPE = 4,        /* unknown dass_dtype / dass_act / dass_axis value */
    DASS_ERR_UNSUPPORTED = 5,  /* a valid request the library has no kernel for */
    DASS_ERR_WORKSPACE = 6,    /* workspace NULL or smaller than the query says */
    DASS_ERR_CUDA = 7,         /* a CUDA runtime / driver call failed */
    DASS_ERR_TIMEOUT = 8,      /* a bounded device-side wait ran out (reported by dass_calib_status / dass_prune_status) */
    DASS_ERR_INTERNAL = 9      /* a consistency check between two passes of a kernel chain failed (dass_prune_status) */
} dass_status;

typedef enum { DASS_BF16 = 0, DASS_F32 = 1 } dass_dtype;
typedef enum { DASS_ACT_SILU = 0, DASS_ACT_GELU_TANH = 1, DASS_ACT_RELU = 2 } dass_act;
/* Which matrix axis an index runs along: ROWS = the row index varies, COLS = the column index varies. */
typedef enum { DASS_AXIS_ROWS = 0, DASS_AXIS_COLS = 1 } dass_axis;

/* ------------------------------------------------------------------ stage (a)
 * Eq. 2 and the per-neuron squared norm:
 *     sumsq[i] += sum_{t < T} ( act(X[t,:] . Wg[i,:]) * (X[t,:] . Wu[i,:]) )^2     for i in [0, I)
 * act = SiLU (SwiGLU), tanh-form GeLU (GeGLU) or ReLU (ReGLU) -- Section 2.2.
 * The intermediate H is never written to memory.
 *
 * X [T x d, ldx], Wg and Wu [I x d, ldw] in `dt`.  bf16: tensor-core path
 * (fp32 accumulation, activation and square in fp32).  f32: plain fp32 FMA path.
 * sumsq [I] doubles, in/out: the call ADDS this batch's contribution, so a
 * calibration set may be fed in any number of batches; the caller zeroes it
 * before the first batch.  The per-batch contribution is reduced in a fixed
 * order, so equal inputs (and an equal workspace size) give bit-equal results.
 * workspace: scratch of dass_calib_workspace_bytes(...) bytes, 256-byte aligned,
 * contents irrelevant on entry; it must not be shared by calls that may overlap
 * on the device.  A workspace sized by the query for T tokens also serves every
 * call with fewer tokens (the call then uses coarser partial sums if it has to).
 * Its first word receives a device status that dass_calib_status reads.
 * Errors: NULL / SHAPE (T, d, I < 1) / ALIGN / DTYPE / WORKSPACE / CUDA. */
dass_status dass_calib_workspace_bytes(int64_t T, int64_t d, int64_t I, dass_dtype dt, size_t *bytes /* HOST */);
dass_status dass_calib_accumulate(const void *X, int64_t T, int64_t ldx,
                                  const void *Wg, const void *Wu, int64_t I, int64_t d, int64_t ldw,
                                  dass_dtype dt, dass_act act,
                                  double *sumsq,
                                  void *workspace, size_t workspace_bytes, void *cuda_stream);
/* Waits for `cuda_stream`, then reports what the last dass_calib_accumulate that used
 * `workspace` left in its status word: DASS_OK, or DASS_ERR_TIMEOUT if a bounded wait inside
 * the kernel gave up (the results of that call are then invalid; the context stays usable). */
dass_status dass_calib_status(const void *workspace, void *cuda_stream);

/* Failure-path self-test (no counterpart in the paper).  Every wait inside the tensor-core kernels is bounded; when one
 * runs out the kernel records DASS_ERR_TIMEOUT in its status word, drains and returns, and the CUDA context stays
 * usable.  This call exercises exactly that mechanism without disturbing the GPU: a one-warp kernel waits, with the same
 * bounded-wait routine, on a barrier that nothing will ever complete, for at most limit_us microseconds (1 .. 1 000 000),
 * and then writes the outcome to status_word (a 4-byte aligned device int), which dass_calib_status reads.
 * Errors: NULL / SHAPE (limit out of range) / ALIGN / CUDA. */
dass_status dass_selftest_wait_timeout(void *status_word, int64_t limit_us, void *cuda_stream);

/* The paper has no counterpart for this entry point: it exists for callers that cannot allocate.
 * Some users of this library may not call cudaMalloc where they calibrate -- code inside a framework's
 * memory-planned region or allocator callback, plugins that own nothing but the tensors they are
 * handed, processes with a device-memory budget fixed at start-up, loops where an allocation's implicit
 * device synchronisation is not acceptable.  dass_calib_accumulate makes them supply the workspace; this
 * variant needs none.  It computes exactly what dass_calib_accumulate computes (same kernels, same
 * fixed reduction order, same arguments and error codes), but its scratch is a fixed array of
 * DASS_STATIC_SCRATCH_BYTES inside the library's device image, which every GPU that loads the library
 * holds until the process exits.  It calls no cudaMalloc / cudaFree and no allocating routine.
 *  - Limit: a problem whose partial sums do not fit into DASS_STATIC_SCRATCH_BYTES even at their coarsest (bf16:
 *    one double per neuron and 4096 tokens) is refused with DASS_ERR_WORKSPACE and nothing is touched (16 MiB
 *    covers a 28672-neuron bf16 layer at 262144 tokens per call; feed larger token counts in several calls).
 *  - The first call on each device (made with that device current) looks up the scratch's device
 *    address once; make that first call before any stream capture begins.  The look-up may be made by
 *    several host threads at once (they cache the same address atomically).
 *  - All calls on a device share the one array, which keeps the previous call's contents; the call
 *    clears the status word itself and overwrites every partial sum it later reads.  Two calls that may
 *    overlap on the GPU (different streams, no ordering between them) race on it: order them.
 *  - scratch_address (HOST pointer, nullable) receives the array's device address, which may be handed
 *    to dass_calib_status to learn whether a bounded device-side wait timed out. */
#define DASS_STATIC_SCRATCH_BYTES (16u << 20)
dass_status dass_calib_accumulate_static(const void *X, int64_t T, int64_t ldx,
                                         const void *Wg, const void *Wu, int64_t I, int64_t d, int64_t ldw,
                                         dass_dtype dt, dass_act act, double *sumsq,
                                         void **scratch_address /* HOST, nullable */, void *cuda_stream);

/* norm[i] = (float) sqrt(sumsq[i]): the l2 norm ||y_i||_2 handed to stage (b).
 * Both operations are correctly rounded, so the value is reproducible bit for bit. */
dass_status dass_norm_finalize(const double *sumsq, int64_t I, float *norm, void *cuda_stream);

/* ------------------------------------------------------------------ stage (b)
 * Eq. 4 / Eq. 5 score and N:M selection.
 *     score(r,c) = |W[r,c]| * scale(norm[k], alpha),   k = r if norm_axis == ROWS, c if COLS
 *     scale(n, alpha) = (float) n^alpha, rounded once: 1 for alpha = 0 (also when n = 0), n for
 *     alpha = 1, sqrt / sqrt(sqrt) / sqrt*sqrt(sqrt) evaluated in double for 1/2, 1/4, 3/4,
 *     pow in double otherwise.  Scores are compared as exact products (no rounding).
 * Groups are m consecutive elements along group_axis (ROWS: rows r..r+m-1 of one column; COLS:
 * columns c..c+m-1 of one row).  In each group the n_keep highest scores are kept; among equal
 * scores the lower index wins.
 *     gate / up, Eq. 4:  W = Wg or Wu [I x d], norm_axis = ROWS, group_axis = ROWS  (input-balanced:
 *                        the weights of one input column are compared across neurons), alpha = 0.5
 *     down, Eq. 5:       W = Wd [d x I],       norm_axis = COLS, group_axis = COLS  (output-balanced),
 *                        alpha = 1
 *     Wanda, Eq. 1:      any W [out x in] with input-feature norms: norm_axis = COLS, group_axis = COLS
 * norm: rows (ROWS) or cols (COLS) floats.  alpha: finite, >= 0.
 * Supported patterns: m in {4, 8}, 1 <= n_keep < m; the group-axis extent must be a multiple of m (the other
 * extent may be any positive value; see the alignment rules above).
 * mask_bits (nullable): rows * ceil(cols/32) words; bit (c % 32) of word r * ceil(cols/32) + c / 32
 *     is 1 iff W[r,c] is kept; padding bits are written as 0.
 * W_pruned (nullable): same dtype and ld as W; survivors are copied bit for bit, the others become +0
 *     ("no weight update").  May be W itself (in place).
 * At least one of the two outputs must be given.
 * Errors: NULL / SHAPE / ALIGN / DTYPE / UNSUPPORTED (alpha < 0 or not finite, m not 4 or 8). */
dass_status dass_score_nm(const void *W, int64_t rows, int64_t cols, int64_t ld, dass_dtype dt,
                          const float *norm, dass_axis norm_axis, float alpha,
                          int n_keep, int m, dass_axis group_axis,
                          uint32_t *mask_bits, void *W_pruned, void *cuda_stream);

/* Compressed N:M form of W under a mask produced by dass_score_nm with the same n_keep, m, group_axis.
 * The paper gives no storage format (it only points to N:M hardware support, Section 2.3); this is a
 * plain, un-swizzled one:
 * values: the n_keep survivors of every group in index order, dtype of W, densely packed:
 *     group_axis = COLS: [rows x cols*n_keep/m];  ROWS: [rows*n_keep/m x cols].
 * meta: one field per group.  2:4: a nibble pos_lo | pos_hi << 2 (positions 0..3 of the two survivors,
 *     pos_lo < pos_hi).  Any other pattern: the m-bit keep mask of the group.  Fields are packed LSB
 *     first along the columns; a line of fields (COLS: one row, cols/m fields; ROWS: one row group,
 *     cols fields) is padded with zeros to whole 32-bit words.
 *     Sizes: COLS: rows * ceil(cols/m / F) words, ROWS: (rows/m) * ceil(cols / F), F = 32 / field bits.
 * A mask that does not hold exactly n_keep survivors in some group gives unspecified output.
 * Errors: NULL / SHAPE / ALIGN / DTYPE / UNSUPPORTED as for dass_score_nm. */
dass_status dass_compress_nm(const void *W, const uint32_t *mask_bits,
                             int64_t rows, int64_t cols, int64_t ld, dass_dtype dt,
                             int n_keep, int m, dass_axis group_axis,
                             void *values, uint32_t *meta, void *cuda_stream);

/* Stage (b) in one pass: dass_score_nm and dass_compress_nm of the same selection from a single read of W.
 * The mask and the compressed form describe one and the same choice of survivors (Section 3, "Extension to N:M
 * Sparsity": every group of m consecutive weights of a comparison line keeps n of them, by the score of Eq. 4 /
 * Eq. 5), so nothing but memory traffic separates the two calls: this entry point reads each weight once and writes
 * whichever of the outputs are asked for -- per bf16 weight 2 bytes in, 2 (pruned copy) + 0.125 (mask) + 1 (values)
 * + 0.125 (metadata) out, against 7.375 bytes for the two calls in sequence.
 * All arguments, layouts, the score, the order and the tie rule are those of dass_score_nm (W, norm, alpha, n_keep, m,
 * axes, mask_bits, W_pruned) and dass_compress_nm (values, meta); the results are bit-identical to theirs.
 * Outputs: mask_bits, W_pruned (may be W itself), values + meta -- each nullable, at least one group required;
 * values and meta are given together or not at all.  values / meta must not overlap W.
 * Errors: NULL (no output, or values without meta) / SHAPE / ALIGN / DTYPE / UNSUPPORTED as for dass_score_nm. */
dass_status dass_prune_nm(const void *W, int64_t rows, int64_t cols, int64_t ld, dass_dtype dt,
                          const float *norm, dass_axis norm_axis, float alpha,
                          int n_keep, int m, dass_axis group_axis,
                          uint32_t *mask_bits, void *W_pruned, void *values, uint32_t *meta, void *cuda_stream);
/* The tuned kernels behind dass_prune_nm (bf16, 2:4 and 4:8) and behind dass_select_unstructured (bf16, lines that
 * are columns) receive their tiles through bulk tensor copies and wait for each on a barrier; every such wait is
 * bounded (2 s).  Waits for `cuda_stream`, then returns DASS_OK, or DASS_ERR_TIMEOUT if a wait of any such call on
 * the current device ran out since the last query (that call's outputs are then incomplete; the context stays
 * usable), or DASS_ERR_INTERNAL if the passes of a dass_select_unstructured call disagreed on how many elements lie
 * at a column's cut (outputs of that call unspecified), and clears the record.  CUDA failure: DASS_ERR_CUDA. */
dass_status dass_prune_status(void *cuda_stream);

/* Eq. 1's input-feature norms (Wanda; the paper prunes the attention projections with it, Section 4.1 "Sparsity"):
 *     sumsq[j] += sum_{t < T} X[t,j]^2      for j in [0, d)
 * X [T x d, ldx] in `dt`; sumsq [d] doubles, in/out (accumulates over calls, fixed reduction order inside a call).
 * dass_norm_finalize turns it into ||X_j||_2; dass_score_nm / dass_select_unstructured with norm_axis = COLS and row
 * lines (group_axis / compare_axis = COLS), alpha = 1, then are Wanda for any weight matrix [out x d].
 * workspace: dass_feature_workspace_bytes(T, d) bytes, 16-byte aligned.
 * Errors: NULL / DTYPE / SHAPE / ALIGN / WORKSPACE / CUDA. */
dass_status dass_feature_workspace_bytes(int64_t T, int64_t d, size_t *bytes /* HOST */);
dass_status dass_feature_sumsq(const void *X, int64_t T, int64_t d, int64_t ldx, dass_dtype dt,
                               double *sumsq, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Unstructured DaSS selection (Section 3, "Pruning Granularity"): inside every comparison line the
 * floor(sparsity * L) weights with the lowest Eq. 4 / Eq. 5 score are pruned, L being the line length.
 *     compare_axis = ROWS: a line is a whole column (all rows at one input: "input-balanced", the paper's
 *                          choice for gate / up, with norm_axis = ROWS and alpha = 0.5)
 *     compare_axis = COLS: a line is a whole row ("output-balanced", the paper's choice for down and what
 *                          Wanda does, with norm_axis = COLS and alpha = 1)
 * Score, scale rounding and order are those of dass_score_nm: exact products, higher score first, lower
 * index first.  sparsity in [0, 1).  mask_bits / W_pruned as for dass_score_nm (at least one; mask_bits is
 * written in full, padding bits 0).  workspace: dass_select_workspace_bytes(...) bytes, 16-byte aligned (holds
 * the rounded norm^alpha vector, the per-column thresholds, the rows left to the slower exact kernel and, per
 * column, the few elements at its cut that are ranked last: about 1.9 KB per column).  A row that the streaming
 * kernel cannot decide is cached in shared memory by the exact kernel: rows of more than about 108 000 bf16 or
 * 54 000 f32 elements are DASS_ERR_UNSUPPORTED; lines that are matrix columns have no such limit (below 2^31
 * elements).  W_pruned may be W itself (in place).
 * Errors: NULL / DTYPE / SHAPE (sizes, sparsity outside [0,1)) / ALIGN / UNSUPPORTED / WORKSPACE / CUDA. */
dass_status dass_select_workspace_bytes(int64_t rows, int64_t cols, dass_axis norm_axis, size_t *bytes /* HOST */);
dass_status dass_select_unstructured(const void *W, int64_t rows, int64_t cols, int64_t ld, dass_dtype dt,
                                     const float *norm, dass_axis norm_axis, float alpha,
                                     double sparsity, dass_axis compare_axis,
                                     uint32_t *mask_bits, void *W_pruned,
                                     void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Forward pass of one GLU MLP layer with the weights given, Eq. 2 then Eq. 3 (Section 2.2):
 *     H[t,i] = act(X[t,:] . Wg[i,:]) * (X[t,:] . Wu[i,:])        rounded to `dt`
 *     Z[t,n] = sum_i H[t,i] * Wd[n,i]                             rounded to `dt`
 * Called with the pruned weights (zeros stored in place, as dass_score_nm's W_pruned writes them) it gives the
 * pruned layer's output, which is what the next layer's calibration reads when a model is pruned layer by
 * layer.  X [T x d, ldx], Wg / Wu [I x d, ldw], Wd [d x I, ldd], Z [T x d, ldz], all in `dt`, row-major, device.
 * bf16: tensor-core path, fp32 accumulation, H held in bf16 between the two contractions (as a bf16 model holds
 * it).  f32: plain fp32 FMA path, H held in fp32.
 * workspace: 256-byte aligned device scratch holding the status word and H for a chunk of tokens.  Any size
 * from *min_bytes up is accepted; with *full_bytes all T tokens go through in one pass, with less the tokens are
 * processed in chunks (whole multiples of 4096 or 256 tokens).  Its first word receives the device status that
 * dass_calib_status reads (DASS_ERR_TIMEOUT if a bounded device-side wait gave up).  It must not be shared by
 * calls that may overlap on the device.  After the call the workspace still holds the last chunk's H, row-major
 * from byte 256 on, with a pitch of I rounded up to 8 (bf16) or 4 (f32) elements -- after a one-pass call, all of H.
 * Errors: NULL / DTYPE / SHAPE (sizes < 1, pitches below the row length) / ALIGN (X, Wg, Wu, Wd 16-byte aligned,
 * their pitches multiples of 16 bytes) / UNSUPPORTED (a dimension beyond the kernels' 32-bit coordinates) /
 * WORKSPACE / CUDA. */
dass_status dass_mlp_forward_workspace_bytes(int64_t T, int64_t d, int64_t I, dass_dtype dt,
                                             size_t *min_bytes /* HOST, nullable */, size_t *full_bytes /* HOST, nullable */);
dass_status dass_mlp_forward(const void *X, int64_t T, int64_t ldx,
                             const void *Wg, const void *Wu, int64_t I, int64_t d, int64_t ldw,
                             const void *Wd, int64_t ldd, dass_dtype dt, dass_act act,
                             void *Z, int64_t ldz,
                             void *workspace, size_t workspace_bytes, void *cuda_stream);

/* ------------------------------------------------------------------ checked-access build
 * (No counterpart in the paper: the stand-in for a memory sanitizer.)  libdass_check.so is this library compiled with
 * -DDASS_BOUNDS_CHECK (python -m paper_2405_01943_b200.build --bounds-check).  In it every entry point registers the
 * address ranges of the buffers it was handed (with the sizes this header states) and every global load and store of
 * the library's kernels is tested against them; an access outside all ranges is skipped -- a load yields zero -- and
 * counted.  Bulk tensor copies are not included: their extents are enforced by the tensor map in hardware.
 * dass_bounds_report waits for `cuda_stream`, returns the number of such accesses since the last report together
 * with the first offender's address, width in bytes and source line (each nullable), and clears the record.
 * dass_bounds_shrink_next is a test hook: the next entry-point call registers every range `bytes` shorter at its end,
 * so that the checker can be seen to catch (and skip) accesses to memory that is in fact valid.
 * In the regular library both return DASS_ERR_UNSUPPORTED (and *violations = 0). */
dass_status dass_bounds_report(int *violations /* HOST */, unsigned long long *first_address /* HOST, nullable */,
                               int *first_bytes /* HOST, nullable */, int *first_line /* HOST, nullable */, void *cuda_stream);
dass_status dass_bounds_shrink_next(size_t bytes);

/* ------------------------------------------------------------------ misc */
const char *dass_status_string(dass_status s);   /* static string, never NULL */
int dass_version(void);                          /* major * 10000 + minor * 100 + patch */

#ifdef __cplusplus
}
#endif
#endif /* DASS_H */
