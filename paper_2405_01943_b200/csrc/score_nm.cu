// Stage (b): Eq. 4 / Eq. 5 score and N:M selection in one streaming pass -- the plain formulation with
// exact double products, used for fp32 weights and for bf16 patterns without a tuned kernel (bf16 weights otherwise
// take the kernels of score_nm_bf16.cu / prune_nm_bf16.cu, which fall back to the same exact selection on ties).
// When the caller asks for them, the compressed values and metadata of the same selection are emitted by the same
// pass (Section 3, "Extension to N:M Sparsity"), so W is read once for every output.
//
// Bandwidth-bound: every weight is read once (128-bit loads), the pruned copy and one mask bit per
// weight are written once; no score matrix and no sort exist.  A warp owns a tile of 32 rows by 256
// columns (each lane 8 consecutive columns = one 16-byte bf16 vector), so a warp-row is one
// contiguous 512-byte segment whichever axis the groups run along:
//   * groups along COLS (down projection, Eq. 5): the 8 elements a lane holds are two groups of 4 or
//     one group of 8; rows are independent;
//   * groups along ROWS (gate / up, Eq. 4, input-balanced): a lane loads the M rows of a row group at
//     its 8 columns and selects per column -- the strided comparison without any transposed access.
// Scores are compared as exact products: |w| (8 or 24 significant bits) times the float scale
// (24 bits) fits a double without rounding.  The scale ||y||^alpha is evaluated once per tile edge
// (per lane for column norms, per row via a shuffle for row norms), not per weight.
#include "dass_device.cuh"
#include "nm_compact.cuh"

namespace dass {

struct ScoreParams {
    const void *W;
    void *Wp;            // nullable
    uint32_t *mask;      // nullable
    void *values;        // nullable (then meta is null too)
    uint32_t *meta;
    const float *norm;
    int64_t rows, cols, ld;
    int64_t wpr;         // mask words per row
    int64_t vcols;       // columns of the values matrix
    int64_t mwpl;        // metadata words per line
    int vec_ok;          // values rows are 16-byte aligned: vector stores allowed
    int64_t col_blocks, row_blocks;
    int n_keep;
    int scale_mode;
    float alpha;
};

constexpr int TILE_ROWS = 32;
constexpr int TILE_COLS = 256;
constexpr int SCORE_THREADS = 256;

// ---------------------------------------------------------------- groups along the columns
template <bool BF16, int M, bool NORM_COLS>
__global__ void __launch_bounds__(SCORE_THREADS) score_group_cols_kernel(const ScoreParams p)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (SCORE_THREADS / 32) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (SCORE_THREADS / 32);
    const int64_t ntasks = p.col_blocks * p.row_blocks;
    constexpr int UNROLL = 4;

    for (int64_t task = warp; task < ntasks; task += nwarps) {
        const int64_t cb = task % p.col_blocks;
        const int64_t rb = task / p.col_blocks;
        const int64_t c0 = cb * TILE_COLS + lane * 8;
        const int64_t left = p.cols - c0;
        const int nvalid = left >= 8 ? 8 : (left > 0 ? (int)left : 0);

        double sc[8];
        float row_scale = 0.0f;
        if constexpr (NORM_COLS) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                sc[j] = j < nvalid ? (double)scale_from_norm(DASS_LD(&p.norm[c0 + j]), p.scale_mode, p.alpha) : 0.0;
        } else {
            const int64_t r = rb * TILE_ROWS + lane;
            if (r < p.rows) row_scale = scale_from_norm(DASS_LD(&p.norm[r]), p.scale_mode, p.alpha);
        }

        for (int i = 0; i < TILE_ROWS; i += UNROLL) {
            const int64_t rbase = rb * TILE_ROWS + i;
            if (rbase >= p.rows) break;   // warp-uniform
            Chunk<BF16> ch[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (rbase + u < p.rows && nvalid > 0) chunk_load<BF16>(ch[u], p.W, (rbase + u) * p.ld + c0, nvalid);
                else chunk_zero<BF16>(ch[u]);
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int64_t r = rbase + u;
                double rs = 0.0;
                if constexpr (!NORM_COLS) rs = (double)__shfl_sync(FULL_MASK, row_scale, i + u);
                uint32_t keep = 0;
#pragma unroll
                for (int g = 0; g < 8 / M; ++g) {
                    double s[M];
#pragma unroll
                    for (int q = 0; q < M; ++q) {
                        const int j = g * M + q;
                        s[q] = (double)chunk_abs<BF16>(ch[u], j) * (NORM_COLS ? sc[j] : rs);
                    }
                    const uint32_t kg = select_group<M>(s, p.n_keep);
                    keep |= (g * M < nvalid ? kg : 0u) << (g * M);
                }
                const uint32_t word = quad_pack_bytes(keep, lane);
                if (p.values) {   // compressed form of the same selection (every lane takes part in the shuffles)
                    Chunk<BF16> out;
                    const int nout = nvalid / M * p.n_keep;
                    uint32_t fb;
                    bool two_four = false;
                    if constexpr (M == 4) two_four = p.n_keep == 2;
                    if (two_four) fb = compact_cols<BF16, 4, true>(ch[u], keep, 2, nout, out);
                    else fb = compact_cols<BF16, M, false>(ch[u], keep, p.n_keep, nout, out);
                    const uint32_t mword = quad_pack_bytes(fb, lane);
                    if (r < p.rows && nvalid > 0) {
                        if ((lane & 3) == 0) DASS_ST(&p.meta[r * p.mwpl + (c0 >> 5)], mword);
                        chunk_store_n<BF16>(out, p.values, r * p.vcols + c0 / M * p.n_keep, nout, p.vec_ok != 0);
                    }
                }
                if (r < p.rows) {
                    if (p.mask && (lane & 3) == 0 && nvalid > 0) DASS_ST(&p.mask[r * p.wpr + (c0 >> 5)], word);
                    if (p.Wp && nvalid > 0) {
                        chunk_apply_mask<BF16>(ch[u], keep);
                        chunk_store<BF16>(ch[u], p.Wp, r * p.ld + c0, nvalid);
                    }
                }
            }
        }
    }
}

// ---------------------------------------------------------------- groups along the rows
// Compressed values and metadata of one row group at a lane's 8 columns (lanes are independent here).
template <bool BF16, int M, bool TWO_FOUR>
__device__ __forceinline__ void emit_rows(const ScoreParams &p, const Chunk<BF16> (&ch)[M], const uint32_t (&keep_row)[M],
                                          int64_t line, int64_t c0, int nvalid)
{
    static_assert(!TWO_FOUR || M == 4, "2:4 has groups of four");
    constexpr int MAXK = TWO_FOUR ? 2 : M - 1;
    Chunk<BF16> out[MAXK];
    uint32_t fields_lo, fields_hi;
    compact_rows<BF16, M, TWO_FOUR, MAXK>(ch, keep_row, p.n_keep, out, fields_lo, fields_hi);
    if constexpr (M == 4) {
        DASS_ST(&p.meta[line * p.mwpl + (c0 >> 3)], fields_lo);
    } else {
        DASS_ST(&p.meta[line * p.mwpl + (c0 >> 2)], fields_lo);
        if (nvalid > 4) DASS_ST(&p.meta[line * p.mwpl + (c0 >> 2) + 1], fields_hi);
    }
#pragma unroll
    for (int k = 0; k < MAXK; ++k)
        if (k < p.n_keep)
            chunk_store_n<BF16>(out[k], p.values, (line * p.n_keep + k) * p.vcols + c0, nvalid, p.vec_ok != 0);
}

template <bool BF16, int M, bool NORM_COLS>
__global__ void __launch_bounds__(SCORE_THREADS) score_group_rows_kernel(const ScoreParams p)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (SCORE_THREADS / 32) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (SCORE_THREADS / 32);
    const int64_t ntasks = p.col_blocks * p.row_blocks;

    for (int64_t task = warp; task < ntasks; task += nwarps) {
        const int64_t cb = task % p.col_blocks;
        const int64_t rb = task / p.col_blocks;
        const int64_t c0 = cb * TILE_COLS + lane * 8;
        const int64_t left = p.cols - c0;
        const int nvalid = left >= 8 ? 8 : (left > 0 ? (int)left : 0);

        double sc[8];
        float row_scale = 0.0f;
        if constexpr (NORM_COLS) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                sc[j] = j < nvalid ? (double)scale_from_norm(DASS_LD(&p.norm[c0 + j]), p.scale_mode, p.alpha) : 0.0;
        } else {
            const int64_t r = rb * TILE_ROWS + lane;
            if (r < p.rows) row_scale = scale_from_norm(DASS_LD(&p.norm[r]), p.scale_mode, p.alpha);
        }

        for (int g = 0; g < TILE_ROWS / M; ++g) {
            const int64_t r0 = rb * TILE_ROWS + g * M;
            if (r0 >= p.rows) break;   // warp-uniform; rows is a multiple of M so the group is whole
            Chunk<BF16> ch[M];
#pragma unroll
            for (int q = 0; q < M; ++q) {
                if (nvalid > 0) chunk_load<BF16>(ch[q], p.W, (r0 + q) * p.ld + c0, nvalid);
                else chunk_zero<BF16>(ch[q]);
            }
            double rs[M];
#pragma unroll
            for (int q = 0; q < M; ++q) {
                rs[q] = 0.0;
                if constexpr (!NORM_COLS) rs[q] = (double)__shfl_sync(FULL_MASK, row_scale, g * M + q);
            }
            uint32_t keep_row[M];   // bit j of keep_row[q]: element (r0+q, c0+j) kept
#pragma unroll
            for (int q = 0; q < M; ++q) keep_row[q] = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                double s[M];
#pragma unroll
                for (int q = 0; q < M; ++q) s[q] = (double)chunk_abs<BF16>(ch[q], j) * (NORM_COLS ? sc[j] : rs[q]);
                const uint32_t kg = j < nvalid ? select_group<M>(s, p.n_keep) : 0u;
#pragma unroll
                for (int q = 0; q < M; ++q) keep_row[q] |= ((kg >> q) & 1u) << j;
            }
            if (p.values && nvalid > 0) {
                bool done = false;
                if constexpr (M == 4) {
                    if (p.n_keep == 2) {
                        emit_rows<BF16, 4, true>(p, ch, keep_row, r0 / M, c0, nvalid);
                        done = true;
                    }
                }
                if (!done) emit_rows<BF16, M, false>(p, ch, keep_row, r0 / M, c0, nvalid);
            }
#pragma unroll
            for (int q = 0; q < M; ++q) {
                const uint32_t word = quad_pack_bytes(keep_row[q], lane);
                if (p.mask && (lane & 3) == 0 && nvalid > 0) DASS_ST(&p.mask[(r0 + q) * p.wpr + (c0 >> 5)], word);
                if (p.Wp && nvalid > 0) {
                    chunk_apply_mask<BF16>(ch[q], keep_row[q]);
                    chunk_store<BF16>(ch[q], p.Wp, (r0 + q) * p.ld + c0, nvalid);
                }
            }
        }
    }
}

template <bool BF16, int M>
static cudaError_t launch_score(const ScoreParams &p, bool norm_cols, bool group_cols, int grid, cudaStream_t st)
{
    if (group_cols) {
        if (norm_cols) score_group_cols_kernel<BF16, M, true><<<grid, SCORE_THREADS, 0, st>>>(p);
        else score_group_cols_kernel<BF16, M, false><<<grid, SCORE_THREADS, 0, st>>>(p);
    } else {
        if (norm_cols) score_group_rows_kernel<BF16, M, true><<<grid, SCORE_THREADS, 0, st>>>(p);
        else score_group_rows_kernel<BF16, M, false><<<grid, SCORE_THREADS, 0, st>>>(p);
    }
    return cudaGetLastError();
}

int device_sm_count();   // dass_abi.cu
cudaError_t score_nm_bf16_launch(const void *W, int64_t rows, int64_t cols, int64_t ld,
                                 const float *norm, bool norm_cols, float alpha, int n_keep, int m, bool group_cols,
                                 uint32_t *mask_bits, void *W_pruned, cudaStream_t st);   // score_nm_bf16.cu

cudaError_t prune_nm_bf16_launch(const void *W, int64_t rows, int64_t cols, int64_t ld,
                                 const float *norm, bool norm_cols, float alpha, int m, bool group_cols,
                                 uint32_t *mask_bits, void *W_pruned, void *values, uint32_t *meta, cudaStream_t st);   // prune_nm_bf16.cu

static cudaError_t generic_launch(const void *W, int64_t rows, int64_t cols, int64_t ld, bool bf16,
                                  const float *norm, bool norm_cols, float alpha, int n_keep, int m, bool group_cols,
                                  uint32_t *mask_bits, void *W_pruned, void *values, uint32_t *meta, cudaStream_t st);

// Host entry of dass_score_nm (arguments already validated by the C ABI).
cudaError_t score_nm_launch(const void *W, int64_t rows, int64_t cols, int64_t ld, bool bf16,
                            const float *norm, bool norm_cols, float alpha, int n_keep, int m, bool group_cols,
                            uint32_t *mask_bits, void *W_pruned, cudaStream_t st)
{
    if (bf16 && 2 * n_keep == m)   // 2:4 and 4:8: the one-pass kernels of prune_nm_bf16.cu, without the compressed outputs
        return prune_nm_bf16_launch(W, rows, cols, ld, norm, norm_cols, alpha, m, group_cols, mask_bits, W_pruned, nullptr, nullptr, st);
    if (bf16)   // other bf16 patterns: the integer / bit-sliced kernels of score_nm_bf16.cu
        return score_nm_bf16_launch(W, rows, cols, ld, norm, norm_cols, alpha, n_keep, m, group_cols, mask_bits, W_pruned, st);
    return generic_launch(W, rows, cols, ld, false, norm, norm_cols, alpha, n_keep, m, group_cols, mask_bits, W_pruned,
                          nullptr, nullptr, st);
}

// Host entry of dass_prune_nm: every requested output of the selection from one read of W.
cudaError_t prune_nm_launch(const void *W, int64_t rows, int64_t cols, int64_t ld, bool bf16,
                            const float *norm, bool norm_cols, float alpha, int n_keep, int m, bool group_cols,
                            uint32_t *mask_bits, void *W_pruned, void *values, uint32_t *meta, cudaStream_t st)
{
    if (bf16 && 2 * n_keep == m)   // 2:4 and 4:8 on bf16: the tuned one-pass kernels
        return prune_nm_bf16_launch(W, rows, cols, ld, norm, norm_cols, alpha, m, group_cols, mask_bits, W_pruned, values, meta, st);
    return generic_launch(W, rows, cols, ld, bf16, norm, norm_cols, alpha, n_keep, m, group_cols, mask_bits, W_pruned,
                          values, meta, st);
}

static cudaError_t generic_launch(const void *W, int64_t rows, int64_t cols, int64_t ld, bool bf16,
                                  const float *norm, bool norm_cols, float alpha, int n_keep, int m, bool group_cols,
                                  uint32_t *mask_bits, void *W_pruned, void *values, uint32_t *meta, cudaStream_t st)
{
    ScoreParams p;
    p.W = W; p.Wp = W_pruned; p.mask = mask_bits; p.norm = norm;
    p.values = values; p.meta = meta;
    p.rows = rows; p.cols = cols; p.ld = ld;
    p.wpr = (cols + 31) / 32;
    {
        const int field_bits = (n_keep == 2 && m == 4) ? 4 : m;
        const int fpw = 32 / field_bits;
        p.vcols = group_cols ? cols / m * n_keep : cols;
        p.mwpl = group_cols ? (cols / m + fpw - 1) / fpw : (cols + fpw - 1) / fpw;
        const int esz = bf16 ? 2 : 4;
        p.vec_ok = ((p.vcols * esz) % 16 == 0) && ((reinterpret_cast<uintptr_t>(values) & 15u) == 0);
    }
    p.col_blocks = (cols + TILE_COLS - 1) / TILE_COLS;
    p.row_blocks = (rows + TILE_ROWS - 1) / TILE_ROWS;
    p.n_keep = n_keep;
    p.scale_mode = (int)scale_mode_for(alpha);
    p.alpha = alpha;
    const int64_t ntasks = p.col_blocks * p.row_blocks;
    const int64_t warps_per_block = SCORE_THREADS / 32;
    const int64_t want = (ntasks + warps_per_block - 1) / warps_per_block;
    const int64_t cap = (int64_t)device_sm_count() * 8;   // 8 blocks of 256 threads fill an SM
    const int grid = (int)(want < cap ? want : cap);
    if (bf16)
        return m == 4 ? launch_score<true, 4>(p, norm_cols, group_cols, grid, st)
                      : launch_score<true, 8>(p, norm_cols, group_cols, grid, st);
    return m == 4 ? launch_score<false, 4>(p, norm_cols, group_cols, grid, st)
                  : launch_score<false, 8>(p, norm_cols, group_cols, grid, st);
}

}  // namespace dass
