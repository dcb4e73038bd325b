// Stage (b): Eq. 4 / Eq. 5 score and N:M selection in one streaming pass -- the plain formulation with
// exact double products, used for fp32 weights (bf16 weights take the tuned kernels of score_nm_bf16.cu,
// which fall back to the same exact selection on ties).
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

namespace dass {

struct ScoreParams {
    const void *W;
    void *Wp;            // nullable
    uint32_t *mask;      // nullable
    const float *norm;
    int64_t rows, cols, ld;
    int64_t wpr;         // mask words per row
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
                sc[j] = j < nvalid ? (double)scale_from_norm(p.norm[c0 + j], p.scale_mode, p.alpha) : 0.0;
        } else {
            const int64_t r = rb * TILE_ROWS + lane;
            if (r < p.rows) row_scale = scale_from_norm(p.norm[r], p.scale_mode, p.alpha);
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
                if (r < p.rows) {
                    if (p.mask && (lane & 3) == 0 && nvalid > 0) p.mask[r * p.wpr + (c0 >> 5)] = word;
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
                sc[j] = j < nvalid ? (double)scale_from_norm(p.norm[c0 + j], p.scale_mode, p.alpha) : 0.0;
        } else {
            const int64_t r = rb * TILE_ROWS + lane;
            if (r < p.rows) row_scale = scale_from_norm(p.norm[r], p.scale_mode, p.alpha);
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
#pragma unroll
            for (int q = 0; q < M; ++q) {
                const uint32_t word = quad_pack_bytes(keep_row[q], lane);
                if (p.mask && (lane & 3) == 0 && nvalid > 0) p.mask[(r0 + q) * p.wpr + (c0 >> 5)] = word;
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

// Host entry used by the C ABI (arguments already validated there).
cudaError_t score_nm_launch(const void *W, int64_t rows, int64_t cols, int64_t ld, bool bf16,
                            const float *norm, bool norm_cols, float alpha, int n_keep, int m, bool group_cols,
                            uint32_t *mask_bits, void *W_pruned, cudaStream_t st)
{
    if (bf16)   // bf16 weights take the integer / bit-sliced kernels of score_nm_bf16.cu
        return score_nm_bf16_launch(W, rows, cols, ld, norm, norm_cols, alpha, n_keep, m, group_cols, mask_bits, W_pruned, st);
    ScoreParams p;
    p.W = W; p.Wp = W_pruned; p.mask = mask_bits; p.norm = norm;
    p.rows = rows; p.cols = cols; p.ld = ld;
    p.wpr = (cols + 31) / 32;
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
    return m == 4 ? launch_score<false, 4>(p, norm_cols, group_cols, grid, st)
                  : launch_score<false, 8>(p, norm_cols, group_cols, grid, st);
}

}  // namespace dass
