// Eq. 1's input-feature norms: sumsq[j] += sum_t X[t,j]^2 (Wanda's ||X_j||_2^2, which the paper uses to prune the
// attention projections).  Feeding sqrt of it to dass_score_nm / dass_select_unstructured with norm_axis = COLS and
// row lines gives Wanda itself.
//
// Bandwidth-bound column reduction: a warp owns 256 columns (a lane 8 consecutive ones, one 16-byte load per row) and a
// slice of the rows; per-slice partial sums go to partial[slice][d] and a second kernel adds the slices in a fixed
// order, so results are bit-reproducible.
#include "dass_device.cuh"

namespace dass {

constexpr int FN_THREADS = 256;
constexpr int FN_MAX_SLICES = 256;

template <bool BF16>
__global__ void __launch_bounds__(FN_THREADS) feature_sumsq_kernel(const void *__restrict__ X, int64_t T, int64_t d, int64_t ldx,
                                                                    int64_t rows_per_slice, int64_t col_blocks, int64_t slices,
                                                                    double *__restrict__ partial /* [slices][d] */)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (FN_THREADS / 32) + (threadIdx.x >> 5);
    const int64_t cb = warp % col_blocks, slice = warp / col_blocks;
    if (slice >= slices) return;          // the last block's spare warps have no slice (and no row of `partial`)
    const int64_t c0 = cb * 256 + lane * 8;
    const int64_t left = d - c0;
    const int nvalid = left >= 8 ? 8 : (left > 0 ? (int)left : 0);
    const int64_t t0 = slice * rows_per_slice;
    double acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.0;
    const int64_t t1 = t0 + rows_per_slice < T ? t0 + rows_per_slice : T;
    if (nvalid > 0) {
        for (int64_t tb = t0; tb < t1; tb += 64) {
            float s[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) s[j] = 0.0f;
            const int64_t te = tb + 64 < t1 ? tb + 64 : t1;
            for (int64_t t = tb; t < te; ++t) {
                Chunk<BF16> ch;
                chunk_load<BF16>(ch, X, t * ldx + c0, nvalid);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float a = chunk_abs<BF16>(ch, j);
                    s[j] = fmaf(a, a, s[j]);
                }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] += (double)s[j];   // 64 fp32 terms at a time, double across blocks
        }
        for (int j = 0; j < nvalid; ++j) DASS_ST(&partial[slice * d + c0 + j], acc[j]);
    }
}

int device_sm_count();   // dass_abi.cu

int64_t feature_slices(int64_t T)
{
    const int64_t want = (T + 255) / 256;
    return want < FN_MAX_SLICES ? (want < 1 ? 1 : want) : FN_MAX_SLICES;
}

cudaError_t feature_sumsq_launch(const void *X, int64_t T, int64_t d, int64_t ldx, bool bf16, double *partial, cudaStream_t st)
{
    const int64_t slices = feature_slices(T);
    const int64_t rows_per_slice = (T + slices - 1) / slices;
    const int64_t col_blocks = (d + 255) / 256;
    const int64_t warps = col_blocks * slices;
    const unsigned grid = (unsigned)((warps + FN_THREADS / 32 - 1) / (FN_THREADS / 32));
    if (bf16) feature_sumsq_kernel<true><<<grid, FN_THREADS, 0, st>>>(X, T, d, ldx, rows_per_slice, col_blocks, slices, partial);
    else feature_sumsq_kernel<false><<<grid, FN_THREADS, 0, st>>>(X, T, d, ldx, rows_per_slice, col_blocks, slices, partial);
    return cudaGetLastError();
}

cudaError_t calib_reduce_launch(const double *partial, int64_t parts, int64_t I, double *sumsq, cudaStream_t st);   // calib_simt.cu

}  // namespace dass

using namespace dass;

extern "C" dass_status dass_feature_workspace_bytes(int64_t T, int64_t d, size_t *bytes)
{
    if (!bytes) return DASS_ERR_NULL;
    if (T < 1 || d < 1) return DASS_ERR_SHAPE;
    *bytes = (size_t)feature_slices(T) * (size_t)d * sizeof(double);
    return DASS_OK;
}

extern "C" dass_status dass_feature_sumsq(const void *X, int64_t T, int64_t d, int64_t ldx, dass_dtype dt,
                                          double *sumsq, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!X || !sumsq) return DASS_ERR_NULL;
    if (dt != DASS_BF16 && dt != DASS_F32) return DASS_ERR_DTYPE;
    if (T < 1 || d < 1 || ldx < d) return DASS_ERR_SHAPE;
    const bool bf16 = dt == DASS_BF16;
    if ((reinterpret_cast<uintptr_t>(X) & 15u) || ldx % (bf16 ? 8 : 4) != 0 || (reinterpret_cast<uintptr_t>(sumsq) & 7u))
        return DASS_ERR_ALIGN;
    size_t need = 0;
    const dass_status qs = dass_feature_workspace_bytes(T, d, &need);
    if (qs != DASS_OK) return qs;
    if (!workspace || workspace_bytes < need) return DASS_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 15u) return DASS_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    double *partial = static_cast<double *>(workspace);
    DASS_BOUNDS_SCOPE(bs);
    DASS_BOUNDS_ADD(bs, X, (size_t)T * ldx * (bf16 ? 2 : 4));
    DASS_BOUNDS_ADD(bs, sumsq, (size_t)d * sizeof(double));
    DASS_BOUNDS_ADD(bs, workspace, workspace_bytes);
    DASS_BOUNDS_COMMIT(bs, st);
    if (feature_sumsq_launch(X, T, d, ldx, bf16, partial, st) != cudaSuccess) return DASS_ERR_CUDA;
    if (calib_reduce_launch(partial, feature_slices(T), d, sumsq, st) != cudaSuccess) return DASS_ERR_CUDA;
    return DASS_OK;
}
