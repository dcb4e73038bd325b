// Stage (a) for fp32 inputs: Eq. 2 and the per-neuron sum of squares with plain fp32 FMAs.
//
// The tensor cores have no fp32 x fp32 mode (tf32 would drop input bits), so fp32 layers take this
// SIMT path: a classic shared-memory tiled double GEMM (gate and up share the X tile) whose epilogue
// applies the activation, the gating product and the square and sums over the tile's tokens, so the
// intermediate activation never leaves registers.  Each block walks a fixed slice of the tokens and
// writes one partial per neuron; the partials are reduced in a fixed order by calib_reduce_kernel.
// Also holds the small helper kernels shared with the tensor-core path (reduce, finalize).
#include "dass_device.cuh"

namespace dass {

constexpr int S_BN = 64;   // neurons per block tile
constexpr int S_BT = 64;   // tokens per block tile
constexpr int S_BK = 16;
constexpr int S_THREADS = 256;

template <int ACT>
__device__ __forceinline__ float act_accurate(float g)
{
    if constexpr (ACT == DASS_ACT_SILU) {
        return g / (1.0f + expf(-g));
    } else if constexpr (ACT == DASS_ACT_GELU_TANH) {
        const float inner = 0.7978845608028654f * (g + 0.044715f * g * g * g);
        return 0.5f * g * (1.0f + tanhf(inner));
    } else {
        return g > 0.0f ? g : 0.0f;
    }
}

template <int ACT>
__global__ void __launch_bounds__(S_THREADS)
calib_simt_kernel(const float *__restrict__ X, int64_t T, int64_t ldx,
                  const float *__restrict__ Wg, const float *__restrict__ Wu, int64_t I, int64_t d, int64_t ldw,
                  double *__restrict__ partial /* [gridDim.y][I] */, int64_t tiles_per_part)
{
    __shared__ float xs[S_BK][S_BT + 4];
    __shared__ float gs[S_BK][S_BN + 4];
    __shared__ float us[S_BK][S_BN + 4];

    const int tid = threadIdx.x;
    const int tx = tid & 15;    // token sub-tile: tokens tx*4 .. tx*4+3
    const int ty = tid >> 4;    // neuron sub-tile: neurons ty*4 .. ty*4+3
    const int64_t n0 = (int64_t)blockIdx.x * S_BN;
    const int64_t tile_begin = (int64_t)blockIdx.y * tiles_per_part;
    const int64_t ntiles = (T + S_BT - 1) / S_BT;
    const int64_t tile_end = tile_begin + tiles_per_part < ntiles ? tile_begin + tiles_per_part : ntiles;

    double sums[4] = {0.0, 0.0, 0.0, 0.0};

    // loader mapping: 64 rows x 16 k per operand tile, one row-quarter (4 consecutive k) per thread
    const int lrow = tid >> 2;
    const int lk = (tid & 3) * 4;

    for (int64_t tile = tile_begin; tile < tile_end; ++tile) {
        const int64_t t0 = tile * S_BT;
        float accg[4][4], accu[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) accg[a][b] = accu[a][b] = 0.0f;

        for (int64_t k0 = 0; k0 < d; k0 += S_BK) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int64_t k = k0 + lk + e;
                const int64_t t = t0 + lrow, n = n0 + lrow;
                xs[lk + e][lrow] = (t < T && k < d) ? DASS_LD(&X[t * ldx + k]) : 0.0f;
                gs[lk + e][lrow] = (n < I && k < d) ? DASS_LD(&Wg[n * ldw + k]) : 0.0f;
                us[lk + e][lrow] = (n < I && k < d) ? DASS_LD(&Wu[n * ldw + k]) : 0.0f;
            }
            __syncthreads();
#pragma unroll
            for (int kk = 0; kk < S_BK; ++kk) {
                float xv[4], gv[4], uv[4];
#pragma unroll
                for (int b = 0; b < 4; ++b) xv[b] = xs[kk][tx * 4 + b];
#pragma unroll
                for (int a = 0; a < 4; ++a) { gv[a] = gs[kk][ty * 4 + a]; uv[a] = us[kk][ty * 4 + a]; }
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        accg[a][b] = fmaf(gv[a], xv[b], accg[a][b]);
                        accu[a][b] = fmaf(uv[a], xv[b], accu[a][b]);
                    }
            }
            __syncthreads();
        }
        // tokens past T were loaded as zero rows: act(0) * 0 = 0 adds nothing
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            float s = 0.0f;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const float h = act_accurate<ACT>(accg[a][b]) * accu[a][b];
                s = fmaf(h, h, s);
            }
            sums[a] += (double)s;
        }
    }

    // the 16 lanes with equal ty (a half warp) hold the same neurons: fixed-order tree over them
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        double v = sums[a];
#pragma unroll
        for (int off = 8; off >= 1; off >>= 1) v += __shfl_xor_sync(FULL_MASK, v, off);
        const int64_t n = n0 + ty * 4 + a;
        if (tx == 0 && n < I) DASS_ST(&partial[(int64_t)blockIdx.y * I + n], v);
    }
}

// sumsq[i] += partial[0][i] + partial[1][i] + ... in that order (bitwise reproducible).
__global__ void calib_reduce_kernel(const double *__restrict__ partial, int64_t parts, int64_t I,
                                    double *__restrict__ sumsq)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= I) return;
    double s = 0.0;
    for (int64_t p = 0; p < parts; ++p) s += DASS_LD(&partial[p * I + i]);
    DASS_ST(&sumsq[i], DASS_LD(&sumsq[i]) + s);
}

__global__ void norm_finalize_kernel(const double *__restrict__ sumsq, int64_t I, float *__restrict__ norm)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < I) DASS_ST(&norm[i], __double2float_rn(sqrt(DASS_LD(&sumsq[i]))));
}

// word 0: device status; word 1: the tensor-core kernel's alignment counter
__global__ void status_clear_kernel(int *status) { DASS_ST(&status[0], 0); DASS_ST(&status[1], 0); }

int64_t calib_simt_parts(int64_t T)
{
    const int64_t ntiles = (T + S_BT - 1) / S_BT;
    return ntiles < 64 ? ntiles : 64;
}

cudaError_t calib_simt_launch(const float *X, int64_t T, int64_t ldx, const float *Wg, const float *Wu,
                              int64_t I, int64_t d, int64_t ldw, int act, double *partial, cudaStream_t st)
{
    const int64_t ntiles = (T + S_BT - 1) / S_BT;
    const int64_t parts = calib_simt_parts(T);
    const int64_t tiles_per_part = (ntiles + parts - 1) / parts;
    dim3 grid((unsigned)((I + S_BN - 1) / S_BN), (unsigned)parts);
    switch (act) {
    case DASS_ACT_SILU:
        calib_simt_kernel<DASS_ACT_SILU><<<grid, S_THREADS, 0, st>>>(X, T, ldx, Wg, Wu, I, d, ldw, partial, tiles_per_part);
        break;
    case DASS_ACT_GELU_TANH:
        calib_simt_kernel<DASS_ACT_GELU_TANH><<<grid, S_THREADS, 0, st>>>(X, T, ldx, Wg, Wu, I, d, ldw, partial, tiles_per_part);
        break;
    default:
        calib_simt_kernel<DASS_ACT_RELU><<<grid, S_THREADS, 0, st>>>(X, T, ldx, Wg, Wu, I, d, ldw, partial, tiles_per_part);
        break;
    }
    return cudaGetLastError();
}

cudaError_t calib_reduce_launch(const double *partial, int64_t parts, int64_t I, double *sumsq, cudaStream_t st)
{
    calib_reduce_kernel<<<(unsigned)((I + 255) / 256), 256, 0, st>>>(partial, parts, I, sumsq);
    return cudaGetLastError();
}

cudaError_t norm_finalize_launch(const double *sumsq, int64_t I, float *norm, cudaStream_t st)
{
    norm_finalize_kernel<<<(unsigned)((I + 255) / 256), 256, 0, st>>>(sumsq, I, norm);
    return cudaGetLastError();
}

cudaError_t status_clear_launch(int *status, cudaStream_t st)
{
    status_clear_kernel<<<1, 1, 0, st>>>(status);
    return cudaGetLastError();
}

}  // namespace dass
