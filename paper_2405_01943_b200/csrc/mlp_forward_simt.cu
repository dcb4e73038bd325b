// Forward pass of the GLU MLP layer for fp32 tensors (Eq. 2 then Eq. 3) on the CUDA cores: a plain shared-memory
// tiled contraction C[t, n] = sum_k B[t, k] * A[n, k] with fp32 accumulation in ascending k.  With GLU = true two
// A matrices (gate, up) share the B tile and the epilogue applies the activation and the gating product.
// Small fp32 layers only; bf16 layers take the tensor-core kernels.
#include "dass_device.cuh"

namespace dass {

constexpr int FS_TILE = 32;
constexpr int FS_ROWS_PER_THREAD = 4;

template <bool GLU, int ACT>
__global__ void __launch_bounds__(FS_TILE * FS_TILE / FS_ROWS_PER_THREAD)
mlp_forward_simt_kernel(const float *__restrict__ B, int64_t T, int64_t ldb,
                        const float *__restrict__ A0, const float *__restrict__ A1, int64_t n_out, int64_t K, int64_t lda,
                        float *__restrict__ out, int64_t ldo)
{
    __shared__ float sb[FS_TILE][FS_TILE + 1];
    __shared__ float sa0[FS_TILE][FS_TILE + 1];
    __shared__ float sa1[GLU ? FS_TILE : 1][FS_TILE + 1];
    const int tx = threadIdx.x & 31;
    const int ty = threadIdx.x >> 5;                       // 0..7
    const int64_t t0 = (int64_t)blockIdx.y * FS_TILE;
    const int64_t n0 = (int64_t)blockIdx.x * FS_TILE;
    float acc0[FS_ROWS_PER_THREAD] = {0.f, 0.f, 0.f, 0.f};
    float acc1[FS_ROWS_PER_THREAD] = {0.f, 0.f, 0.f, 0.f};
    for (int64_t k0 = 0; k0 < K; k0 += FS_TILE) {
#pragma unroll
        for (int r = 0; r < FS_ROWS_PER_THREAD; ++r) {
            const int row = ty + 8 * r;
            const int64_t k = k0 + tx;
            const bool kin = k < K;
            sb[row][tx] = (kin && t0 + row < T) ? DASS_LD(&B[(t0 + row) * ldb + k]) : 0.f;
            sa0[row][tx] = (kin && n0 + row < n_out) ? DASS_LD(&A0[(n0 + row) * lda + k]) : 0.f;
            if constexpr (GLU) sa1[row][tx] = (kin && n0 + row < n_out) ? DASS_LD(&A1[(n0 + row) * lda + k]) : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int k = 0; k < FS_TILE; ++k) {
            const float a0 = sa0[tx][k];
            const float a1 = GLU ? sa1[tx][k] : 0.f;
#pragma unroll
            for (int r = 0; r < FS_ROWS_PER_THREAD; ++r) {
                const float b = sb[ty + 8 * r][k];
                acc0[r] = fmaf(b, a0, acc0[r]);
                if constexpr (GLU) acc1[r] = fmaf(b, a1, acc1[r]);
            }
        }
        __syncthreads();
    }
    const int64_t n = n0 + tx;
    if (n >= n_out) return;
#pragma unroll
    for (int r = 0; r < FS_ROWS_PER_THREAD; ++r) {
        const int64_t t = t0 + ty + 8 * r;
        if (t >= T) continue;
        if constexpr (GLU) {
            // accurate activation here: fp32 layers are compared with the fp64 definition at 1e-5
            const float g = acc0[r];
            float a;
            if constexpr (ACT == DASS_ACT_SILU) a = g / (1.0f + expf(-g));
            else if constexpr (ACT == DASS_ACT_GELU_TANH) a = 0.5f * g * (1.0f + tanhf(0.7978845608028654f * (g + 0.044715f * g * g * g)));
            else a = fmaxf(g, 0.0f);
            DASS_ST(&out[t * ldo + n], a * acc1[r]);
        } else {
            DASS_ST(&out[t * ldo + n], acc0[r]);
        }
    }
}

cudaError_t mlp_forward_simt_launch(const float *X, int64_t T, int64_t ldx, const float *Wg, const float *Wu,
                                    int64_t I, int64_t d, int64_t ldw, const float *Wd, int64_t ldd, int act,
                                    float *H, int64_t ldh, float *Z, int64_t ldz, cudaStream_t st)
{
    const dim3 block(FS_TILE * FS_TILE / FS_ROWS_PER_THREAD);
    const int64_t ty = (T + FS_TILE - 1) / FS_TILE;
    if (ty > 65535) return cudaErrorInvalidConfiguration;
    const dim3 grid_g((unsigned)((I + FS_TILE - 1) / FS_TILE), (unsigned)ty);
    switch (act) {
    case DASS_ACT_SILU:
        mlp_forward_simt_kernel<true, DASS_ACT_SILU><<<grid_g, block, 0, st>>>(X, T, ldx, Wg, Wu, I, d, ldw, H, ldh); break;
    case DASS_ACT_GELU_TANH:
        mlp_forward_simt_kernel<true, DASS_ACT_GELU_TANH><<<grid_g, block, 0, st>>>(X, T, ldx, Wg, Wu, I, d, ldw, H, ldh); break;
    default:
        mlp_forward_simt_kernel<true, DASS_ACT_RELU><<<grid_g, block, 0, st>>>(X, T, ldx, Wg, Wu, I, d, ldw, H, ldh); break;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const dim3 grid_d((unsigned)((d + FS_TILE - 1) / FS_TILE), (unsigned)ty);
    mlp_forward_simt_kernel<false, DASS_ACT_SILU><<<grid_d, block, 0, st>>>(H, T, ldh, Wd, nullptr, d, I, ldd, Z, ldz);
    return cudaGetLastError();
}

}  // namespace dass
