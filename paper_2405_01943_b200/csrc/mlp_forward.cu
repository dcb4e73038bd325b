// C ABI of the layer's forward pass (Eq. 2 then Eq. 3): validation, token chunking and dispatch.
// See include/dass.h.  The kernels are in mlp_forward_tc.cu (bf16) and mlp_forward_simt.cu (fp32).
#include <cstdint>

#include "dass_device.cuh"

namespace dass {

dass_status mlp_forward_tc_launch(const void *X, int64_t T, int64_t ldx, const void *Wg, const void *Wu,
                                  int64_t I, int64_t d, int64_t ldw, const void *Wd, int64_t ldd, int act,
                                  void *H, int64_t ldh, void *Z, int64_t ldz, int *words, cudaStream_t st);
cudaError_t mlp_forward_counters_clear(int *words, cudaStream_t st);
cudaError_t mlp_forward_simt_launch(const float *X, int64_t T, int64_t ldx, const float *Wg, const float *Wu,
                                    int64_t I, int64_t d, int64_t ldw, const float *Wd, int64_t ldd, int act,
                                    float *H, int64_t ldh, float *Z, int64_t ldz, cudaStream_t st);
cudaError_t status_clear_launch(int *status, cudaStream_t st);   // calib_simt.cu

constexpr size_t FWD_HEADER = 256;        // status word and alignment counters; the H buffer starts here
constexpr int64_t FWD_MIN_ROWS = 256;     // smallest token chunk (one token tile)
constexpr int64_t FWD_BAND_ROWS = 4096;   // chunks of whole 16-tile bands keep the L2 sharing pattern intact

static inline int64_t fwd_ldh(int64_t I, bool bf16) { return bf16 ? (I + 7) / 8 * 8 : (I + 3) / 4 * 4; }
static inline bool fwd_aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace dass

using namespace dass;

extern "C" {

dass_status dass_mlp_forward_workspace_bytes(int64_t T, int64_t d, int64_t I, dass_dtype dt,
                                             size_t *min_bytes, size_t *full_bytes)
{
    if (!min_bytes && !full_bytes) return DASS_ERR_NULL;
    if (dt != DASS_BF16 && dt != DASS_F32) return DASS_ERR_DTYPE;
    if (T < 1 || d < 1 || I < 1) return DASS_ERR_SHAPE;
    const bool bf16 = dt == DASS_BF16;
    const size_t row_bytes = (size_t)fwd_ldh(I, bf16) * (bf16 ? 2 : 4);
    const int64_t rows_min = T < FWD_MIN_ROWS ? T : FWD_MIN_ROWS;
    if (min_bytes) *min_bytes = FWD_HEADER + (size_t)rows_min * row_bytes;
    if (full_bytes) *full_bytes = FWD_HEADER + (size_t)T * row_bytes;
    return DASS_OK;
}

dass_status dass_mlp_forward(const void *X, int64_t T, int64_t ldx,
                             const void *Wg, const void *Wu, int64_t I, int64_t d, int64_t ldw,
                             const void *Wd, int64_t ldd, dass_dtype dt, dass_act act,
                             void *Z, int64_t ldz, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!X || !Wg || !Wu || !Wd || !Z) return DASS_ERR_NULL;
    if (dt != DASS_BF16 && dt != DASS_F32) return DASS_ERR_DTYPE;
    if (act != DASS_ACT_SILU && act != DASS_ACT_GELU_TANH && act != DASS_ACT_RELU) return DASS_ERR_DTYPE;
    if (T < 1 || d < 1 || I < 1 || ldx < d || ldw < d || ldd < I || ldz < d) return DASS_ERR_SHAPE;
    const bool bf16 = dt == DASS_BF16;
    const int64_t unit = bf16 ? 8 : 4;
    if (!fwd_aligned16(X) || !fwd_aligned16(Wg) || !fwd_aligned16(Wu) || !fwd_aligned16(Wd)) return DASS_ERR_ALIGN;
    if (ldx % unit || ldw % unit || ldd % unit) return DASS_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(Z) & (bf16 ? 1u : 3u)) return DASS_ERR_ALIGN;
    if (!bf16 && T > 65535ll * 32) return DASS_ERR_UNSUPPORTED;       // the fp32 kernels' grid limit
    size_t need = 0;
    const dass_status qs = dass_mlp_forward_workspace_bytes(T, d, I, dt, &need, nullptr);
    if (qs != DASS_OK) return qs;
    if (!workspace || workspace_bytes < need) return DASS_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return DASS_ERR_ALIGN;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int *words = static_cast<int *>(workspace);
    char *hbuf = static_cast<char *>(workspace) + FWD_HEADER;
    const int64_t ldh = fwd_ldh(I, bf16);
    const size_t elt = bf16 ? 2 : 4;
    const size_t row_bytes = (size_t)ldh * elt;

    // tokens per chunk: all of them when the H buffer holds them, else whole bands, else whole token tiles
    int64_t rows = (int64_t)((workspace_bytes - FWD_HEADER) / row_bytes);
    if (rows >= T) rows = T;
    else if (rows >= FWD_BAND_ROWS) rows -= rows % FWD_BAND_ROWS;
    else rows -= rows % FWD_MIN_ROWS;
    if (rows < 1) return DASS_ERR_WORKSPACE;

    DASS_BOUNDS_SCOPE(bs);
    DASS_BOUNDS_ADD(bs, X, (size_t)T * ldx * elt);
    DASS_BOUNDS_ADD(bs, Wg, (size_t)I * ldw * elt);
    DASS_BOUNDS_ADD(bs, Wu, (size_t)I * ldw * elt);
    DASS_BOUNDS_ADD(bs, Wd, (size_t)d * ldd * elt);
    DASS_BOUNDS_ADD(bs, Z, ((size_t)(T - 1) * ldz + d) * elt);
    DASS_BOUNDS_ADD(bs, workspace, workspace_bytes);
    DASS_BOUNDS_COMMIT(bs, st);
    if (status_clear_launch(words, st) != cudaSuccess) return DASS_ERR_CUDA;
    for (int64_t t0 = 0; t0 < T; t0 += rows) {
        const int64_t tc = T - t0 < rows ? T - t0 : rows;
        const char *xc = static_cast<const char *>(X) + (size_t)t0 * (size_t)ldx * elt;
        char *zc = static_cast<char *>(Z) + (size_t)t0 * (size_t)ldz * elt;
        if (bf16) {
            if (mlp_forward_counters_clear(words, st) != cudaSuccess) return DASS_ERR_CUDA;
            const dass_status s = mlp_forward_tc_launch(xc, tc, ldx, Wg, Wu, I, d, ldw, Wd, ldd, (int)act,
                                                        hbuf, ldh, zc, ldz, words, st);
            if (s != DASS_OK) return s;
        } else {
            if (mlp_forward_simt_launch(reinterpret_cast<const float *>(xc), tc, ldx, static_cast<const float *>(Wg),
                                        static_cast<const float *>(Wu), I, d, ldw, static_cast<const float *>(Wd), ldd,
                                        (int)act, reinterpret_cast<float *>(hbuf), ldh, reinterpret_cast<float *>(zc), ldz,
                                        st) != cudaSuccess)
                return DASS_ERR_CUDA;
        }
    }
    return DASS_OK;
}

}  // extern "C"
