// dass_calib_accumulate_static: stage (a) for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc at the point where they calibrate: code running
// inside a framework's memory-planned region or allocator callback, plugins that are handed their
// tensors and nothing else, processes whose device-memory budget is fixed up front, and latency
// critical loops where an allocation (an implicit device synchronisation) is unacceptable.  The
// regular entry point makes such callers bring a workspace; this one brings its own: a fixed-size
// scratch array that lives in the library's device image.  It is the same computation through the
// same kernels, only the scratch pointer differs.
//
// The array's name is only a host-side handle.  Its device address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and cached; kernels are always given that address.
#include <atomic>
#include "dass_device.cuh"

namespace dass {

// launchers defined beside the kernels
int64_t calib_simt_parts(int64_t T);
cudaError_t calib_simt_launch(const float *X, int64_t T, int64_t ldx, const float *Wg, const float *Wu,
                              int64_t I, int64_t d, int64_t ldw, int act, double *partial, cudaStream_t st);
cudaError_t calib_reduce_launch(const double *partial, int64_t parts, int64_t I, double *sumsq, cudaStream_t st);
cudaError_t status_clear_launch(int *status, cudaStream_t st);
int calib_tc_band_tiles(int64_t T, int64_t I, int64_t d, int64_t partial_budget_bytes);
int64_t calib_tc_parts_for(int64_t T, int band_tiles);
dass_status calib_tc_launch(const void *X, int64_t T, int64_t ldx, const void *Wg, const void *Wu,
                            int64_t I, int64_t d, int64_t ldw, int act, int band_tiles, double *partial, int *status,
                            cudaStream_t st);

// Held by every GPU that loads this library, until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[DASS_STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
static std::atomic<void *> g_scratch_addr[MAX_DEVICES];   // device address of g_static_scratch, per device ordinal

// One-time set-up for the current device: resolve the symbol to its device address.
static dass_status static_scratch_for_current_device(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return DASS_ERR_CUDA;
    void *ptr = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!ptr) {                         // two host threads may both resolve it: they store the same address
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr) return DASS_ERR_CUDA;
        g_scratch_addr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return DASS_OK;
}

}  // namespace dass

using namespace dass;

extern "C" dass_status dass_calib_accumulate_static(const void *X, int64_t T, int64_t ldx,
                                                    const void *Wg, const void *Wu, int64_t I, int64_t d, int64_t ldw,
                                                    dass_dtype dt, dass_act act, double *sumsq,
                                                    void **scratch_address, void *cuda_stream)
{
    if (!X || !Wg || !Wu || !sumsq) return DASS_ERR_NULL;
    if (dt != DASS_BF16 && dt != DASS_F32) return DASS_ERR_DTYPE;
    if (act != DASS_ACT_SILU && act != DASS_ACT_GELU_TANH && act != DASS_ACT_RELU) return DASS_ERR_DTYPE;
    if (T < 1 || d < 1 || I < 1 || ldx < d || ldw < d) return DASS_ERR_SHAPE;
    const bool bf16 = dt == DASS_BF16;
    const int64_t ldmul = bf16 ? 8 : 4;
    if ((reinterpret_cast<uintptr_t>(X) & 15u) || (reinterpret_cast<uintptr_t>(Wg) & 15u) ||
        (reinterpret_cast<uintptr_t>(Wu) & 15u) || ldx % ldmul || ldw % ldmul ||
        (reinterpret_cast<uintptr_t>(sumsq) & 7u))
        return DASS_ERR_ALIGN;
    // room for the status header and the partial sums of bands of 16 token tiles (bf16) is the least the call needs
    const int64_t parts_min = bf16 ? calib_tc_parts_for(T, 16) : calib_simt_parts(T);
    const size_t need = 256 + (size_t)parts_min * (size_t)I * sizeof(double);
    if (need > (size_t)DASS_STATIC_SCRATCH_BYTES) return DASS_ERR_WORKSPACE;   // too large for the fixed scratch

    void *scratch = nullptr;
    const dass_status ss = static_scratch_for_current_device(&scratch);
    if (ss != DASS_OK) return ss;
    if (scratch_address) *scratch_address = scratch;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int *status = static_cast<int *>(scratch);
    double *partial = reinterpret_cast<double *>(static_cast<unsigned char *>(scratch) + 256);
    DASS_BOUNDS_SCOPE(bs);
    DASS_BOUNDS_ADD(bs, X, (size_t)T * ldx * (bf16 ? 2 : 4));
    DASS_BOUNDS_ADD(bs, Wg, (size_t)I * ldw * (bf16 ? 2 : 4));
    DASS_BOUNDS_ADD(bs, Wu, (size_t)I * ldw * (bf16 ? 2 : 4));
    DASS_BOUNDS_ADD(bs, sumsq, (size_t)I * sizeof(double));
    DASS_BOUNDS_ADD(bs, scratch, (size_t)DASS_STATIC_SCRATCH_BYTES);
    DASS_BOUNDS_COMMIT(bs, st);
    // the status word must start at zero; the partial sums are overwritten in full by the kernels
    if (status_clear_launch(status, st) != cudaSuccess) return DASS_ERR_CUDA;
    int64_t parts;
    if (bf16) {
        const int band_tiles = calib_tc_band_tiles(T, I, d, (int64_t)DASS_STATIC_SCRATCH_BYTES - 256);
        parts = calib_tc_parts_for(T, band_tiles);
        const dass_status ts = calib_tc_launch(X, T, ldx, Wg, Wu, I, d, ldw, (int)act, band_tiles, partial, status, st);
        if (ts != DASS_OK) return ts;
    } else {
        parts = calib_simt_parts(T);
        if (calib_simt_launch(static_cast<const float *>(X), T, ldx, static_cast<const float *>(Wg),
                              static_cast<const float *>(Wu), I, d, ldw, (int)act, partial, st) != cudaSuccess)
            return DASS_ERR_CUDA;
    }
    if (calib_reduce_launch(partial, parts, I, sumsq, st) != cudaSuccess) return DASS_ERR_CUDA;
    return DASS_OK;
}
