// C ABI of the DaSS CUDA library: argument validation and dispatch only.  See include/dass.h.
#include <atomic>
#include <cmath>
#include <cstdint>

#include "dass_device.cuh"

namespace dass {

// kernels' host launchers (defined beside the kernels)
cudaError_t score_nm_launch(const void *W, int64_t rows, int64_t cols, int64_t ld, bool bf16,
                            const float *norm, bool norm_cols, float alpha, int n_keep, int m, bool group_cols,
                            uint32_t *mask_bits, void *W_pruned, cudaStream_t st);
cudaError_t prune_nm_launch(const void *W, int64_t rows, int64_t cols, int64_t ld, bool bf16,
                            const float *norm, bool norm_cols, float alpha, int n_keep, int m, bool group_cols,
                            uint32_t *mask_bits, void *W_pruned, void *values, uint32_t *meta, cudaStream_t st);
cudaError_t prune_status_read(int *host_value, cudaStream_t st);
cudaError_t compress_nm_launch(const void *W, const uint32_t *mask_bits, int64_t rows, int64_t cols, int64_t ld,
                               bool bf16, int n_keep, int m, bool group_cols,
                               void *values, uint32_t *meta, cudaStream_t st);
int64_t calib_simt_parts(int64_t T);
cudaError_t calib_simt_launch(const float *X, int64_t T, int64_t ldx, const float *Wg, const float *Wu,
                              int64_t I, int64_t d, int64_t ldw, int act, double *partial, cudaStream_t st);
cudaError_t calib_reduce_launch(const double *partial, int64_t parts, int64_t I, double *sumsq, cudaStream_t st);
cudaError_t norm_finalize_launch(const double *sumsq, int64_t I, float *norm, cudaStream_t st);
cudaError_t status_clear_launch(int *status, cudaStream_t st);
int64_t calib_tc_parts(int64_t T, int64_t I, int64_t d);
int calib_tc_band_tiles(int64_t T, int64_t I, int64_t d, int64_t partial_budget_bytes);
int64_t calib_tc_parts_for(int64_t T, int band_tiles);
dass_status calib_tc_launch(const void *X, int64_t T, int64_t ldx, const void *Wg, const void *Wu,
                            int64_t I, int64_t d, int64_t ldw, int act, int band_tiles, double *partial, int *status,
                            cudaStream_t st);

cudaError_t bounded_wait_selftest_launch(int *status, unsigned long long limit_ns, cudaStream_t st);

// SM count of the current device (148 when there is none, e.g. for the host-only size queries).  One atomic slot
// per device ordinal, so host threads on different devices never see each other's value.
int device_sm_count()
{
    static std::atomic<int> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return 148;
    int sms = dev < 64 ? cached[dev].load(std::memory_order_relaxed) : 0;
    if (sms <= 0) {
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
        if (dev < 64) cached[dev].store(sms, std::memory_order_relaxed);
    }
    return sms;
}

constexpr size_t WS_HEADER = 256;   // status word + padding; partial sums start here

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline bool ld_ok(int64_t ld, bool bf16) { return ld % (bf16 ? 8 : 4) == 0; }

static dass_status check_nm(int64_t rows, int64_t cols, int64_t ld, int dt, int n_keep, int m, int group_axis)
{
    if (dt != DASS_BF16 && dt != DASS_F32) return DASS_ERR_DTYPE;
    if (group_axis != DASS_AXIS_ROWS && group_axis != DASS_AXIS_COLS) return DASS_ERR_DTYPE;
    if (rows < 1 || cols < 1 || ld < cols) return DASS_ERR_SHAPE;
    if (m != 4 && m != 8) return (m >= 2 && m <= 64) ? DASS_ERR_UNSUPPORTED : DASS_ERR_SHAPE;
    if (n_keep < 1 || n_keep >= m) return DASS_ERR_SHAPE;
    const int64_t extent = group_axis == DASS_AXIS_ROWS ? rows : cols;
    if (extent % m != 0) return DASS_ERR_SHAPE;
    if (!ld_ok(ld, dt == DASS_BF16)) return DASS_ERR_ALIGN;
    return DASS_OK;
}

// Checking build: the address ranges of a stage-(b) call's buffers (sizes as include/dass.h states them).
#ifdef DASS_BOUNDS_CHECK
static void register_nm_ranges(BoundsScope &bs, const void *W, int64_t rows, int64_t cols, int64_t ld, int dt,
                               const float *norm, int norm_axis, int n_keep, int m, int group_axis,
                               const uint32_t *mask_bits, const void *W_pruned, const void *values, const uint32_t *meta)
{
    const size_t esz = dt == DASS_BF16 ? 2 : 4;
    bs.add(W, (size_t)rows * ld * esz);
    bs.add(W_pruned, (size_t)rows * ld * esz);
    bs.add(norm, (size_t)(norm_axis == DASS_AXIS_ROWS ? rows : cols) * sizeof(float));
    bs.add(mask_bits, (size_t)rows * ((cols + 31) / 32) * sizeof(uint32_t));
    const int field_bits = (n_keep == 2 && m == 4) ? 4 : m;
    const int64_t fpw = 32 / field_bits;
    if (group_axis == DASS_AXIS_COLS) {
        bs.add(values, (size_t)rows * (cols / m * n_keep) * esz);
        bs.add(meta, (size_t)rows * ((cols / m + fpw - 1) / fpw) * sizeof(uint32_t));
    } else {
        bs.add(values, (size_t)(rows / m * n_keep) * cols * esz);
        bs.add(meta, (size_t)(rows / m) * ((cols + fpw - 1) / fpw) * sizeof(uint32_t));
    }
}
#define DASS_BOUNDS_REF(name) (name)
#else
#define register_nm_ranges(...) do { } while (0)
#define DASS_BOUNDS_REF(name) 0
#endif

}  // namespace dass

using namespace dass;

extern "C" {

const char *dass_status_string(dass_status s)
{
    switch (s) {
    case DASS_OK: return "ok";
    case DASS_ERR_NULL: return "null pointer";
    case DASS_ERR_SHAPE: return "bad shape";
    case DASS_ERR_ALIGN: return "bad alignment";
    case DASS_ERR_DTYPE: return "bad enum value";
    case DASS_ERR_UNSUPPORTED: return "unsupported";
    case DASS_ERR_WORKSPACE: return "workspace too small";
    case DASS_ERR_CUDA: return "CUDA error";
    case DASS_ERR_TIMEOUT: return "device-side wait timed out";
    case DASS_ERR_INTERNAL: return "passes of a kernel chain disagree";
    }
    return "unknown status";
}

int dass_version(void) { return 100; }

dass_status dass_calib_workspace_bytes(int64_t T, int64_t d, int64_t I, dass_dtype dt, size_t *bytes)
{
    if (!bytes) return DASS_ERR_NULL;
    if (dt != DASS_BF16 && dt != DASS_F32) return DASS_ERR_DTYPE;
    if (T < 1 || d < 1 || I < 1) return DASS_ERR_SHAPE;
    const int64_t parts = dt == DASS_BF16 ? calib_tc_parts(T, I, d) : calib_simt_parts(T);
    *bytes = WS_HEADER + (size_t)parts * (size_t)I * sizeof(double);
    return DASS_OK;
}

dass_status dass_calib_accumulate(const void *X, int64_t T, int64_t ldx,
                                  const void *Wg, const void *Wu, int64_t I, int64_t d, int64_t ldw,
                                  dass_dtype dt, dass_act act, double *sumsq,
                                  void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!X || !Wg || !Wu || !sumsq) return DASS_ERR_NULL;
    if (dt != DASS_BF16 && dt != DASS_F32) return DASS_ERR_DTYPE;
    if (act != DASS_ACT_SILU && act != DASS_ACT_GELU_TANH && act != DASS_ACT_RELU) return DASS_ERR_DTYPE;
    if (T < 1 || d < 1 || I < 1 || ldx < d || ldw < d) return DASS_ERR_SHAPE;
    const bool bf16 = dt == DASS_BF16;
    if (!aligned16(X) || !aligned16(Wg) || !aligned16(Wu) || !ld_ok(ldx, bf16) || !ld_ok(ldw, bf16)) return DASS_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(sumsq) & 7u) != 0) return DASS_ERR_ALIGN;
    // The query's size is what the call would like; what it needs is room for bands of 16 token tiles (bf16), so
    // a workspace sized by the query for some token count also serves every shorter batch.
    const int64_t parts_min = bf16 ? calib_tc_parts_for(T, 16) : calib_simt_parts(T);
    const size_t need = WS_HEADER + (size_t)parts_min * (size_t)I * sizeof(double);
    if (!workspace || workspace_bytes < need) return DASS_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return DASS_ERR_ALIGN;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int *status = static_cast<int *>(workspace);
    double *partial = reinterpret_cast<double *>(static_cast<char *>(workspace) + WS_HEADER);
    DASS_BOUNDS_SCOPE(bs);
    DASS_BOUNDS_ADD(bs, X, (size_t)T * ldx * (bf16 ? 2 : 4));
    DASS_BOUNDS_ADD(bs, Wg, (size_t)I * ldw * (bf16 ? 2 : 4));
    DASS_BOUNDS_ADD(bs, Wu, (size_t)I * ldw * (bf16 ? 2 : 4));
    DASS_BOUNDS_ADD(bs, sumsq, (size_t)I * sizeof(double));
    DASS_BOUNDS_ADD(bs, workspace, workspace_bytes);
    DASS_BOUNDS_COMMIT(bs, st);
    if (status_clear_launch(status, st) != cudaSuccess) return DASS_ERR_CUDA;
    int64_t parts;
    if (bf16) {
        const int band_tiles = calib_tc_band_tiles(T, I, d, (int64_t)(workspace_bytes - WS_HEADER));
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

dass_status dass_calib_status(const void *workspace, void *cuda_stream)
{
    if (!workspace) return DASS_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int host = 0;
    if (cudaMemcpyAsync(&host, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return DASS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return DASS_ERR_CUDA;
    return host == 0 ? DASS_OK : DASS_ERR_TIMEOUT;
}

dass_status dass_selftest_wait_timeout(void *status_word, int64_t limit_us, void *cuda_stream)
{
    if (!status_word) return DASS_ERR_NULL;
    if (limit_us < 1 || limit_us > 1000000) return DASS_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(status_word) & 3u) return DASS_ERR_ALIGN;
    DASS_BOUNDS_SCOPE(bs);
    DASS_BOUNDS_ADD(bs, status_word, sizeof(int));
    DASS_BOUNDS_COMMIT(bs, static_cast<cudaStream_t>(cuda_stream));
    if (bounded_wait_selftest_launch(static_cast<int *>(status_word), (unsigned long long)limit_us * 1000ull,
                                     static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return DASS_ERR_CUDA;
    return DASS_OK;
}

dass_status dass_norm_finalize(const double *sumsq, int64_t I, float *norm, void *cuda_stream)
{
    if (!sumsq || !norm) return DASS_ERR_NULL;
    if (I < 1) return DASS_ERR_SHAPE;
    DASS_BOUNDS_SCOPE(bs);
    DASS_BOUNDS_ADD(bs, sumsq, (size_t)I * sizeof(double));
    DASS_BOUNDS_ADD(bs, norm, (size_t)I * sizeof(float));
    DASS_BOUNDS_COMMIT(bs, static_cast<cudaStream_t>(cuda_stream));
    if (norm_finalize_launch(sumsq, I, norm, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return DASS_ERR_CUDA;
    return DASS_OK;
}

dass_status dass_score_nm(const void *W, int64_t rows, int64_t cols, int64_t ld, dass_dtype dt,
                          const float *norm, dass_axis norm_axis, float alpha,
                          int n_keep, int m, dass_axis group_axis,
                          uint32_t *mask_bits, void *W_pruned, void *cuda_stream)
{
    if (!W || !norm || (!mask_bits && !W_pruned)) return DASS_ERR_NULL;
    if (norm_axis != DASS_AXIS_ROWS && norm_axis != DASS_AXIS_COLS) return DASS_ERR_DTYPE;
    const dass_status cs = check_nm(rows, cols, ld, (int)dt, n_keep, m, (int)group_axis);
    if (cs != DASS_OK) return cs;
    if (!std::isfinite(alpha) || alpha < 0.0f) return DASS_ERR_UNSUPPORTED;
    if (!aligned16(W) || (W_pruned && !aligned16(W_pruned))) return DASS_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(norm) & 3u) || (reinterpret_cast<uintptr_t>(mask_bits) & 3u)) return DASS_ERR_ALIGN;
    DASS_BOUNDS_SCOPE(bs);
    register_nm_ranges(DASS_BOUNDS_REF(bs), W, rows, cols, ld, dt, norm, norm_axis, n_keep, m, group_axis, mask_bits, W_pruned, nullptr, nullptr);
    DASS_BOUNDS_COMMIT(bs, static_cast<cudaStream_t>(cuda_stream));
    if (score_nm_launch(W, rows, cols, ld, dt == DASS_BF16, norm, norm_axis == DASS_AXIS_COLS, alpha, n_keep, m,
                        group_axis == DASS_AXIS_COLS, mask_bits, W_pruned,
                        static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return DASS_ERR_CUDA;
    return DASS_OK;
}

dass_status dass_prune_nm(const void *W, int64_t rows, int64_t cols, int64_t ld, dass_dtype dt,
                          const float *norm, dass_axis norm_axis, float alpha,
                          int n_keep, int m, dass_axis group_axis,
                          uint32_t *mask_bits, void *W_pruned, void *values, uint32_t *meta, void *cuda_stream)
{
    if (!W || !norm || (!mask_bits && !W_pruned && !values)) return DASS_ERR_NULL;
    if ((values == nullptr) != (meta == nullptr)) return DASS_ERR_NULL;      // the compressed form is both or neither
    if (norm_axis != DASS_AXIS_ROWS && norm_axis != DASS_AXIS_COLS) return DASS_ERR_DTYPE;
    const dass_status cs = check_nm(rows, cols, ld, (int)dt, n_keep, m, (int)group_axis);
    if (cs != DASS_OK) return cs;
    if (!std::isfinite(alpha) || alpha < 0.0f) return DASS_ERR_UNSUPPORTED;
    if (!aligned16(W) || (W_pruned && !aligned16(W_pruned))) return DASS_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(norm) & 3u) || (reinterpret_cast<uintptr_t>(mask_bits) & 3u) ||
        (reinterpret_cast<uintptr_t>(meta) & 3u))
        return DASS_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(values) & (dt == DASS_BF16 ? 1u : 3u)) return DASS_ERR_ALIGN;
    DASS_BOUNDS_SCOPE(bs);
    register_nm_ranges(DASS_BOUNDS_REF(bs), W, rows, cols, ld, dt, norm, norm_axis, n_keep, m, group_axis, mask_bits, W_pruned, values, meta);
    DASS_BOUNDS_COMMIT(bs, static_cast<cudaStream_t>(cuda_stream));
    if (prune_nm_launch(W, rows, cols, ld, dt == DASS_BF16, norm, norm_axis == DASS_AXIS_COLS, alpha, n_keep, m,
                        group_axis == DASS_AXIS_COLS, mask_bits, W_pruned, values, meta,
                        static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return DASS_ERR_CUDA;
    return DASS_OK;
}

dass_status dass_prune_status(void *cuda_stream)
{
    int value = 0;
    if (prune_status_read(&value, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return DASS_ERR_CUDA;
    return value == DASS_ERR_INTERNAL ? DASS_ERR_INTERNAL : (value == 0 ? DASS_OK : DASS_ERR_TIMEOUT);
}

dass_status dass_compress_nm(const void *W, const uint32_t *mask_bits,
                             int64_t rows, int64_t cols, int64_t ld, dass_dtype dt,
                             int n_keep, int m, dass_axis group_axis,
                             void *values, uint32_t *meta, void *cuda_stream)
{
    if (!W || !mask_bits || !values || !meta) return DASS_ERR_NULL;
    const dass_status cs = check_nm(rows, cols, ld, (int)dt, n_keep, m, (int)group_axis);
    if (cs != DASS_OK) return cs;
    if (!aligned16(W)) return DASS_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(mask_bits) & 3u) || (reinterpret_cast<uintptr_t>(meta) & 3u)) return DASS_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(values) & (dt == DASS_BF16 ? 1u : 3u)) return DASS_ERR_ALIGN;
    DASS_BOUNDS_SCOPE(bs);
    register_nm_ranges(DASS_BOUNDS_REF(bs), W, rows, cols, ld, dt, nullptr, DASS_AXIS_ROWS, n_keep, m, group_axis, mask_bits, nullptr, values, meta);
    DASS_BOUNDS_COMMIT(bs, static_cast<cudaStream_t>(cuda_stream));
    if (compress_nm_launch(W, mask_bits, rows, cols, ld, dt == DASS_BF16, n_keep, m, group_axis == DASS_AXIS_COLS,
                           values, meta, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return DASS_ERR_CUDA;
    return DASS_OK;
}

}  // extern "C"
