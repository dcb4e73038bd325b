// Host side of the checked-access build (see bounds_check.cuh): the report and the test hook.  Both entry points
// exist in the regular build too, where they answer DASS_ERR_UNSUPPORTED.
#include "dass_device.cuh"

using namespace dass;

extern "C" dass_status dass_bounds_report(int *violations, unsigned long long *first_address, int *first_bytes,
                                          int *first_line, void *cuda_stream)
{
    if (!violations) return DASS_ERR_NULL;
#ifdef DASS_BOUNDS_CHECK
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    BoundsReport rep;
    if (cudaMemcpyFromSymbolAsync(&rep, g_bounds_report, sizeof(rep), 0, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return DASS_ERR_CUDA;
    *violations = (int)rep.violations;
    if (first_address) *first_address = rep.first_addr;
    if (first_bytes) *first_bytes = (int)rep.first_bytes;
    if (first_line) *first_line = (int)rep.first_line;
    const BoundsReport zero = {0u, 0u, 0u, 0ull};
    if (cudaMemcpyToSymbolAsync(g_bounds_report, &zero, sizeof(zero), 0, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return DASS_ERR_CUDA;
    return DASS_OK;
#else
    (void)first_address; (void)first_bytes; (void)first_line; (void)cuda_stream;
    *violations = 0;
    return DASS_ERR_UNSUPPORTED;
#endif
}

extern "C" dass_status dass_bounds_shrink_next(size_t bytes)
{
#ifdef DASS_BOUNDS_CHECK
    bounds_shrink_next() = bytes;
    return DASS_OK;
#else
    (void)bytes;
    return DASS_ERR_UNSUPPORTED;
#endif
}
