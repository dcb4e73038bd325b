// placeholder until the tensor-core kernel lands
#include "dass_device.cuh"
namespace dass {
int64_t calib_tc_parts(int64_t T, int64_t I) { (void)I; (void)T; return 1; }
dass_status calib_tc_launch(const void *, int64_t, int64_t, const void *, const void *, int64_t, int64_t, int64_t, int,
                            double *, int *, cudaStream_t) { return DASS_ERR_UNSUPPORTED; }
}
