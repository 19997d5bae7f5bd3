// Backward of the bias-fused pass for every storage type: the multiplication of Eq. 4 and the
// column sums of its stored results.  Every product and sum is written with an explicitly
// rounded intrinsic, so the contraction setting of this unit does not matter.
#include "nfad_bias.cuh"
#include "nfad_internal.h"

namespace nfad {

cudaError_t launch_bias_backward(int dtype, const void* g, const void* d, void* gin, float* grad_bias, void* scratch,
                                 size_t rows, size_t cols, cudaStream_t st)
{
    switch (dtype) {
    case kF32:  return launch_bias_backward<StoreF32>(g, d, gin, grad_bias, scratch, rows, cols, st);
    case kBF16: return launch_bias_backward<StoreBF16>(g, d, gin, grad_bias, scratch, rows, cols, st);
    case kF16:  return launch_bias_backward<StoreF16>(g, d, gin, grad_bias, scratch, rows, cols, st);
    }
    return cudaErrorInvalidValue;
}

cudaError_t bias_backward_scratch(int dtype, size_t rows, size_t cols, size_t* bytes)
{
    DeviceInfo di;
    cudaError_t e = device_info(&di);
    if (e != cudaSuccess) return e;
    *bytes = dtype == kF32 ? bias_backward_scratch_bytes<4>(rows, cols, di.sm_count)
                           : bias_backward_scratch_bytes<8>(rows, cols, di.sm_count);
    return cudaSuccess;
}

}  // namespace nfad
