// bf16 / fp16-storage kernels (Fast precision policy: fp32 math on MUFU ex2 /
// rcp, no compensation).  Built with contraction on: nothing here depends on an
// error-free transformation, and fusing across primitive boundaries saves issue
// slots, which for 16-bit storage are as scarce as HBM bytes.
#include "nfad_bias.cuh"
#include "nfad_dispatch.cuh"

namespace nfad {

cudaError_t launch_16(OpCode op, int kind, int dtype, const void* const* in, void* const* out, size_t n, cudaStream_t st)
{
    if (dtype == kBF16) return dispatch_kind<StoreBF16, Fast>(op, kind, in, out, n, st);
    if (dtype == kF16) return dispatch_kind<StoreF16, Fast>(op, kind, in, out, n, st);
    return cudaErrorInvalidValue;
}

template <class S>
static cudaError_t bias_forward_kind(int kind, const void* x, const void* bias, void* y, void* d, size_t rows, size_t cols,
                                     cudaStream_t st)
{
    switch (kind) {
    case kGeluErf:  return launch_bias_forward<S, GeluErf, Fast>(x, bias, y, d, rows, cols, st);
    case kGeluTanh: return launch_bias_forward<S, GeluTanh, Fast>(x, bias, y, d, rows, cols, st);
    case kSwish:    return launch_bias_forward<S, Swish, Fast>(x, bias, y, d, rows, cols, st);
    case kMish:     return launch_bias_forward<S, Mish, Fast>(x, bias, y, d, rows, cols, st);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_bias_forward_16(int kind, int dtype, const void* x, const void* bias, void* y, void* d, size_t rows,
                                   size_t cols, cudaStream_t st)
{
    if (dtype == kBF16) return bias_forward_kind<StoreBF16>(kind, x, bias, y, d, rows, cols, st);
    if (dtype == kF16) return bias_forward_kind<StoreF16>(kind, x, bias, y, d, rows, cols, st);
    return cudaErrorInvalidValue;
}

}  // namespace nfad
