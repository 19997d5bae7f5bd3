// fp32-storage kernels (Full precision policy).  Build with -fmad=false: the
// compensated arithmetic in nfad_numerics.cuh names every fused multiply-add
// explicitly and must not have others introduced by contraction.
#include "nfad_bias.cuh"
#include "nfad_dispatch.cuh"
#include "nfad_strict.cuh"

namespace nfad {

cudaError_t launch_f32(OpCode op, int kind, const void* const* in, void* const* out, size_t n, cudaStream_t st)
{
    if (op == kOpProbe11) return launch_stream<StoreF32, ProbeOp<1, 1>>(in, out, n, st);
    if (op == kOpProbe12) return launch_stream<StoreF32, ProbeOp<1, 2>>(in, out, n, st);
    if (op == kOpProbe21) return launch_stream<StoreF32, ProbeOp<2, 1>>(in, out, n, st);
    if (op == kOpForwardStrict) {
        switch (kind) {
        case kGeluErf:  return launch_stream<StoreF32, ForwardStrictOp<GeluErf>>(in, out, n, st);
        case kGeluTanh: return launch_stream<StoreF32, ForwardStrictOp<GeluTanh>>(in, out, n, st);
        case kSwish:    return launch_stream<StoreF32, ForwardStrictOp<Swish>>(in, out, n, st);
        case kMish:     return launch_stream<StoreF32, ForwardStrictOp<Mish>>(in, out, n, st);
        }
        return cudaErrorInvalidValue;
    }
    return dispatch_kind<StoreF32, Full, false>(op, kind, in, out, n, st);
}

cudaError_t launch_bias_forward_f32(int kind, const void* x, const void* bias, void* y, void* d, size_t rows, size_t cols,
                                    cudaStream_t st)
{
    switch (kind) {
    case kGeluErf:  return launch_bias_forward<StoreF32, GeluErf, Full>(x, bias, y, d, rows, cols, st);
    case kGeluTanh: return launch_bias_forward<StoreF32, GeluTanh, Full>(x, bias, y, d, rows, cols, st);
    case kSwish:    return launch_bias_forward<StoreF32, Swish, Full>(x, bias, y, d, rows, cols, st);
    case kMish:     return launch_bias_forward<StoreF32, Mish, Full>(x, bias, y, d, rows, cols, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace nfad
