// fp32-storage kernels (Full precision policy).  Build with -fmad=false: the
// compensated arithmetic in nfad_numerics.cuh names every fused multiply-add
// explicitly and must not have others introduced by contraction.
#include "nfad_dispatch.cuh"

namespace nfad {

cudaError_t launch_f32(OpCode op, int kind, const void* const* in, void* const* out, size_t n, cudaStream_t st)
{
    if (op == kOpProbe11) return launch_stream<StoreF32, ProbeOp<1, 1>>(in, out, n, st);
    if (op == kOpProbe12) return launch_stream<StoreF32, ProbeOp<1, 2>>(in, out, n, st);
    if (op == kOpProbe21) return launch_stream<StoreF32, ProbeOp<2, 1>>(in, out, n, st);
    return dispatch_kind<StoreF32, Full, false>(op, kind, in, out, n, st);
}

}  // namespace nfad
