// bf16 / fp16-storage kernels (Fast precision policy: fp32 math on MUFU ex2 /
// rcp, no compensation).  Built with contraction on: nothing here depends on an
// error-free transformation, and fusing across primitive boundaries saves issue
// slots, which for 16-bit storage are as scarce as HBM bytes.
#include "nfad_dispatch.cuh"

namespace nfad {

cudaError_t launch_16(OpCode op, int kind, int dtype, const void* const* in, void* const* out, size_t n, cudaStream_t st)
{
    if (dtype == kBF16) return dispatch_kind<StoreBF16, Fast, true>(op, kind, in, out, n, st);
    if (dtype == kF16) return dispatch_kind<StoreF16, Fast, false>(op, kind, in, out, n, st);
    return cudaErrorInvalidValue;
}

}  // namespace nfad
