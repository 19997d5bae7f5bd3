// Run-time FAD sequences and single-operator kernels (Fast policy arithmetic for every
// storage type: plain fp32).  Built with contraction on, like the 16-bit kernels.
#include "nfad_internal.h"
#include "nfad_seq.cuh"

namespace nfad {

namespace {

template <class T> bool aligned16(const T* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

unsigned grid_for(size_t items)
{
    size_t blocks = (items + kBlock - 1) / kBlock;
    if (blocks == 0) blocks = 1;
    return (unsigned)(blocks < size_t(0x7fffffff) ? blocks : size_t(0x7fffffff));
}

template <class K, class A> cudaError_t launch_pdl(K kernel, unsigned grid, cudaStream_t st, const A& args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kBlock);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args);
}

template <class S>
cudaError_t seq_forward_t(const SeqProgram& prog, const void* x, void* const* y, void* const* d, int m, size_t n, cudaStream_t st)
{
    SeqForwardArgs a;
    a.x = x;
    uintptr_t mis = reinterpret_cast<uintptr_t>(x) & 15u;
    bool congruent = true;
    for (int k = 0; k < kSeqMaxOut; ++k) {
        a.y[k] = k < m ? y[k] : nullptr;
        a.d[k] = k < m ? d[k] : nullptr;
        if (k < m) congruent = congruent && ((reinterpret_cast<uintptr_t>(y[k]) & 15u) == mis) && ((reinterpret_cast<uintptr_t>(d[k]) & 15u) == mis);
    }
    a.m = m;
    a.n = n;
    constexpr size_t esz = sizeof(typename S::elem);
    if (congruent) {
        size_t head = ((16u - mis) & 15u) / esz;
        a.head = head > n ? n : head;
        a.packets = (n - a.head) / S::kVec;
    } else {                       // no common packet grid: everything through the element-wise edge path
        a.head = n;
        a.packets = 0;
    }
    a.prog = prog;
    return launch_pdl(seq_forward_kernel<S>, grid_for(a.packets), st, a);
}

template <class S>
cudaError_t seq_backward_t(const void* const* g, const void* const* d, int m, void* gin, size_t n, cudaStream_t st)
{
    SeqBackwardArgs a;
    bool al = aligned16(gin);
    for (int k = 0; k < kSeqMaxOut; ++k) {
        a.g[k] = k < m ? g[k] : nullptr;
        a.d[k] = k < m ? d[k] : nullptr;
        if (k < m) al = al && aligned16(g[k]) && aligned16(d[k]);
    }
    a.gin = gin;
    a.m = m;
    a.n = n;
    a.packets = al ? n / S::kVec : 0;
    const int u = seq_bwd_unroll(m);
    const unsigned grid = grid_for(al ? (a.packets + u - 1) / u : 0);
    switch (m) {
    case 1: return launch_pdl(seq_backward_kernel<S, 1>, grid, st, a);
    case 2: return launch_pdl(seq_backward_kernel<S, 2>, grid, st, a);
    case 3: return launch_pdl(seq_backward_kernel<S, 3>, grid, st, a);
    default: return launch_pdl(seq_backward_kernel<S, 4>, grid, st, a);
    }
}

template <class S>
cudaError_t ew_t(int op, int backward, float c, const void* const* in, void* const* out, size_t n, cudaStream_t st)
{
    EwArgs a;
    bool al = true;
    for (int k = 0; k < 3; ++k) { a.in[k] = in[k]; if (in[k]) al = al && aligned16(in[k]); }
    for (int k = 0; k < 2; ++k) { a.out[k] = out[k]; if (out[k]) al = al && aligned16(out[k]); }
    a.op = op;
    a.backward = backward;
    a.c = c;
    a.n = n;
    a.packets = al ? n / S::kVec : 0;
    const unsigned grid = grid_for(al ? (a.packets + kEwUnroll - 1) / kEwUnroll : 0);
#define NFAD_EW_CASE(OPC) \
    case OPC: return backward ? launch_pdl(ew_kernel<S, OPC, true>, grid, st, a) : launch_pdl(ew_kernel<S, OPC, false>, grid, st, a);
    switch (op) {
        NFAD_EW_CASE(kSeqAdd) NFAD_EW_CASE(kSeqMul) NFAD_EW_CASE(kSeqScale) NFAD_EW_CASE(kSeqAddConst) NFAD_EW_CASE(kSeqExp)
        NFAD_EW_CASE(kSeqLog1p) NFAD_EW_CASE(kSeqTanh) NFAD_EW_CASE(kSeqErf) NFAD_EW_CASE(kSeqSoftplus) NFAD_EW_CASE(kSeqSigmoid)
        NFAD_EW_CASE(kSeqHalfOnePlusTanh) NFAD_EW_CASE(kSeqHalfOnePlusErf)
    }
#undef NFAD_EW_CASE
    return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_seq_forward(const SeqProgramHost& p, int dtype, const void* x, void* const* y, void* const* d, int m, size_t n,
                               cudaStream_t st)
{
    const int mode = seq_executor_mode();
    if (mode != 1) {
        cudaError_t e = launch_seq_forward_compiled(p, dtype, x, y, d, m, n, st);
        if (e == cudaSuccess) {
            seq_note_executor(2);
            return e;
        }
        if (mode == 2 || e != cudaErrorNotSupported) return e;
    }
    seq_note_executor(1);
    SeqProgram prog;
    prog.n_ops = p.n_ops;
    for (int i = 0; i < p.n_ops; ++i) prog.ops[i] = SeqOp{p.op[i], p.a[i], p.b[i], p.dst[i], p.c[i]};
    if (dtype == kF32) return seq_forward_t<StoreF32>(prog, x, y, d, m, n, st);
    if (dtype == kBF16) return seq_forward_t<StoreBF16>(prog, x, y, d, m, n, st);
    return seq_forward_t<StoreF16>(prog, x, y, d, m, n, st);
}

cudaError_t launch_seq_backward(int dtype, const void* const* g, const void* const* d, int m, void* gin, size_t n, cudaStream_t st)
{
    if (dtype == kF32) return seq_backward_t<StoreF32>(g, d, m, gin, n, st);
    if (dtype == kBF16) return seq_backward_t<StoreBF16>(g, d, m, gin, n, st);
    return seq_backward_t<StoreF16>(g, d, m, gin, n, st);
}

cudaError_t launch_ew(int op, int backward, float c, int dtype, const void* const* in, void* const* out, size_t n, cudaStream_t st)
{
    if (dtype == kF32) return ew_t<StoreF32>(op, backward, c, in, out, n, st);
    if (dtype == kBF16) return ew_t<StoreBF16>(op, backward, c, in, out, n, st);
    return ew_t<StoreF16>(op, backward, c, in, out, n, st);
}

}  // namespace nfad
