// Run-time FAD sequences and single-operator kernels: the fp32 primitives for 16-bit storage, the
// double-precision ones for fp32 storage.  Built with contraction on, like the 16-bit kernels.
#include "nfad_internal.h"
#include "nfad_seq.cuh"

namespace nfad {

namespace {

unsigned grid_for(size_t items)
{
    size_t blocks = (items + kBlock - 1) / kBlock;
    if (blocks == 0) blocks = 1;
    return (unsigned)(blocks < size_t(0x7fffffff) ? blocks : size_t(0x7fffffff));
}

// Where the packet grid of a call starts: if every tensor has the same offset modulo 16 bytes, `head` elements
// come before the first common 16-byte boundary and whole packets follow; if not, no packet grid exists and every
// element goes through the kernels' element-wise path (head = n), which then gets a grid that fills the device.
struct PacketSplit { size_t head, packets; bool congruent; };

PacketSplit packet_split(const void* const* ptrs, int count, size_t n, size_t esz)
{
    uintptr_t mis = 0;
    bool congruent = true, first = true;
    for (int k = 0; k < count; ++k) {
        if (!ptrs[k]) continue;
        uintptr_t m = reinterpret_cast<uintptr_t>(ptrs[k]) & 15u;
        if (first) { mis = m; first = false; }
        congruent = congruent && m == mis;
    }
    if (!congruent || (mis % esz) != 0) return {n, 0, false};
    size_t head = ((16u - mis) & 15u) / esz;
    if (head > n) head = n;
    return {head, (n - head) / (16 / esz), true};
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
    const void* ptrs[1 + 2 * kSeqMaxOut] = {x};
    for (int k = 0; k < kSeqMaxOut; ++k) {
        a.y[k] = k < m ? y[k] : nullptr;
        a.d[k] = k < m ? d[k] : nullptr;
        ptrs[1 + 2 * k] = a.y[k];
        ptrs[2 + 2 * k] = a.d[k];
    }
    a.m = m;
    a.n = n;
    const PacketSplit sp = packet_split(ptrs, 1 + 2 * kSeqMaxOut, n, sizeof(typename S::elem));
    a.head = sp.head;
    a.packets = sp.packets;
    a.prog = prog;
    return launch_pdl(seq_forward_kernel<S>, sp.congruent ? grid_for(a.packets) : edge_grid_blocks(n, kBlock), st, a);
}

template <class S>
cudaError_t seq_backward_t(const void* const* g, const void* const* d, int m, void* gin, size_t n, cudaStream_t st)
{
    SeqBackwardArgs a;
    const void* ptrs[1 + 2 * kSeqMaxOut] = {gin};
    for (int k = 0; k < kSeqMaxOut; ++k) {
        a.g[k] = k < m ? g[k] : nullptr;
        a.d[k] = k < m ? d[k] : nullptr;
        ptrs[1 + 2 * k] = a.g[k];
        ptrs[2 + 2 * k] = a.d[k];
    }
    a.gin = gin;
    a.m = m;
    a.n = n;
    const PacketSplit sp = packet_split(ptrs, 1 + 2 * kSeqMaxOut, n, sizeof(typename S::elem));
    a.head = sp.head;
    a.packets = sp.packets;
    const int u = seq_bwd_unroll(m);
    const unsigned grid = sp.congruent ? grid_for((a.packets + u - 1) / u) : edge_grid_blocks(n, kBlock);
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
    const void* ptrs[5];
    for (int k = 0; k < 3; ++k) { a.in[k] = in[k]; ptrs[k] = in[k]; }
    for (int k = 0; k < 2; ++k) { a.out[k] = out[k]; ptrs[3 + k] = out[k]; }
    a.op = op;
    a.backward = backward;
    a.c = c;
    a.n = n;
    const PacketSplit sp = packet_split(ptrs, 5, n, sizeof(typename S::elem));
    a.head = sp.head;
    a.packets = sp.packets;
    const unsigned grid = sp.congruent ? grid_for((a.packets + kEwUnroll - 1) / kEwUnroll) : edge_grid_blocks(n, kBlock);
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
