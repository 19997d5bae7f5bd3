// nfad_seq.cuh -- FAD sequences composed at run time.
//
// A FAD sequence (Section IV: the run of fad operators between the NY and YN
// states) is a straight-line program over at most kSeqRegs dual registers;
// register 0 holds the seed (x, 1).  Every instruction is one primitive operation
// of Section III-A: unary, binary with both inputs from the same source (add, mul:
// the "merge" of two branches), or binary with a constant.  OUT copies a register
// to one of m <= kSeqMaxOut outputs: one source, M results (R^1 -> R^M).  One kernel
// interprets the whole program per element on dual numbers, so no intermediate and
// no intermediate derivative reaches memory; per output only y_k and dy_k/dx do.
//
// The program is the same for every element, so the interpreter's control flow is
// uniform; registers are indexed at run time and therefore live in local memory.
// This executor trades speed for generality; the four activations of Table I have
// the dedicated kernels.
#pragma once

#include "nfad_dual.cuh"
#include "nfad_stream.cuh"

namespace nfad {

constexpr int kSeqMaxOps = 32;
constexpr int kSeqRegs = 12;
constexpr int kSeqMaxOut = 4;

enum SeqOpcode {
    kSeqAdd = 0, kSeqMul = 1, kSeqScale = 2, kSeqAddConst = 3, kSeqExp = 4, kSeqLog1p = 5, kSeqTanh = 6, kSeqErf = 7,
    kSeqSoftplus = 8, kSeqSigmoid = 9, kSeqHalfOnePlusTanh = 10, kSeqHalfOnePlusErf = 11, kSeqOut = 12, kSeqOpcodeCount = 13
};

struct SeqOp { int op, a, b, dst; float c; };
struct SeqProgram { int n_ops; SeqOp ops[kSeqMaxOps]; };

// The policy a storage type's sequences run under, and that policy's scalar: fp32 tensors get the double-precision
// primitives (results within an fp32 rounding or two of the exact ones), 16-bit tensors the fp32 ones.
template <class S> struct SeqPolicy { using type = Fast; };
template <> struct SeqPolicy<StoreF32> { using type = Wide; };
template <class P> struct ScalarOf { using type = float; };
template <> struct ScalarOf<Wide> { using type = double; };

// One primitive on duals.
template <class P>
__device__ __forceinline__ Dual<P> seq_apply(const SeqOp& o, const Dual<P>& a, const Dual<P>& b)
{
    using T = typename ScalarOf<P>::type;
    switch (o.op) {
    case kSeqAdd: return dual_add(a, b);
    case kSeqMul: return dual_mul(a, b);
    case kSeqScale: return dual_scale(T(o.c), a);
    case kSeqAddConst: return dual_add_const(T(o.c), a);
    case kSeqExp: return dual_exp(a);
    case kSeqLog1p: return dual_log1p(a);
    case kSeqTanh: return dual_tanh(a);
    case kSeqErf: return dual_erf(a);
    case kSeqSoftplus: return dual_softplus(a);
    case kSeqSigmoid: return as_dual(dual_sigmoid(a));
    case kSeqHalfOnePlusTanh: return as_dual(dual_half_one_plus_tanh(a));
    case kSeqHalfOnePlusErf: return as_dual(dual_half_one_plus_erf(a));
    default: return a;
    }
}

// Interprets the program for V elements, kSeqGroup at a time: the register file is indexed at
// run time and so lives in local memory, and kSeqRegs x 2 x kSeqGroup scalars per thread is what
// has to stay inside L1 for every resident thread.
constexpr int kSeqGroup = 2;

template <class P, int V>
__device__ __forceinline__ void seq_run(const SeqProgram& prog, const float (&x)[V], float (&yv)[kSeqMaxOut][V],
                                        float (&yt)[kSeqMaxOut][V])
{
    using T = typename ScalarOf<P>::type;
    constexpr int G = V < kSeqGroup ? V : kSeqGroup;
#pragma unroll
    for (int e0 = 0; e0 < V; e0 += G) {
        T rv[kSeqRegs][G], rt[kSeqRegs][G];
#pragma unroll
        for (int e = 0; e < G; ++e) { rv[0][e] = T(x[e0 + e]); rt[0][e] = T(1); }
        for (int i = 0; i < prog.n_ops; ++i) {
            const SeqOp o = prog.ops[i];
            if (o.op == kSeqOut) {
#pragma unroll
                for (int e = 0; e < G; ++e) {
                    const Dual<P> r{rv[o.a][e], rt[o.a][e]};
                    yv[o.dst][e0 + e] = dual_value(r);
                    yt[o.dst][e0 + e] = dual_tangent(r);
                }
            } else {
#pragma unroll
                for (int e = 0; e < G; ++e) {
                    Dual<P> r = seq_apply<P>(o, Dual<P>{rv[o.a][e], rt[o.a][e]}, Dual<P>{rv[o.b][e], rt[o.b][e]});
                    rv[o.dst][e] = r.v;
                    rt[o.dst][e] = r.t;
                }
            }
        }
    }
}

struct SeqForwardArgs {
    const void* x;
    void* y[kSeqMaxOut];
    void* d[kSeqMaxOut];
    int m;
    size_t n, head, packets;
    SeqProgram prog;
};

template <class S>
__global__ void __launch_bounds__(kBlock) seq_forward_kernel(const SeqForwardArgs a)
{
    using E = typename S::elem;
    constexpr int V = S::kVec;
    const size_t byte_off = a.head * sizeof(E);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (size_t pk = size_t(blockIdx.x) * kBlock + threadIdx.x; pk < a.packets; pk += size_t(gridDim.x) * kBlock) {
        uint4 raw = load_packet(reinterpret_cast<const uint4*>(static_cast<const char*>(a.x) + byte_off) + pk);
        float xv[V], yv[kSeqMaxOut][V], yt[kSeqMaxOut][V];
        S::unpack(raw, xv);
        seq_run<typename SeqPolicy<S>::type, V>(a.prog, xv, yv, yt);
        for (int k = 0; k < a.m; ++k) {
            *(reinterpret_cast<uint4*>(static_cast<char*>(a.y[k]) + byte_off) + pk) = S::pack(yv[k]);
            __stcs(reinterpret_cast<uint4*>(static_cast<char*>(a.d[k]) + byte_off) + pk, S::pack(yt[k]));
        }
    }
    // elements outside the packet grid, one by one, spread over the whole grid: a few at the ragged ends when the tensors
    // share one offset modulo 16 bytes, all n of them when they do not (head = n, packets = 0)
    {
        const size_t tail_begin = a.head + a.packets * V;
        const size_t n_edge = a.head + (a.n - tail_begin);
        for (size_t j = size_t(blockIdx.x) * kBlock + threadIdx.x; j < n_edge; j += size_t(gridDim.x) * kBlock) {
            const size_t i = j < a.head ? j : tail_begin + (j - a.head);
            float xv[1] = {S::load1(static_cast<const E*>(a.x) + i)};
            float yv[kSeqMaxOut][1], yt[kSeqMaxOut][1];
            seq_run<typename SeqPolicy<S>::type, 1>(a.prog, xv, yv, yt);
            for (int k = 0; k < a.m; ++k) {
                S::store1(static_cast<E*>(a.y[k]) + i, yv[k][0]);
                S::store1(static_cast<E*>(a.d[k]) + i, yt[k][0]);
            }
        }
    }
}

// Backward of a sequence with M outputs (Section II-E: the transposed Jacobian of the whole
// sequence applied to the upstream gradients): grad_in = sum_k grad_out_k * dy_k/dx, accumulated
// in fp32 in the order k = 0 .. m-1 with fused multiply-adds, rounded once at the store.
struct SeqBackwardArgs {
    const void* g[kSeqMaxOut];
    const void* d[kSeqMaxOut];
    void* gin;
    int m;
    size_t n;
    size_t head;       // elements before the first 16-byte boundary (the same for every tensor; n if they do not agree)
    size_t packets;    // whole 16-byte packets after the head
};

// M is a template parameter so that all 2 M loads of a packet are issued before the first use; a CTA takes one
// tile of kBlock * U packets, U = 2 for one or two results and 1 beyond (what 64 registers hold).
__host__ __device__ constexpr int seq_bwd_unroll(int m) { return m <= 2 ? 2 : 1; }

template <class S, int M>
__global__ void __launch_bounds__(kBlock, 4) seq_backward_kernel(const SeqBackwardArgs a)
{
    using E = typename S::elem;
    constexpr int V = S::kVec;
    constexpr int U = seq_bwd_unroll(M);
    const size_t byte_off = a.head * sizeof(E);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const size_t tile = size_t(kBlock) * U;
    for (size_t base = size_t(blockIdx.x) * tile + threadIdx.x; base < a.packets; base += size_t(gridDim.x) * tile) {
        uint4 rg[U][M], rd[U][M];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t pk = base + size_t(u) * kBlock;
            if (pk < a.packets) {
#pragma unroll
                for (int k = 0; k < M; ++k) {
                    rg[u][k] = load_packet(reinterpret_cast<const uint4*>(static_cast<const char*>(a.g[k]) + byte_off) + pk);
                    rd[u][k] = load_packet(reinterpret_cast<const uint4*>(static_cast<const char*>(a.d[k]) + byte_off) + pk);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t pk = base + size_t(u) * kBlock;
            if (pk >= a.packets) continue;
            float acc[V], gv[V], dv[V];
            S::unpack(rg[u][0], gv);
            S::unpack(rd[u][0], dv);
#pragma unroll
            for (int e = 0; e < V; ++e) acc[e] = gv[e] * dv[e];
#pragma unroll
            for (int k = 1; k < M; ++k) {
                S::unpack(rg[u][k], gv);
                S::unpack(rd[u][k], dv);
#pragma unroll
                for (int e = 0; e < V; ++e) acc[e] = fmaf(gv[e], dv[e], acc[e]);
            }
            *(reinterpret_cast<uint4*>(static_cast<char*>(a.gin) + byte_off) + pk) = S::pack(acc);
        }
    }
    {   // outside the packet grid: spread over the whole grid (see seq_forward_kernel)
        const size_t tail_begin = a.head + a.packets * V;
        const size_t n_edge = a.head + (a.n - tail_begin);
        for (size_t j = size_t(blockIdx.x) * kBlock + threadIdx.x; j < n_edge; j += size_t(gridDim.x) * kBlock) {
            const size_t i = j < a.head ? j : tail_begin + (j - a.head);
            float acc = S::load1(static_cast<const E*>(a.g[0]) + i) * S::load1(static_cast<const E*>(a.d[0]) + i);
#pragma unroll
            for (int k = 1; k < M; ++k)
                acc = fmaf(S::load1(static_cast<const E*>(a.g[k]) + i), S::load1(static_cast<const E*>(a.d[k]) + i), acc);
            S::store1(static_cast<E*>(a.gin) + i, acc);
        }
    }
}

// ---------------------------------------------------------------- one operator at a time
//
// The same primitives as separate kernels, the way a framework runs them when every operator
// is its own node (Section II-C approach 1): forward writes the operator's output tensor,
// backward applies the operator's own rule to the upstream gradient and whatever the rule
// needs (an operand or the output), which therefore has to be kept alive until then.
struct EwArgs {
    const void* in[3];
    void* out[2];
    int op;
    int backward;
    float c;
    size_t n;
    size_t head, packets;    // as in SeqBackwardArgs
};

template <class P>
__device__ __forceinline__ void ew_apply(int op, int backward, float c, float i0, float i1, float i2, float& o0, float& o1)
{
    using T = typename ScalarOf<P>::type;
    const Dual<P> a{T(i0), T(0)};
    o1 = 0.0f;
    if (!backward) {
        switch (op) {
        case kSeqAdd: o0 = i0 + i1; break;
        case kSeqMul: o0 = i0 * i1; break;
        case kSeqScale: o0 = c * i0; break;
        case kSeqAddConst: o0 = c + i0; break;
        case kSeqExp: o0 = dual_value(dual_exp(a)); break;
        case kSeqLog1p: o0 = dual_value(dual_log1p(a)); break;
        case kSeqTanh: o0 = dual_value(dual_tanh(a)); break;
        case kSeqErf: o0 = dual_value(dual_erf(a)); break;
        case kSeqSoftplus: o0 = dual_value(dual_softplus(a)); break;
        case kSeqSigmoid: o0 = dual_value(dual_sigmoid(a)); break;
        case kSeqHalfOnePlusTanh: o0 = dual_value(dual_half_one_plus_tanh(a)); break;
        case kSeqHalfOnePlusErf: o0 = dual_value(dual_half_one_plus_erf(a)); break;
        default: o0 = i0; break;
        }
    } else {
        // i0 = upstream gradient; i1, i2 = what the rule kept.  The rule's own factor is the tangent that the
        // primitive returns for a unit input tangent, wherever the rule keeps the operator's INPUT; where it keeps the
        // OUTPUT the factor is the usual closed form in that output.
        const float g = i0;
        const Dual<P> in{T(i1), T(1)};
        switch (op) {
        case kSeqMul: o0 = g * i2; o1 = g * i1; break;                        // kept: both operands
        case kSeqScale: o0 = c * g; break;
        case kSeqExp: o0 = g * i1; break;                                     // kept: the output
        case kSeqLog1p: o0 = g * dual_tangent(dual_log1p(in)); break;         // kept: the input
        case kSeqTanh: o0 = g * fmaf(-i1, i1, 1.0f); break;                   // kept: the output
        case kSeqErf: o0 = g * dual_tangent(dual_erf(in)); break;             // input
        case kSeqSoftplus: o0 = g * dual_tangent(dual_softplus(in)); break;   // input
        case kSeqSigmoid: o0 = g * (i1 * (1.0f - i1)); break;                 // kept: the output
        case kSeqHalfOnePlusTanh: o0 = g * ((i1 + i1) * (1.0f - i1)); break;  // kept: the output
        case kSeqHalfOnePlusErf: o0 = g * dual_tangent(dual_half_one_plus_erf(in)); break;   // input
        default: o0 = g; break;
        }
    }
}

// (Tiled like the other kernels -- two packets per thread, every load issued before the first use -- so that the
// operator-by-operator comparator runs each operator at the bandwidth a framework's own element-wise kernel reaches.)
constexpr int kEwUnroll = 2;

// OP and BWD are template parameters: each operator gets its own specialised kernel, as in a framework.
template <class S, int OP, bool BWD>
__global__ void __launch_bounds__(kBlock, 4) ew_kernel(const EwArgs a)
{
    using E = typename S::elem;
    constexpr int V = S::kVec;
    constexpr int U = kEwUnroll;
    const size_t byte_off = a.head * sizeof(E);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const size_t tile = size_t(kBlock) * U;
    for (size_t base = size_t(blockIdx.x) * tile + threadIdx.x; base < a.packets; base += size_t(gridDim.x) * tile) {
        uint4 r0[U], r1[U], r2[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t pk = base + size_t(u) * kBlock;
            if (pk < a.packets) {
                r0[u] = load_packet(reinterpret_cast<const uint4*>(static_cast<const char*>(a.in[0]) + byte_off) + pk);
                if (a.in[1]) r1[u] = load_packet(reinterpret_cast<const uint4*>(static_cast<const char*>(a.in[1]) + byte_off) + pk);
                if (a.in[2]) r2[u] = load_packet(reinterpret_cast<const uint4*>(static_cast<const char*>(a.in[2]) + byte_off) + pk);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t pk = base + size_t(u) * kBlock;
            if (pk >= a.packets) continue;
            float i0[V], i1[V], i2[V], o0[V], o1[V];
            S::unpack(r0[u], i0);
            if (a.in[1]) S::unpack(r1[u], i1);
            if (a.in[2]) S::unpack(r2[u], i2);
#pragma unroll
            for (int e = 0; e < V; ++e) ew_apply<typename SeqPolicy<S>::type>(OP, BWD, a.c, i0[e], a.in[1] ? i1[e] : 0.0f, a.in[2] ? i2[e] : 0.0f, o0[e], o1[e]);
            *(reinterpret_cast<uint4*>(static_cast<char*>(a.out[0]) + byte_off) + pk) = S::pack(o0);
            if (a.out[1]) *(reinterpret_cast<uint4*>(static_cast<char*>(a.out[1]) + byte_off) + pk) = S::pack(o1);
        }
    }
    {   // outside the packet grid: spread over the whole grid (see seq_forward_kernel)
        const size_t tail_begin = a.head + a.packets * V;
        const size_t n_edge = a.head + (a.n - tail_begin);
        for (size_t j = size_t(blockIdx.x) * kBlock + threadIdx.x; j < n_edge; j += size_t(gridDim.x) * kBlock) {
            const size_t i = j < a.head ? j : tail_begin + (j - a.head);
            float i0 = S::load1(static_cast<const E*>(a.in[0]) + i);
            float i1 = a.in[1] ? S::load1(static_cast<const E*>(a.in[1]) + i) : 0.0f;
            float i2 = a.in[2] ? S::load1(static_cast<const E*>(a.in[2]) + i) : 0.0f;
            float o0, o1;
            ew_apply<typename SeqPolicy<S>::type>(OP, BWD, a.c, i0, i1, i2, o0, o1);
            S::store1(static_cast<E*>(a.out[0]) + i, o0);
            if (a.out[1]) S::store1(static_cast<E*>(a.out[1]) + i, o1);
        }
    }
}

}  // namespace nfad
