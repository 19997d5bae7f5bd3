// nfad_jit_kernel.cuh -- the kernel skeleton around a FAD sequence that is compiled at run time.
//
// The host turns a sequence into straight-line device code over the dual primitives -- one line per
// instruction, registers as named values -- and compiles this header around it, so that the whole
// sequence is one kernel with every dual number in hardware registers (Section IV: one fused FAD
// sequence, no intermediate in memory), as the dedicated activation kernels are.  The generated part
// is the body of jit_element; everything else is fixed.
#pragma once

namespace nfad {

constexpr int kJitMaxOut = 4;
constexpr int kJitUnroll = 4;          // packets per thread and tile

// Identical on the host (which fills it) and in the generated kernel (which reads it).
struct JitArgs {
    const void* x;
    void* y[kJitMaxOut];
    void* d[kJitMaxOut];
    unsigned long long n, head, packets;
};

}  // namespace nfad

#ifdef __CUDACC_RTC__

#include "nfad_dual.cuh"
#include "nfad_storage.cuh"

namespace nfad {

// y_k and dy_k/dx of one element: defined by the generated code
template <int M> __device__ __forceinline__ void jit_element(float x, float (&yv)[M], float (&yt)[M]);

template <class S, int M> __device__ __forceinline__ void jit_forward(const JitArgs& a)
{
    typedef typename S::elem E;
    constexpr int V = S::kVec;
    const unsigned long long byte_off = a.head * sizeof(E);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // one tile of blockDim.x * kJitUnroll packets per CTA (the loop only matters beyond 2^31-1 tiles); a thread
    // issues all its loads before the first use
    const unsigned long long tile = (unsigned long long)blockDim.x * kJitUnroll;
    for (unsigned long long base = (unsigned long long)blockIdx.x * tile + threadIdx.x; base < a.packets;
         base += (unsigned long long)gridDim.x * tile) {
        uint4 raw[kJitUnroll];
#pragma unroll
        for (int u = 0; u < kJitUnroll; ++u) {
            const unsigned long long pk = base + (unsigned long long)u * blockDim.x;
            if (pk < a.packets) raw[u] = load_packet(reinterpret_cast<const uint4*>(static_cast<const char*>(a.x) + byte_off) + pk);
        }
#pragma unroll
        for (int u = 0; u < kJitUnroll; ++u) {
            const unsigned long long pk = base + (unsigned long long)u * blockDim.x;
            if (pk >= a.packets) continue;
            float xv[V], yv[M][V], yt[M][V];
            S::unpack(raw[u], xv);
#pragma unroll
            for (int e = 0; e < V; ++e) {
                float v[M], t[M];
                jit_element<M>(xv[e], v, t);
#pragma unroll
                for (int k = 0; k < M; ++k) { yv[k][e] = v[k]; yt[k][e] = t[k]; }
            }
#pragma unroll
            for (int k = 0; k < M; ++k) {
                store_packet<true>(reinterpret_cast<uint4*>(static_cast<char*>(a.y[k]) + byte_off) + pk, S::pack(yv[k]));
                store_packet<false>(reinterpret_cast<uint4*>(static_cast<char*>(a.d[k]) + byte_off) + pk, S::pack(yt[k]));
            }
        }
    }
    {   // outside the packet grid, one element at a time with the same code, spread over the whole grid: a few at the
        // ragged ends, or all n when the tensors share no offset modulo 16 bytes (head = n, packets = 0)
        const unsigned long long tail_begin = a.head + a.packets * V;
        const unsigned long long n_edge = a.head + (a.n - tail_begin);
        for (unsigned long long j = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; j < n_edge;
             j += (unsigned long long)gridDim.x * blockDim.x) {
            const unsigned long long i = j < a.head ? j : tail_begin + (j - a.head);
            float v[M], t[M];
            jit_element<M>(S::load1(static_cast<const E*>(a.x) + i), v, t);
#pragma unroll
            for (int k = 0; k < M; ++k) {
                S::store1(static_cast<E*>(a.y[k]) + i, v[k]);
                S::store1(static_cast<E*>(a.d[k]) + i, t[k]);
            }
        }
    }
}

}  // namespace nfad

#endif  // __CUDACC_RTC__
