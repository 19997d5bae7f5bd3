// nfad_stream.cuh -- the HBM-streaming engine shared by every kernel of the
// activation pass.  Each kernel is an element-wise map from NIN flat input
// tensors to NOUT flat output tensors of one storage type; nothing is reused, so
// the only jobs are (1) move 16-byte packets with fully coalesced accesses and
// enough of them in flight to cover HBM latency, and (2) spend as few issue
// slots per element as possible between the load and the store.
//
// Work decomposition: a tile is kBlock * U consecutive packets (U = 4, or the op's choice); thread t
// of a CTA owns packets t, t + kBlock, ... of the tile, so every warp-level
// access is one contiguous 512-byte run.  One CTA per tile; each thread issues
// all U * NIN loads of its tile before the first use.  Elements before the first and after the
// last whole packet (unaligned base, ragged tail) are handled one by one by the
// first warps of CTA 0 with the very same per-element code, so the vector and
// scalar paths agree bit for bit.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "nfad_storage.cuh"

namespace nfad {

constexpr int kBlock = 256;
constexpr int kDefaultUnroll = 4;          // packets per thread and tile unless the op states its own
// ---------------------------------------------------------------- kernel

template <int NIN, int NOUT> struct StreamArgs {
    const void* in[NIN];
    void* out[NOUT];
    size_t n;          // elements
    size_t head;       // elements before the first 16-byte boundary (same for every tensor)
    size_t packets;    // whole packets after the head
};

// Op: struct with
//   static constexpr int kIn, kOut;  static constexpr bool keep(int out_slot);
//   static __device__ void apply(const float (&in)[kIn], float (&out)[kOut]);
//   static constexpr int kMinBlocks: resident CTAs per SM to leave room for (0: the storage type's default);
//   static constexpr int kUnroll: packets per thread and tile (0: the default, 4);
//   static constexpr bool kPairs; if set, apply2(const float2 (&in)[kIn], float2 (&out)[kOut]) does two elements at once
//   with the same results as apply on each (packed fp32 arithmetic: half the issue slots for multiplies and adds).
template <class S, class Op>
__device__ __forceinline__ void scalar_element(const StreamArgs<Op::kIn, Op::kOut>& a, size_t i)
{
    using E = typename S::elem;
    float in[Op::kIn], out[Op::kOut];
#pragma unroll
    for (int k = 0; k < Op::kIn; ++k) in[k] = S::load1(static_cast<const E*>(a.in[k]) + i);
    Op::apply(in, out);
#pragma unroll
    for (int k = 0; k < Op::kOut; ++k) S::store1(static_cast<E*>(a.out[k]) + i, out[k]);
}

template <class S, class Op>
__device__ __forceinline__ void packet_compute_store(const StreamArgs<Op::kIn, Op::kOut>& a, size_t pk,
                                                     const uint4 (&raw)[Op::kIn])
{
    constexpr int V = S::kVec;
    float vin[Op::kIn][V];
    float vout[Op::kOut][V];
#pragma unroll
    for (int k = 0; k < Op::kIn; ++k) S::unpack(raw[k], vin[k]);
    if constexpr (Op::kPairs) {                 // two elements per call on packed fp32 arithmetic
#pragma unroll
        for (int e = 0; e < V; e += 2) {
            float2 in[Op::kIn], out[Op::kOut];
#pragma unroll
            for (int k = 0; k < Op::kIn; ++k) in[k] = make_float2(vin[k][e], vin[k][e + 1]);
            Op::apply2(in, out);
#pragma unroll
            for (int k = 0; k < Op::kOut; ++k) { vout[k][e] = out[k].x; vout[k][e + 1] = out[k].y; }
        }
    } else {
#pragma unroll
        for (int e = 0; e < V; ++e) {
            float in[Op::kIn], out[Op::kOut];
#pragma unroll
            for (int k = 0; k < Op::kIn; ++k) in[k] = vin[k][e];
            Op::apply(in, out);
#pragma unroll
            for (int k = 0; k < Op::kOut; ++k) vout[k][e] = out[k];
        }
    }
    const size_t byte_off = a.head * sizeof(typename S::elem);
#pragma unroll
    for (int k = 0; k < Op::kOut; ++k) {
        uint4* dst = reinterpret_cast<uint4*>(static_cast<char*>(a.out[k]) + byte_off) + pk;
        uint4 v = S::pack(vout[k]);
        if (Op::keep(k)) store_packet<true>(dst, v);
        else store_packet<false>(dst, v);
    }
}

// Packets per thread and tile: the op's own choice if it states one, else the default.
template <class Op> struct UnrollOf { static constexpr int value = Op::kUnroll ? Op::kUnroll : kDefaultUnroll; };

template <class S, class Op>
__global__ void __launch_bounds__(kBlock, (Op::kMinBlocks ? Op::kMinBlocks : S::kMinBlocks)) stream_kernel(const StreamArgs<Op::kIn, Op::kOut> a)
{
    constexpr int V = S::kVec;
    constexpr int kUnroll = UnrollOf<Op>::value;
    const size_t byte_off = a.head * sizeof(typename S::elem);
    const size_t tile_packets = size_t(kBlock) * kUnroll;
    const size_t n_tiles = (a.packets + tile_packets - 1) / tile_packets;

    // Programmatic dependent launch: let the next kernel of the stream be scheduled onto SMs
    // as this grid's last CTAs drain (it is only released once every CTA of this grid has
    // started), and do not touch memory before the previous kernel of the stream has
    // completed and its writes are visible.  Both are no-ops for a launch without the
    // programmatic-serialisation attribute.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    for (size_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const size_t base = tile * tile_packets + threadIdx.x;
        uint4 raw[kUnroll][Op::kIn];
        if (base + size_t(kUnroll - 1) * kBlock < a.packets) {          // whole tile: no predicates
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
#pragma unroll
                for (int k = 0; k < Op::kIn; ++k)
                    raw[u][k] = load_packet(reinterpret_cast<const uint4*>(static_cast<const char*>(a.in[k]) + byte_off) +
                                            base + size_t(u) * kBlock);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) packet_compute_store<S, Op>(a, base + size_t(u) * kBlock, raw[u]);
        } else {
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const size_t pk = base + size_t(u) * kBlock;
                if (pk < a.packets) {
#pragma unroll
                    for (int k = 0; k < Op::kIn; ++k)
                        raw[u][k] = load_packet(reinterpret_cast<const uint4*>(static_cast<const char*>(a.in[k]) + byte_off) + pk);
                }
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const size_t pk = base + size_t(u) * kBlock;
                if (pk < a.packets) packet_compute_store<S, Op>(a, pk, raw[u]);
            }
        }
    }

    // ragged ends: at most V-1 elements before the first packet and after the last
    if (blockIdx.x == 0) {
        const size_t tail_begin = a.head + a.packets * V;
        const size_t n_edge = a.head + (a.n - tail_begin);
        for (size_t j = threadIdx.x; j < n_edge; j += kBlock) {
            const size_t i = j < a.head ? j : tail_begin + (j - a.head);
            scalar_element<S, Op>(a, i);
        }
    }
}

// Every element one by one: taken when the tensors do not share one offset
// modulo 16 bytes, so that no common packet grid exists.
template <class S, class Op>
__global__ void __launch_bounds__(kBlock) scalar_kernel(const StreamArgs<Op::kIn, Op::kOut> a)
{
    const size_t stride = size_t(gridDim.x) * kBlock;
    for (size_t i = size_t(blockIdx.x) * kBlock + threadIdx.x; i < a.n; i += stride) scalar_element<S, Op>(a, i);
}

// ---------------------------------------------------------------- launch

struct DeviceInfo { int sm_count; };

inline cudaError_t device_info(DeviceInfo* out)
{
    static thread_local int cached_dev = -1;
    static thread_local DeviceInfo cached;
    int dev;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev != cached_dev) {
        e = cudaDeviceGetAttribute(&cached.sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        cached_dev = dev;
    }
    *out = cached;
    return cudaSuccess;
}

template <class S, class Op>
cudaError_t launch_stream(const void* const* in, void* const* out, size_t n, cudaStream_t st)
{
    if (n == 0) return cudaSuccess;
    StreamArgs<Op::kIn, Op::kOut> a;
    uintptr_t mis = 0;
    bool congruent = true;
    for (int k = 0; k < Op::kIn; ++k) {
        a.in[k] = in[k];
        uintptr_t m = reinterpret_cast<uintptr_t>(in[k]) & 15u;
        if (k == 0) mis = m;
        congruent = congruent && (m == mis);
    }
    for (int k = 0; k < Op::kOut; ++k) {
        a.out[k] = out[k];
        congruent = congruent && ((reinterpret_cast<uintptr_t>(out[k]) & 15u) == mis);
    }
    a.n = n;
    DeviceInfo di;
    cudaError_t e = device_info(&di);
    if (e != cudaSuccess) return e;

    static thread_local int occ_scalar = 0;   // per instantiation
    if (!congruent) {
        if (occ_scalar == 0) {
            e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_scalar, scalar_kernel<S, Op>, kBlock, 0);
            if (e != cudaSuccess) return e;
        }
        a.head = 0;
        a.packets = 0;
        size_t blocks = (n + kBlock - 1) / kBlock;
        size_t cap = size_t(di.sm_count) * occ_scalar;
        scalar_kernel<S, Op><<<(unsigned)(blocks < cap ? blocks : cap), kBlock, 0, st>>>(a);
        return cudaPeekAtLastError();
    }
    constexpr size_t esz = sizeof(typename S::elem);
    size_t head = ((16u - mis) & 15u) / esz;
    if (head > n) head = n;
    a.head = head;
    a.packets = (n - head) / S::kVec;
    // One tile per CTA, handed out in address order by the hardware as CTAs retire: measured
    // on B200 this moves a 1-read-2-write stream ~15 % faster than a resident grid striding over
    // the tiles (the window of addresses in flight stays compact), and it balances the SMs at
    // tile granularity.  (Shrinking the tile so that the tiles fill a whole number of waves of
    // resident CTAs -- 1446 tiles of 1088 packets instead of 1229 of 1280 for a 12.6M-element bf16
    // tensor on 740 slots -- was measured too: 3-6 % slower, the hardware's hand-out already evens
    // the waves out.)  The kernel's tile loop only matters beyond 2^31-1 tiles.
    const size_t tile_packets = size_t(kBlock) * UnrollOf<Op>::value;
    size_t tiles = (a.packets + tile_packets - 1) / tile_packets;
    if (tiles == 0) tiles = 1;                                  // edges only
    size_t grid = tiles < size_t(0x7fffffff) ? tiles : size_t(0x7fffffff);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kBlock);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, stream_kernel<S, Op>, a);
}

}  // namespace nfad
