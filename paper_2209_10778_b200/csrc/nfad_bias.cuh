// nfad_bias.cuh -- the activation pass fused with its producer's bias.
//
// A linear layer hands over x[rows, cols] (row-major) and a bias b[cols]; the
// activation sees z = x + b.  Seen from x the addition is a binary operation
// with one constant input, i.e. unary (Section III-A), with dz/dx = 1: the saved
// tensor is still f'(z) and back-propagation still the one multiplication of
// Eq. 4.  Seen from b, dz/db = 1 on every row, so grad_b[c] is the column sum
// of that same product.  Fusing both here removes one write and one read of the
// pre-activation tensor in the forward pass and one read of grad_in in the
// backward pass.
//
// Work decomposition (both directions): a thread owns ONE 16-byte column packet
// and walks down the rows, so the bias packet is loaded and widened once per
// thread and the bias gradient accumulates in registers with no exchange between
// threads.  A CTA is a strip of B adjacent column packets (B a multiple of 32
// chosen per call so that strips tile the row with the fewest idle lanes: every
// warp access is a contiguous 512-byte run, a CTA's accesses a contiguous run of
// B * 16 bytes per row) times a chunk of consecutive rows; CTA ids run along the
// row first, so neighbouring CTAs touch neighbouring memory.
//   forward:  chunks of kBiasRows rows (one "tile" per CTA, as in the plain pass);
//   backward: chunks sized so that the device is filled a few times over; each CTA
//             writes its column sums to partial[chunk][col] and a second, tiny
//             kernel adds the chunks in order: the result does not depend on
//             scheduling, and the element-wise fallback kernels add in the same order.
#pragma once

#include "nfad_ops.cuh"
#include "nfad_stream.cuh"

namespace nfad {

constexpr int kBiasRows = 4;               // rows a thread loads before it uses the first
constexpr int kBiasMaxBlock = 256;

// Threads per CTA: the multiple of 32 in [64, 256] that leaves the fewest idle lanes in the last strip
// of a row (the largest such on a tie).
inline unsigned bias_block(size_t row_packets)
{
    unsigned best = kBiasMaxBlock;
    size_t best_waste = ~size_t(0);
    for (unsigned b = kBiasMaxBlock; b >= 64; b -= 32) {
        size_t waste = (row_packets + b - 1) / b * b - row_packets;
        if (waste < best_waste) { best_waste = waste; best = b; }
    }
    return best;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline void bias_launch_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, size_t grid, unsigned block, cudaStream_t st,
                               bool pdl)
{
    *cfg = cudaLaunchConfig_t{};
    cfg->gridDim = dim3((unsigned)grid);
    cfg->blockDim = dim3(block);
    cfg->stream = st;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg->attrs = attr;
    cfg->numAttrs = pdl ? 1 : 0;
}

// ---------------------------------------------------------------- forward

struct BiasForwardArgs {
    const void* x;
    const void* bias;
    void* y;
    void* d;
    size_t rows;
    size_t n;              // rows * cols
    size_t work;           // row chunks (vector path)
    uint32_t cols;
    uint32_t row_packets;  // cols / V
    uint32_t strips;       // CTAs along a row
};

// z = x + b, one fp32 addition that the compiler may not merge into anything
__device__ __forceinline__ float bias_sum(float x, float b) { return __fadd_rn(x, b); }

// kTrain: y and f'; otherwise y alone (d is not touched)
template <class S, class K, class P, bool kTrain>
__device__ __forceinline__ void bias_forward_packet(const uint4& rx, const float (&vb)[S::kVec], uint4* y, uint4* d)
{
    constexpr int V = S::kVec;
    float vx[V], vy[V], vd[V];
    S::unpack(rx, vx);
    // the same width per call as the plain pass uses for this kind (two elements on packed fp32 arithmetic for the
    // GELU-erf training forward and the value-only GELU forwards of 16-bit storage; the same bits either way)
    constexpr bool kPairs = kTrain ? ForwardTrainOp<K, P>::kPairs : ForwardInferOp<K, P>::kPairs;
    if constexpr (kPairs) {
#pragma unroll
        for (int e = 0; e < V; e += 2) {
            const float2 z = make_float2(bias_sum(vx[e], vb[e]), bias_sum(vx[e + 1], vb[e + 1]));
            if (kTrain) {
                ActOut2 o = evaluate(K{}, Fast2{}, z);
                vy[e] = o.y.x; vy[e + 1] = o.y.y;
                vd[e] = o.dydx.x; vd[e + 1] = o.dydx.y;
            } else {
                float2 y2 = evaluate_value(K{}, Fast2{}, z);
                vy[e] = y2.x; vy[e + 1] = y2.y;
            }
        }
    } else {
#pragma unroll
        for (int e = 0; e < V; ++e) {
            if (kTrain) {
                ActOut o = evaluate<K, P>(bias_sum(vx[e], vb[e]));
                vy[e] = o.y;
                vd[e] = o.dydx;
            } else {
                vy[e] = evaluate_value(K{}, P{}, bias_sum(vx[e], vb[e]));
            }
        }
    }
    store_packet<true>(y, S::pack(vy));
    if (kTrain) store_packet<false>(d, S::pack(vd));
}

// Vector path: cols a multiple of the packet size and every pointer 16-byte aligned.
template <class S, class K, class P, bool kTrain>
__global__ void __launch_bounds__(kBiasMaxBlock, S::kMinBlocks) bias_forward_kernel(const BiasForwardArgs a)
{
    constexpr int V = S::kVec;
    constexpr int U = kBiasRows;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint4* x4 = static_cast<const uint4*>(a.x);
    uint4* y4 = static_cast<uint4*>(a.y);
    uint4* d4 = static_cast<uint4*>(a.d);
    // grid: x = strip along the row (fastest, so neighbouring CTAs touch neighbouring memory), y = row chunk
    const uint32_t cp = blockIdx.x * blockDim.x + threadIdx.x;
    if (cp >= a.row_packets) return;
    for (size_t chunk = blockIdx.y; chunk < a.work; chunk += gridDim.y) {
        const size_t r0 = chunk * U;
        float vb[V];
        S::unpack(__ldg(static_cast<const uint4*>(a.bias) + cp), vb);
        const size_t pk0 = r0 * a.row_packets + cp;
        const uint32_t rp = a.row_packets;
        uint4 rx[U];
        if (r0 + U <= a.rows) {                                        // whole tile: no predicates
#pragma unroll
            for (int u = 0; u < U; ++u) rx[u] = load_packet(x4 + pk0 + size_t(u) * rp);
#pragma unroll
            for (int u = 0; u < U; ++u) bias_forward_packet<S, K, P, kTrain>(rx[u], vb, y4 + pk0 + size_t(u) * rp, d4 + pk0 + size_t(u) * rp);
        } else {
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (r0 + u < a.rows) rx[u] = load_packet(x4 + pk0 + size_t(u) * rp);
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (r0 + u < a.rows) bias_forward_packet<S, K, P, kTrain>(rx[u], vb, y4 + pk0 + size_t(u) * rp, d4 + pk0 + size_t(u) * rp);
        }
    }
}

// Any cols, any (element-aligned) pointers: one element at a time, the same per-element code.
template <class S, class K, class P, bool kTrain>
__global__ void __launch_bounds__(kBlock) bias_forward_scalar_kernel(const BiasForwardArgs a)
{
    using E = typename S::elem;
    const size_t stride = size_t(gridDim.x) * kBlock;
    for (size_t i = size_t(blockIdx.x) * kBlock + threadIdx.x; i < a.n; i += stride) {
        const uint32_t c = uint32_t(i % a.cols);
        const float z = bias_sum(S::load1(static_cast<const E*>(a.x) + i), S::load1(static_cast<const E*>(a.bias) + c));
        if (kTrain) {
            ActOut o = evaluate<K, P>(z);
            S::store1(static_cast<E*>(a.y) + i, o.y);
            S::store1(static_cast<E*>(a.d) + i, o.dydx);
        } else {
            S::store1(static_cast<E*>(a.y) + i, evaluate_value(K{}, P{}, z));
        }
    }
}

// d == nullptr: the value-only pass
template <class S, class K, class P>
cudaError_t launch_bias_forward(const void* x, const void* bias, void* y, void* d, size_t rows, size_t cols, cudaStream_t st)
{
    const bool train = d != nullptr;
    constexpr int V = S::kVec;
    BiasForwardArgs a;
    a.x = x; a.bias = bias; a.y = y; a.d = d;
    a.rows = rows;
    a.n = rows * cols;
    a.cols = uint32_t(cols);
    if (a.n == 0) return cudaSuccess;
    DeviceInfo di;
    cudaError_t e = device_info(&di);
    if (e != cudaSuccess) return e;
    const bool vec = cols % V == 0 && aligned16(x) && aligned16(bias) && aligned16(y) && (!train || aligned16(d));
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    if (!vec) {
        a.work = 0; a.row_packets = 0; a.strips = 0;
        size_t blocks = (a.n + kBlock - 1) / kBlock;
        size_t cap = size_t(di.sm_count) * 8;
        bias_launch_config(&cfg, attr, blocks < cap ? blocks : cap, kBlock, st, false);
        return train ? cudaLaunchKernelEx(&cfg, bias_forward_scalar_kernel<S, K, P, true>, a)
                     : cudaLaunchKernelEx(&cfg, bias_forward_scalar_kernel<S, K, P, false>, a);
    }
    a.row_packets = uint32_t(cols / V);
    const unsigned block = bias_block(a.row_packets);
    a.strips = (a.row_packets + block - 1) / block;
    a.work = (rows + kBiasRows - 1) / kBiasRows;
    bias_launch_config(&cfg, attr, a.strips, block, st, true);
    cfg.gridDim.y = (unsigned)(a.work < 65535 ? a.work : 65535);
    return train ? cudaLaunchKernelEx(&cfg, bias_forward_kernel<S, K, P, true>, a)
                 : cudaLaunchKernelEx(&cfg, bias_forward_kernel<S, K, P, false>, a);
}

// ---------------------------------------------------------------- backward with the bias gradient

struct BiasBackwardArgs {
    const void* g;
    const void* d;
    void* gin;
    float* partial;          // [chunks][cols] sums, or grad_bias itself when chunks == 1
    size_t rows;
    uint32_t cols;
    uint32_t row_packets;    // cols / V (vector path)
    uint32_t strips;
    uint32_t chunk_rows;     // rows per chunk
};

// How the rows are cut into chunks: enough CTAs to fill the device kBiasWaves times over,
// never fewer than kBiasRows rows per chunk, at most kBiasMaxChunks chunks.  The plan depends on
// the shape, the storage type and the device only -- not on pointer alignment -- so that the
// vector and the element-wise kernels add the same numbers in the same order.
constexpr int kBiasMaxChunks = 256;
constexpr int kBiasWaves = 2;

struct BiasPlan { unsigned block; uint32_t strips, chunks, chunk_rows; };

template <int V>
inline BiasPlan bias_plan(size_t rows, size_t cols, int sm_count)
{
    BiasPlan p;
    const size_t row_packets = (cols + V - 1) / V;
    p.block = bias_block(row_packets);
    p.strips = uint32_t((row_packets + p.block - 1) / p.block);
    if (p.strips == 0) p.strips = 1;
    const size_t target = size_t(sm_count) * (1024 / p.block) * kBiasWaves;
    size_t chunks = (target + p.strips - 1) / p.strips;
    const size_t max_by_rows = (rows + kBiasRows - 1) / kBiasRows;
    if (chunks > max_by_rows) chunks = max_by_rows;
    if (chunks > size_t(kBiasMaxChunks)) chunks = kBiasMaxChunks;
    if (chunks < 1) chunks = 1;
    size_t cr = (rows + chunks - 1) / chunks;
    cr = (cr + kBiasRows - 1) / kBiasRows * kBiasRows;
    if (cr == 0) cr = kBiasRows;
    p.chunk_rows = uint32_t(cr);
    p.chunks = uint32_t((rows + cr - 1) / cr);
    if (p.chunks == 0) p.chunks = 1;
    return p;
}

template <class S>
__global__ void __launch_bounds__(kBiasMaxBlock, 4) bias_backward_kernel(const BiasBackwardArgs a)
{
    constexpr int V = S::kVec;
    constexpr int U = kBiasRows;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint4* g4 = static_cast<const uint4*>(a.g);
    const uint4* d4 = static_cast<const uint4*>(a.d);
    uint4* o4 = static_cast<uint4*>(a.gin);
    const uint32_t cp = blockIdx.x * blockDim.x + threadIdx.x;     // grid: x = strip along the row, y = chunk of rows
    if (cp >= a.row_packets) return;
    {
        const size_t chunk = blockIdx.y;
        const size_t r0 = chunk * a.chunk_rows;
        const size_t r1 = r0 + a.chunk_rows < a.rows ? r0 + a.chunk_rows : a.rows;
        float acc[V];
#pragma unroll
        for (int e = 0; e < V; ++e) acc[e] = 0.0f;
        for (size_t r = r0; r < r1; r += U) {
            uint4 rg[U], rd[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (r + u < r1) {
                    rg[u] = load_packet(g4 + (r + u) * a.row_packets + cp);
                    rd[u] = load_packet(d4 + (r + u) * a.row_packets + cp);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (r + u < r1) {
                    float vin[2][V], vout[1][V];
                    S::unpack(rg[u], vin[0]);
                    S::unpack(rd[u], vin[1]);
#pragma unroll
                    for (int e = 0; e < V; ++e) vout[0][e] = __fmul_rn(vin[0][e], vin[1][e]);
                    const uint4 packed = S::pack(vout[0]);
                    o4[(r + u) * a.row_packets + cp] = packed;
                    // the STORED values, widened again: what a reduction over the stored tensor would read
                    float stored[V];
                    S::unpack(packed, stored);
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[e] = __fadd_rn(acc[e], stored[e]);
                }
            }
        }
        float* dst = a.partial + chunk * a.cols + size_t(cp) * V;
#pragma unroll
        for (int e = 0; e < V; ++e) dst[e] = acc[e];
    }
}

// Any cols / alignment: a thread per column, the same chunks, rows added in the same order.
template <class S>
__global__ void __launch_bounds__(kBlock) bias_backward_scalar_kernel(const BiasBackwardArgs a)
{
    using E = typename S::elem;
    const size_t col = size_t(blockIdx.x) * kBlock + threadIdx.x;
    if (col >= a.cols) return;
    const size_t r0 = size_t(blockIdx.y) * a.chunk_rows;
    const size_t r1 = r0 + a.chunk_rows < a.rows ? r0 + a.chunk_rows : a.rows;
    float acc = 0.0f;
    for (size_t r = r0; r < r1; ++r) {
        const size_t i = r * a.cols + col;
        float in[2] = {S::load1(static_cast<const E*>(a.g) + i), S::load1(static_cast<const E*>(a.d) + i)};
        float out[1];
        BackwardOp::apply(in, out);
        S::store1(static_cast<E*>(a.gin) + i, out[0]);
        acc = __fadd_rn(acc, S::load1(static_cast<const E*>(a.gin) + i));
    }
    a.partial[size_t(blockIdx.y) * a.cols + col] = acc;
}

// grad_bias[c] from partial[k][c], k < chunks, in a fixed order: the chunks are cut into kBiasGroups runs of
// consecutive chunks, each run is summed in chunk order by one thread, and the runs' sums are added in run order.
// A CTA takes 32 columns (one 128-byte line of every partial row) times the kBiasGroups runs; a thread's loads
// are issued eight at a time before the first is used.
constexpr int kBiasGroups = 32;
static __global__ void __launch_bounds__(32 * kBiasGroups) bias_reduce_chunks_kernel(const float* partial, float* grad_bias,
                                                                                     uint32_t chunks, uint32_t cols)
{
    __shared__ float smem[kBiasGroups][32];
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int lane = threadIdx.x & 31, group = threadIdx.x >> 5;
    const size_t col = size_t(blockIdx.x) * 32 + lane;
    const uint32_t per = (chunks + kBiasGroups - 1) / kBiasGroups;
    const uint32_t k0 = group * per;
    const uint32_t k1 = k0 + per < chunks ? k0 + per : chunks;
    float s = 0.0f;
    if (col < cols) {
        for (uint32_t k = k0; k < k1; k += 8) {
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = k + j < k1 ? partial[size_t(k + j) * cols + col] : 0.0f;
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (k + j < k1) s = __fadd_rn(s, v[j]);
        }
    }
    smem[group][lane] = s;
    __syncthreads();
    if (group == 0 && col < cols) {
        float t = smem[0][lane];
#pragma unroll
        for (int j = 1; j < kBiasGroups; ++j) t = __fadd_rn(t, smem[j][lane]);
        grad_bias[col] = t;
    }
}

template <int V>
inline size_t bias_backward_scratch_bytes(size_t rows, size_t cols, int sm_count)
{
    BiasPlan p = bias_plan<V>(rows, cols, sm_count);
    return p.chunks > 1 ? size_t(p.chunks) * cols * sizeof(float) : 0;
}

template <class S>
cudaError_t launch_bias_backward(const void* g, const void* d, void* gin, float* grad_bias, void* scratch, size_t rows,
                                 size_t cols, cudaStream_t st)
{
    constexpr int V = S::kVec;
    DeviceInfo di;
    cudaError_t e = device_info(&di);
    if (e != cudaSuccess) return e;
    if (cols == 0) return cudaSuccess;
    if (rows == 0) return cudaMemsetAsync(grad_bias, 0, cols * sizeof(float), st);
    const BiasPlan p = bias_plan<V>(rows, cols, di.sm_count);
    BiasBackwardArgs a;
    a.g = g; a.d = d; a.gin = gin;
    a.partial = p.chunks > 1 ? static_cast<float*>(scratch) : grad_bias;
    a.rows = rows;
    a.cols = uint32_t(cols);
    a.row_packets = uint32_t(cols / V);
    a.strips = p.strips;
    a.chunk_rows = p.chunk_rows;
    const bool vec = cols % V == 0 && aligned16(g) && aligned16(d) && aligned16(gin);
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    if (vec) {
        bias_launch_config(&cfg, attr, p.strips, p.block, st, true);
        cfg.gridDim.y = p.chunks;
        e = cudaLaunchKernelEx(&cfg, bias_backward_kernel<S>, a);
    } else {
        bias_launch_config(&cfg, attr, (cols + kBlock - 1) / kBlock, kBlock, st, false);
        cfg.gridDim.y = p.chunks;
        e = cudaLaunchKernelEx(&cfg, bias_backward_scalar_kernel<S>, a);
    }
    if (e != cudaSuccess || p.chunks == 1) return e;
    bias_launch_config(&cfg, attr, (cols + 31) / 32, 32 * kBiasGroups, st, true);
    return cudaLaunchKernelEx(&cfg, bias_reduce_chunks_kernel, static_cast<const float*>(a.partial), grad_bias, p.chunks,
                              uint32_t(cols));
}

}  // namespace nfad
