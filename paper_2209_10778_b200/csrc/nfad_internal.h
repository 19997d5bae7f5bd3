// nfad_internal.h -- launchers behind the C-ABI, one set per translation unit:
// the fp32-storage kernels are built with floating-point contraction off (their
// compensated arithmetic depends on it), the 16-bit-storage kernels with it on.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>

#include <string>

namespace nfad {

enum Kind { kGeluErf = 0, kGeluTanh = 1, kSwish = 2, kMish = 3 };
enum DType { kF32 = 0, kBF16 = 1, kF16 = 2 };

// Which map to run.  Tensor order in `in` / `out` is fixed per op:
//   kOpForward        in {x}            out {y, dfdx}
//   kOpForwardInfer   in {x}            out {y}
//   kOpBackward       in {g, dfdx}      out {gin}
//   kOpConvBackward   in {g, x}         out {gin}
//   kOpRecompute1     in {x}            out {h}
//   kOpRecompute2     in {g, x, h}      out {gin}
//   kOpProbe11/12/21  in {a[, b]}       out {o0[, o1]}   (traffic probes: fp32 storage only)
//   kOpForwardStrict  in {x}            out {y, dfdx}    (fp32 storage only)
//   kOpProbe10        in {a}            out {sink}       (read-only probe; sink: one word, written only on a checksum match)
//   kOpProbe01        in {}             out {o0}         (write-only probe)
enum OpCode { kOpForward, kOpForwardInfer, kOpBackward, kOpConvBackward, kOpRecompute1, kOpRecompute2,
              kOpProbe11, kOpProbe12, kOpProbe21, kOpForwardStrict, kOpProbe10, kOpProbe01 };

cudaError_t launch_f32(OpCode op, int kind, const void* const* in, void* const* out, size_t n, cudaStream_t st);
cudaError_t launch_16(OpCode op, int kind, int dtype, const void* const* in, void* const* out, size_t n, cudaStream_t st);

// Run-time FAD sequences (nfad_seq.cuh): the program as plain arrays, so that this header
// stays free of device code.
constexpr int kSeqMaxOpsHost = 32;
struct SeqProgramHost { int n_ops; int op[kSeqMaxOpsHost], a[kSeqMaxOpsHost], b[kSeqMaxOpsHost], dst[kSeqMaxOpsHost]; float c[kSeqMaxOpsHost]; };

cudaError_t launch_seq_forward(const SeqProgramHost& p, int dtype, const void* x, void* const* y, void* const* d, int m, size_t n,
                               cudaStream_t st);
// The same sequence compiled at run time into one kernel (nfad_jit.cu).  cudaErrorNotSupported: not available here.
cudaError_t launch_seq_forward_compiled(const SeqProgramHost& p, int dtype, const void* x, void* const* y, void* const* d, int m,
                                        size_t n, cudaStream_t st);
int seq_executor_mode();                 // 0 automatic, 1 interpreter only, 2 compiled only
void seq_set_executor_mode(int mode);
int seq_last_executor();                 // of the calling thread: 0 none yet, 1 interpreter, 2 compiled
void seq_note_executor(int which);
const char* seq_jit_log();
std::string seq_generate_source(const SeqProgramHost& p, int dtype, int m);   // what the compiled executor would compile
cudaError_t launch_seq_backward(int dtype, const void* const* g, const void* const* d, int m, void* gin, size_t n, cudaStream_t st);
cudaError_t launch_ew(int op, int backward, float c, int dtype, const void* const* in, void* const* out, size_t n, cudaStream_t st);

// CTAs for a launch that takes n elements one by one with a grid-stride loop: enough to fill the current device
// (32 CTAs of `block` threads per SM at most), never more than the elements need.
unsigned edge_grid_blocks(size_t n, unsigned block);

// Records the cudaError_t behind an NFAD_E_CUDA of the calling thread (what nfad_last_cuda_error() returns).
void note_cuda_error(cudaError_t e);

// The pass fused with its producer's bias (nfad_bias.cuh).  x, y, d, g, gin: [rows, cols] row-major; bias: [cols].
cudaError_t launch_bias_forward_f32(int kind, const void* x, const void* bias, void* y, void* d, size_t rows, size_t cols,
                                    cudaStream_t st);
cudaError_t launch_bias_forward_16(int kind, int dtype, const void* x, const void* bias, void* y, void* d, size_t rows,
                                   size_t cols, cudaStream_t st);
cudaError_t launch_bias_backward(int dtype, const void* g, const void* d, void* gin, float* grad_bias, void* scratch,
                                 size_t rows, size_t cols, cudaStream_t st);
cudaError_t bias_backward_scratch(int dtype, size_t rows, size_t cols, size_t* bytes);   // on the current device

}  // namespace nfad
