// nfad_api.cu -- the extern "C" boundary: argument validation, aliasing rules,
// and dispatch to the per-storage-type launchers.  No arithmetic lives here.
#include <stdint.h>

#include <mutex>
#include <string>

#include "../../include/nfad.h"
#include "nfad_internal.h"

namespace {

thread_local int g_last_cuda_error = 0;

size_t elem_size(int dtype) { return dtype == NFAD_F32 ? 4 : 2; }

bool overlaps(const void* a, const void* b, size_t bytes_a, size_t bytes_b)
{
    uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + bytes_b && b0 < a0 + bytes_a;
}

// Validates the tensors of one launch.  Inputs may be exactly equal to outputs;
// any other overlap that involves an output is rejected.
int check(int kind, int dtype, const void* const* in, int nin, void* const* out, int nout, size_t n)
{
    if (kind < 0 || kind > 3) return NFAD_E_KIND;
    if (dtype < 0 || dtype > 2) return NFAD_E_DTYPE;
    if (n == 0) return NFAD_OK;
    const size_t es = elem_size(dtype), bytes = n * es;
    for (int i = 0; i < nin; ++i) {
        if (!in[i]) return NFAD_E_NULL;
        if (reinterpret_cast<uintptr_t>(in[i]) % es) return NFAD_E_ALIGN;
    }
    for (int i = 0; i < nout; ++i) {
        if (!out[i]) return NFAD_E_NULL;
        if (reinterpret_cast<uintptr_t>(out[i]) % es) return NFAD_E_ALIGN;
    }
    for (int i = 0; i < nout; ++i) {
        for (int j = i + 1; j < nout; ++j)
            if (overlaps(out[i], out[j], bytes, bytes)) return NFAD_E_OVERLAP;
        for (int j = 0; j < nin; ++j)
            if (in[j] != out[i] && overlaps(out[i], in[j], bytes, bytes)) return NFAD_E_OVERLAP;
    }
    return NFAD_OK;
}

int run(nfad::OpCode op, int kind, int dtype, const void* const* in, void* const* out, size_t n, nfad_stream_t stream)
{
    if (n == 0) return NFAD_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = dtype == NFAD_F32 ? nfad::launch_f32(op, kind, in, out, n, st)
                                      : nfad::launch_16(op, kind, dtype, in, out, n, st);
    if (e != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(e);
        return NFAD_E_CUDA;
    }
    return NFAD_OK;
}

// Tensors kept by operator-by-operator back-propagation under the usual rules
// (mul keeps both operands; tanh / sigmoid keep their output; erf / softplus
// keep their input; add and scale-by-constant keep nothing).
//   Swish     mul(x, sigmoid x)                      {x, sigmoid}           = 2  (the paper's v1, v2)
//   Mish      mul(x, tanh(softplus x))               {x, tanh}              = 2
//   GELU-tanh mul(0.5 x, 1 + tanh(c (x + a x^3)))    {x, 0.5x, tanh, 1+tanh} = 4
//   GELU-erf  mul(0.5 x, 1 + erf(x / sqrt2))         {x/sqrt2, 0.5x, 1+erf} = 3
int op_by_op_tensors(int kind)
{
    switch (kind) {
    case NFAD_SWISH: return 2;
    case NFAD_MISH: return 2;
    case NFAD_GELU_TANH: return 4;
    default: return 3;
    }
}

// ---- built-in scratch for nfad_cmp_recompute_backward_noalloc ----------------------------
//
// The array below lives in the library image: loading the library on a GPU reserves it
// there until the process exits.  In HOST code the name `g_noalloc_scratch` is only a
// handle for the runtime, not an address a kernel can use; the device address has to be
// asked for, once per device, with that device current.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NFAD_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
void* g_noalloc_ptr[kMaxDevices] = {};

// Device address of the built-in scratch on the current device; looked up on first use.
cudaError_t noalloc_scratch(void** out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_noalloc_ptr[dev] = p;
    }
    *out = g_noalloc_ptr[dev];
    return cudaSuccess;
}

// [rows, cols] of the bias-fused entry points: cols must fit 31 bits, the element count a size_t of bytes.
int check_shape(size_t rows, size_t cols, size_t* n)
{
    if (cols >= (size_t(1) << 31)) return NFAD_E_TOO_LARGE;
    if (rows && cols > (~size_t(0) / 8) / rows) return NFAD_E_TOO_LARGE;
    *n = rows * cols;
    return NFAD_OK;
}

}  // namespace

namespace nfad {
void note_cuda_error(cudaError_t e) { g_last_cuda_error = static_cast<int>(e); }

unsigned edge_grid_blocks(size_t n, unsigned block)
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 128;
    size_t need = (n + block - 1) / block;
    size_t cap = size_t(sms) * 32;
    if (need == 0) need = 1;
    return (unsigned)(need < cap ? need : cap);
}
}  // namespace nfad

extern "C" {

int nfad_act_forward(int kind, int dtype, const void* x, void* y, void* dfdx, size_t n, nfad_stream_t stream)
{
    const void* in[1] = {x};
    void* out[2] = {y, dfdx};
    int rc = check(kind, dtype, in, 1, out, 2, n);
    return rc ? rc : run(nfad::kOpForward, kind, dtype, in, out, n, stream);
}

int nfad_act_forward_strict(int kind, int dtype, const void* x, void* y, void* dfdx, size_t n, nfad_stream_t stream)
{
    if (dtype != NFAD_F32) return NFAD_E_DTYPE;
    const void* in[1] = {x};
    void* out[2] = {y, dfdx};
    int rc = check(kind, dtype, in, 1, out, 2, n);
    return rc ? rc : run(nfad::kOpForwardStrict, kind, dtype, in, out, n, stream);
}

int nfad_act_forward_infer(int kind, int dtype, const void* x, void* y, size_t n, nfad_stream_t stream)
{
    const void* in[1] = {x};
    void* out[1] = {y};
    int rc = check(kind, dtype, in, 1, out, 1, n);
    return rc ? rc : run(nfad::kOpForwardInfer, kind, dtype, in, out, n, stream);
}

int nfad_act_backward(int kind, int dtype, const void* grad_out, const void* dfdx, void* grad_in, size_t n,
                      nfad_stream_t stream)
{
    const void* in[2] = {grad_out, dfdx};
    void* out[1] = {grad_in};
    int rc = check(kind, dtype, in, 2, out, 1, n);
    return rc ? rc : run(nfad::kOpBackward, kind, dtype, in, out, n, stream);
}

int nfad_cmp_conv_backward(int kind, int dtype, const void* grad_out, const void* x, void* grad_in, size_t n,
                           nfad_stream_t stream)
{
    const void* in[2] = {grad_out, x};
    void* out[1] = {grad_in};
    int rc = check(kind, dtype, in, 2, out, 1, n);
    return rc ? rc : run(nfad::kOpConvBackward, kind, dtype, in, out, n, stream);
}

size_t nfad_cmp_recompute_scratch_bytes(int kind, int dtype, size_t n)
{
    if (kind < 0 || kind > 3 || dtype < 0 || dtype > 2) return 0;
    size_t b = n * elem_size(dtype);
    return (b + 15) & ~size_t(15);
}

int nfad_cmp_recompute_backward(int kind, int dtype, const void* grad_out, const void* x, void* scratch,
                                size_t scratch_bytes, void* grad_in, size_t n, nfad_stream_t stream)
{
    if (kind < 0 || kind > 3) return NFAD_E_KIND;
    if (dtype < 0 || dtype > 2) return NFAD_E_DTYPE;
    if (n == 0) return NFAD_OK;
    if (!scratch) return NFAD_E_NULL;
    if (scratch_bytes < nfad_cmp_recompute_scratch_bytes(kind, dtype, n)) return NFAD_E_SCRATCH;
    {
        const void* in[1] = {x};
        void* out[1] = {scratch};
        int rc = check(kind, dtype, in, 1, out, 1, n);
        if (rc) return rc;
        if (x == scratch) return NFAD_E_OVERLAP;
    }
    const void* in2[3] = {grad_out, x, scratch};
    void* out2[1] = {grad_in};
    int rc = check(kind, dtype, in2, 3, out2, 1, n);
    if (rc) return rc;
    if (grad_in == x || grad_in == scratch) return NFAD_E_OVERLAP;
    const void* in1[1] = {x};
    void* out1[1] = {scratch};
    rc = run(nfad::kOpRecompute1, kind, dtype, in1, out1, n, stream);
    if (rc) return rc;
    return run(nfad::kOpRecompute2, kind, dtype, in2, out2, n, stream);
}

int nfad_probe_stream(int reads, int writes, const void* a, const void* b, void* o0, void* o1, size_t n_words,
                      nfad_stream_t stream)
{
    nfad::OpCode op;
    if (reads == 1 && writes == 1) op = nfad::kOpProbe11;
    else if (reads == 1 && writes == 2) op = nfad::kOpProbe12;
    else if (reads == 2 && writes == 1) op = nfad::kOpProbe21;
    else if (reads == 1 && writes == 0) op = nfad::kOpProbe10;
    else if (reads == 0 && writes == 1) op = nfad::kOpProbe01;
    else return NFAD_E_LAYOUT;
    if (writes == 0 || reads == 0) {
        // one-sided probes: whole 16-byte packets only; o0 is a one-word sink for the read probe
        if (n_words == 0) return NFAD_OK;
        if (!o0 || (reads && !a)) return NFAD_E_NULL;
        const void* p = reads ? a : o0;
        if ((reinterpret_cast<uintptr_t>(p) & 15u) || (reinterpret_cast<uintptr_t>(o0) & 3u) || (n_words & 3u)) return NFAD_E_ALIGN;
        if (reads && overlaps(a, o0, n_words * 4, 4)) return NFAD_E_OVERLAP;
        const void* in1[1] = {a};
        void* out1[1] = {o0};
        return run(op, 0, NFAD_F32, in1, out1, n_words, stream);
    }
    const void* in[2] = {a, b};
    void* out[2] = {o0, o1};
    int rc = check(0, NFAD_F32, in, reads, out, writes, n_words);
    return rc ? rc : run(op, 0, NFAD_F32, in, out, n_words, stream);
}

// ---- the pass fused with its producer's bias ----------------------------------------------

// dfdx == nullptr selects the value-only pass
static int bias_forward_common(int kind, int dtype, const void* x, const void* bias, void* y, void* dfdx, bool train, size_t rows,
                               size_t cols, nfad_stream_t stream)
{
    if (kind < 0 || kind > 3) return NFAD_E_KIND;
    if (dtype < 0 || dtype > 2) return NFAD_E_DTYPE;
    size_t n = 0;
    int rc = check_shape(rows, cols, &n);
    if (rc) return rc;
    const void* in[1] = {x};
    void* out[2] = {y, dfdx};
    rc = check(kind, dtype, in, 1, out, train ? 2 : 1, n);
    if (rc || n == 0) return rc;
    const size_t es = elem_size(dtype);
    if (!bias) return NFAD_E_NULL;
    if (reinterpret_cast<uintptr_t>(bias) % es) return NFAD_E_ALIGN;
    if (overlaps(bias, y, cols * es, n * es) || (train && overlaps(bias, dfdx, cols * es, n * es))) return NFAD_E_OVERLAP;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    void* d = train ? dfdx : nullptr;
    cudaError_t e = dtype == NFAD_F32 ? nfad::launch_bias_forward_f32(kind, x, bias, y, d, rows, cols, st)
                                      : nfad::launch_bias_forward_16(kind, dtype, x, bias, y, d, rows, cols, st);
    if (e != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(e);
        return NFAD_E_CUDA;
    }
    return NFAD_OK;
}

int nfad_bias_act_forward(int kind, int dtype, const void* x, const void* bias, void* y, void* dfdx, size_t rows,
                          size_t cols, nfad_stream_t stream)
{
    return bias_forward_common(kind, dtype, x, bias, y, dfdx, true, rows, cols, stream);
}

int nfad_bias_act_forward_infer(int kind, int dtype, const void* x, const void* bias, void* y, size_t rows, size_t cols,
                                nfad_stream_t stream)
{
    return bias_forward_common(kind, dtype, x, bias, y, nullptr, false, rows, cols, stream);
}

size_t nfad_bias_act_backward_scratch_bytes(int dtype, size_t rows, size_t cols)
{
    if (dtype < 0 || dtype > 2) return 0;
    size_t n = 0, bytes = 0;
    if (check_shape(rows, cols, &n) != NFAD_OK || n == 0) return 0;
    cudaError_t e = nfad::bias_backward_scratch(dtype, rows, cols, &bytes);
    if (e != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(e);
        return 0;
    }
    return bytes;
}

int nfad_bias_act_backward(int kind, int dtype, const void* grad_out, const void* dfdx, void* grad_in, float* grad_bias,
                           void* scratch, size_t scratch_bytes, size_t rows, size_t cols, nfad_stream_t stream)
{
    if (kind < 0 || kind > 3) return NFAD_E_KIND;
    if (dtype < 0 || dtype > 2) return NFAD_E_DTYPE;
    size_t n = 0;
    int rc = check_shape(rows, cols, &n);
    if (rc) return rc;
    if (cols == 0) return NFAD_OK;
    const void* in[2] = {grad_out, dfdx};
    void* out[1] = {grad_in};
    rc = check(kind, dtype, in, 2, out, 1, n);
    if (rc) return rc;
    if (!grad_bias) return NFAD_E_NULL;
    if (reinterpret_cast<uintptr_t>(grad_bias) % sizeof(float)) return NFAD_E_ALIGN;
    const size_t es = elem_size(dtype), gb_bytes = cols * sizeof(float);
    size_t need = 0;
    cudaError_t e = cudaSuccess;
    if (n) {
        if (overlaps(grad_bias, grad_in, gb_bytes, n * es) || overlaps(grad_bias, grad_out, gb_bytes, n * es) ||
            overlaps(grad_bias, dfdx, gb_bytes, n * es))
            return NFAD_E_OVERLAP;
        e = nfad::bias_backward_scratch(dtype, rows, cols, &need);
        if (e == cudaSuccess && need) {
            if (!scratch) return NFAD_E_NULL;
            if (reinterpret_cast<uintptr_t>(scratch) % sizeof(float)) return NFAD_E_ALIGN;
            if (scratch_bytes < need) return NFAD_E_SCRATCH;
            if (overlaps(scratch, grad_in, need, n * es) || overlaps(scratch, grad_out, need, n * es) ||
                overlaps(scratch, dfdx, need, n * es) || overlaps(scratch, grad_bias, need, gb_bytes))
                return NFAD_E_OVERLAP;
        }
    }
    if (e == cudaSuccess)
        e = nfad::launch_bias_backward(dtype, grad_out, dfdx, grad_in, grad_bias, scratch, rows, cols,
                                       static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(e);
        return NFAD_E_CUDA;
    }
    return NFAD_OK;
}

int nfad_cmp_recompute_backward_noalloc(int kind, int dtype, const void* grad_out, const void* x, void* grad_in,
                                        size_t n, nfad_stream_t stream)
{
    if (kind < 0 || kind > 3) return NFAD_E_KIND;
    if (dtype < 0 || dtype > 2) return NFAD_E_DTYPE;
    if (n == 0) return NFAD_OK;
    if (n > NFAD_NOALLOC_SCRATCH_BYTES / elem_size(dtype)) return NFAD_E_TOO_LARGE;
    void* scratch = nullptr;
    cudaError_t e = noalloc_scratch(&scratch);
    if (e != cudaSuccess) {
        g_last_cuda_error = static_cast<int>(e);
        return NFAD_E_CUDA;
    }
    // from here on exactly the two launches of nfad_cmp_recompute_backward, on the built-in array
    return nfad_cmp_recompute_backward(kind, dtype, grad_out, x, scratch, NFAD_NOALLOC_SCRATCH_BYTES, grad_in, n, stream);
}

// Validates a sequence and copies it into the launcher's form.
static int parse_program(const nfad_seq_op* program, int n_ops, int m, nfad::SeqProgramHost* out)
{
    if (!program) return NFAD_E_NULL;
    if (n_ops < 1 || n_ops > nfad::kSeqMaxOpsHost || m < 1 || m > 4) return NFAD_E_PROGRAM;
    nfad::SeqProgramHost& p = *out;
    p = nfad::SeqProgramHost{};
    p.n_ops = n_ops;
    constexpr int kRegs = 12;
    bool written[kRegs] = {true};
    bool produced[4] = {false, false, false, false};
    for (int i = 0; i < n_ops; ++i) {
        const nfad_seq_op& o = program[i];
        if (o.op < 0 || o.op > NFAD_OP_OUT) return NFAD_E_PROGRAM;
        if (o.a < 0 || o.a >= kRegs || !written[o.a]) return NFAD_E_PROGRAM;
        const bool binary = o.op == NFAD_OP_ADD || o.op == NFAD_OP_MUL;
        if (binary && (o.b < 0 || o.b >= kRegs || !written[o.b])) return NFAD_E_PROGRAM;
        if (o.op == NFAD_OP_OUT) {
            if (o.dst < 0 || o.dst >= m) return NFAD_E_PROGRAM;
            produced[o.dst] = true;
        } else {
            if (o.dst < 1 || o.dst >= kRegs) return NFAD_E_PROGRAM;  // register 0 is the source and stays it
            written[o.dst] = true;
        }
        p.op[i] = o.op; p.a[i] = o.a; p.b[i] = binary ? o.b : o.a; p.dst[i] = o.dst; p.c[i] = o.c;
    }
    for (int k = 0; k < m; ++k) if (!produced[k]) return NFAD_E_PROGRAM;
    return NFAD_OK;
}

const char* nfad_seq_compiled_source(const nfad_seq_op* program, int n_ops, int dtype, int m)
{
    static thread_local std::string text;
    nfad::SeqProgramHost p;
    if (dtype < 0 || dtype > 2 || parse_program(program, n_ops, m, &p) != NFAD_OK) return nullptr;
    text = nfad::seq_generate_source(p, dtype, m);
    return text.c_str();
}

int nfad_seq_forward(const nfad_seq_op* program, int n_ops, int dtype, const void* x, void* const* y, void* const* dfdx,
                     int m, size_t n, nfad_stream_t stream)
{
    if (dtype < 0 || dtype > 2) return NFAD_E_DTYPE;
    if (!program || !y || !dfdx) return NFAD_E_NULL;
    nfad::SeqProgramHost p;
    {
        int prc = parse_program(program, n_ops, m, &p);
        if (prc) return prc;
    }
    const void* in[1] = {x};
    void* out[8];
    for (int k = 0; k < m; ++k) { out[k] = y[k]; out[m + k] = dfdx[k]; }
    int rc = check(0, dtype, in, 1, out, 2 * m, n);
    if (rc) return rc;
    if (n == 0) return NFAD_OK;
    for (int k = 0; k < 2 * m; ++k) if (out[k] == x) return NFAD_E_OVERLAP;
    cudaError_t e = nfad::launch_seq_forward(p, dtype, x, y, dfdx, m, n, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { g_last_cuda_error = static_cast<int>(e); return NFAD_E_CUDA; }
    return NFAD_OK;
}

int nfad_seq_set_executor(int mode)
{
    if (mode < 0 || mode > 2) return NFAD_E_LAYOUT;
    nfad::seq_set_executor_mode(mode);
    return NFAD_OK;
}

int nfad_seq_last_executor(void) { return nfad::seq_last_executor(); }

const char* nfad_seq_compile_log(void) { return nfad::seq_jit_log(); }

int nfad_seq_backward(int dtype, const void* const* grad_out, const void* const* dfdx, int m, void* grad_in, size_t n,
                      nfad_stream_t stream)
{
    if (dtype < 0 || dtype > 2) return NFAD_E_DTYPE;
    if (!grad_out || !dfdx) return NFAD_E_NULL;
    if (m < 1 || m > 4) return NFAD_E_PROGRAM;
    const void* in[8];
    for (int k = 0; k < m; ++k) { in[k] = grad_out[k]; in[m + k] = dfdx[k]; }
    void* out[1] = {grad_in};
    int rc = check(0, dtype, in, 2 * m, out, 1, n);
    if (rc) return rc;
    if (n == 0) return NFAD_OK;
    if (m == 1) {                                   // one result: exactly the multiplication of nfad_act_backward
        const void* in1[2] = {grad_out[0], dfdx[0]};
        return run(nfad::kOpBackward, 0, dtype, in1, out, n, stream);
    }
    cudaError_t e = nfad::launch_seq_backward(dtype, grad_out, dfdx, m, grad_in, n, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { g_last_cuda_error = static_cast<int>(e); return NFAD_E_CUDA; }
    return NFAD_OK;
}

int nfad_ew_op(int op, int backward, float c, int dtype, const void* in0, const void* in1, const void* in2, void* out0,
               void* out1, size_t n, nfad_stream_t stream)
{
    if (dtype < 0 || dtype > 2) return NFAD_E_DTYPE;
    if (op < 0 || op >= NFAD_OP_OUT) return NFAD_E_PROGRAM;
    const void* in[3];
    int nin = 0;
    in[nin++] = in0;
    if (in1) in[nin++] = in1;
    if (in2) in[nin++] = in2;
    void* out[2];
    int nout = 0;
    out[nout++] = out0;
    if (out1) out[nout++] = out1;
    int rc = check(0, dtype, in, nin, out, nout, n);
    if (rc) return rc;
    if (n == 0) return NFAD_OK;
    const void* in3[3] = {in0, in1, in2};
    void* out2[2] = {out0, out1};
    cudaError_t e = nfad::launch_ew(op, backward ? 1 : 0, c, dtype, in3, out2, n, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { g_last_cuda_error = static_cast<int>(e); return NFAD_E_CUDA; }
    return NFAD_OK;
}

int nfad_saved_bytes_per_element(int kind, int dtype, int layout)
{
    if (kind < 0 || kind > 3) return -NFAD_E_KIND;
    if (dtype < 0 || dtype > 2) return -NFAD_E_DTYPE;
    int s = static_cast<int>(elem_size(dtype));
    switch (layout) {
    case NFAD_LAYOUT_NESTED: return s;         // f'(x)
    case NFAD_LAYOUT_CONVENTIONAL: return s;   // x
    case NFAD_LAYOUT_RECOMPUTE: return s;      // x
    case NFAD_LAYOUT_OP_BY_OP: return s * op_by_op_tensors(kind);
    default: return -NFAD_E_LAYOUT;
    }
}

int nfad_last_cuda_error(void) { return g_last_cuda_error; }

const char* nfad_status_string(int status)
{
    switch (status) {
    case NFAD_OK: return "ok";
    case NFAD_E_KIND: return "unknown activation kind";
    case NFAD_E_DTYPE: return "unknown storage dtype";
    case NFAD_E_NULL: return "null tensor pointer";
    case NFAD_E_OVERLAP: return "tensors overlap in a way that is not exact in-place use";
    case NFAD_E_CUDA: return "CUDA error (see nfad_last_cuda_error)";
    case NFAD_E_ALIGN: return "pointer not aligned to the element size";
    case NFAD_E_SCRATCH: return "scratch buffer too small";
    case NFAD_E_LAYOUT: return "unknown layout";
    case NFAD_E_TOO_LARGE: return "tensors larger than the library's built-in scratch";
    case NFAD_E_PROGRAM: return "malformed FAD sequence";
    default: return "unknown status";
    }
}

const char* nfad_version(void) { return "0.1.0"; }

}  // extern "C"
