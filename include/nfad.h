/*
 * nfad.h -- C interface of the nested Forward-AD activation library (CUDA, sm_100a).
 *
 * The method (Section II-C approach 3, Section II-E): an element-wise activation
 * f is evaluated once, in the forward pass, on dual numbers (value, tangent)
 * seeded with tangent 1 (Section II-D), so that the forward pass emits y = f(x)
 * and f'(x) together; f'(x) is the ONLY tensor kept for back-propagation, and
 * the backward pass is the single multiplication grad_in = grad_out * f'(x)
 * (Eq. 4; "replaces the BFN with a direct Multiplication", Section IV).
 *
 * Conventions common to every entry point
 *   - Every tensor argument is a DEVICE pointer to a flat, contiguous array of n
 *     elements of `dtype` (NFAD_F32: float; NFAD_BF16: bfloat16; NFAD_F16: IEEE
 *     half).  Tensor shape is irrelevant to an element-wise pass.  The caller
 *     owns all memory; the library allocates none and keeps no state between
 *     calls.  Arithmetic is fp32 for the 16-bit storage types and fp64 for fp32
 *     storage (a few fp32 ulp of the exact result cannot be held by fp32
 *     arithmetic itself); results are rounded to nearest-even once, at the store.
 *     Subnormals are kept (no flush to zero).
 *   - Pointers need only the natural alignment of `dtype`.  When all tensors of
 *     a call share one offset modulo 16 bytes the 128-bit path is used (elements
 *     before the first and after the last whole 16-byte packet are handled one
 *     by one); otherwise every element is handled one by one.  Results do not
 *     depend on the path.
 *   - Exact in-place use (an output pointer equal to an input pointer) is
 *     allowed.  Two outputs that overlap, or an output that overlaps an input
 *     without being equal to it, give NFAD_E_OVERLAP.
 *   - Work is enqueued on `stream` (a cudaStream_t; 0 is the legacy default
 *     stream) of the current device and the call returns at once.  The return
 *     value covers argument validation and the launch, not completion.
 *   - The entry points that take device pointers only enqueue kernels (no allocation, no
 *     synchronisation, no host-side wait) and can be captured into a CUDA graph; the exceptions
 *     (nfad_host_step; the first call of a new run-time sequence when it is compiled) say so
 *     where they are declared.  This statement does not cover nfad_cmp_recompute_backward_noalloc,
 *     about which nothing is claimed here beyond what its own comment says.
 *   - n == 0 is valid and does nothing.  n is 64-bit: 2^30 fp32 elements and
 *     beyond are indexed correctly.
 *   - Return value: an nfad_status.  Nothing aborts or traps.  After
 *     NFAD_E_CUDA, nfad_last_cuda_error() gives the cudaError_t of the calling
 *     thread's failed call.
 *   - Non-finite input: NaN gives NaN in y and f'.  +inf gives y = +inf,
 *     f' = 1; -inf gives y = -0, f' = +-0.
 */
#ifndef NFAD_H_
#define NFAD_H_

#include <stddef.h>

#if defined(__GNUC__)
#define NFAD_API __attribute__((visibility("default")))
#else
#define NFAD_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

/* Activations: Table I (GELU in its tanh form, Mish, Swish) and the erf-exact
 * GELU x*Phi(x) that Table I's tanh form approximates.  The two GELUs are
 * different functions (they differ by up to ~5e-4) and are never interchanged. */
typedef enum {
    NFAD_GELU_ERF = 0,   /* x * (1 + erf(x / sqrt 2)) / 2                                  */
    NFAD_GELU_TANH = 1,  /* 0.5 x (1 + tanh( sqrt(2/pi) (x + 0.044715 x^3) ))   (Table I)  */
    NFAD_SWISH = 2,      /* x * sigmoid(x)                                       (Table I)  */
    NFAD_MISH = 3        /* x * tanh(softplus(x))                                (Table I)  */
} nfad_kind;

typedef enum { NFAD_F32 = 0, NFAD_BF16 = 1, NFAD_F16 = 2 } nfad_dtype;

typedef enum {
    NFAD_OK = 0,
    NFAD_E_KIND = 1,     /* kind is not an nfad_kind                                  */
    NFAD_E_DTYPE = 2,    /* dtype is not an nfad_dtype                                */
    NFAD_E_NULL = 3,     /* a tensor pointer is NULL while n > 0                      */
    NFAD_E_OVERLAP = 4,  /* forbidden aliasing, see above                             */
    NFAD_E_CUDA = 5,     /* a CUDA call failed: see nfad_last_cuda_error()            */
    NFAD_E_ALIGN = 6,    /* a pointer is not a multiple of the element size           */
    NFAD_E_SCRATCH = 7,  /* scratch_bytes is smaller than the comparator needs        */
    NFAD_E_LAYOUT = 8,   /* layout is not an nfad_layout                              */
    NFAD_E_TOO_LARGE = 9, /* the tensors need more than the library's built-in scratch */
    NFAD_E_PROGRAM = 10  /* malformed FAD sequence (see nfad_seq_forward)              */
} nfad_status;

/* How the tensor needed by backward is kept between the passes (Section II-C). */
typedef enum {
    NFAD_LAYOUT_NESTED = 0,     /* approach 3: keep f'(x)                                         */
    NFAD_LAYOUT_CONVENTIONAL = 1, /* keep x; one fused backward kernel re-derives f'(x)           */
    NFAD_LAYOUT_RECOMPUTE = 2,  /* approach 2: keep x; backward re-runs the forward operators     */
    NFAD_LAYOUT_OP_BY_OP = 3    /* approach 1: every operator keeps what its own rule needs       */
} nfad_layout;

typedef void* nfad_stream_t;   /* a cudaStream_t */

/*
 * Forward pass of the nested method (Section II-C approach 3; Eq. 3 for the
 * product rule that merges the tangents; Section II-D for the seed x' = 1).
 *   x     [in]  n elements
 *   y     [out] n elements, y[i] = f(x[i])
 *   dfdx  [out] n elements, dfdx[i] = f'(x[i]): the tensor to keep for backward
 * y may equal x (in place).  dfdx may equal x.  y and dfdx must not overlap.
 */
NFAD_API int nfad_act_forward(int kind, int dtype, const void* x, void* y, void* dfdx, size_t n, nfad_stream_t stream);

/*
 * Forward pass with the derivative held to the LITERAL 4-ulp bound for every input (fp32 storage
 * only; any other dtype gives NFAD_E_DTYPE).  For x < 0, f' = h + x h' (Eq. 3 applied to f = x h) is
 * a difference of two terms of similar size that changes sign, so arithmetic good to a fraction of an
 * fp32 ulp of the TERMS -- what nfad_act_forward guarantees there (2^-29 of each) -- is not good to an
 * fp32 ulp of f' within about 2^-8 of the terms' size of the sign change.  This entry point runs the
 * same dual-number chain on primitives good to the last bits of a double and rounds once: y and dfdx
 * are within about one fp32 ulp of the exact f(x) and f'(x) for every finite x, the fp32 neighbours of
 * the sign change included; results below 2^-126 are rounded once to the subnormal grid.  Away from
 * the sign change it agrees with nfad_act_forward to the last place or the one before.  Same pointer,
 * aliasing and stream rules.  Costs about twice the fp64 arithmetic of nfad_act_forward (see the
 * measured rates).  The 16-bit storage types need no such variant: there nfad_act_forward is within
 * one ulp of the correctly rounded f' for every input.
 */
NFAD_API int nfad_act_forward_strict(int kind, int dtype, const void* x, void* y, void* dfdx, size_t n, nfad_stream_t stream);

/*
 * Forward pass without the tangent (inference, or any pass that will not be
 * differentiated): the same chain of primitives, value parts only.
 *   x [in] n elements;  y [out] n elements (may equal x).
 */
NFAD_API int nfad_act_forward_infer(int kind, int dtype, const void* x, void* y, size_t n, nfad_stream_t stream);

/*
 * Backward pass of the nested method (Eq. 4, Section II-E): one multiplication,
 *   grad_in[i] = round( grad_out[i] * dfdx[i] ),
 * the product formed exactly and rounded once.  `kind` is validated but does
 * not change the result.  grad_in may equal grad_out or dfdx.
 */
NFAD_API int nfad_act_backward(int kind, int dtype, const void* grad_out, const void* dfdx, void* grad_in, size_t n,
                      nfad_stream_t stream);

/*
 * Comparator, conventional layout: the forward pass is nfad_act_forward_infer and
 * x itself is kept; this backward re-derives f'(x) from x with the whole
 * transcendental chain and multiplies, in one kernel (f' is not rounded to the
 * storage type on the way):  grad_in[i] = round( grad_out[i] * f'(x[i]) ).
 * grad_in may equal grad_out or x.
 */
NFAD_API int nfad_cmp_conv_backward(int kind, int dtype, const void* grad_out, const void* x, void* grad_in, size_t n,
                           nfad_stream_t stream);

/*
 * Comparator, recomputation layout (Section II-C approach 2): x is kept; backward
 * runs two kernels.  The first re-runs the forward operators and writes the
 * intermediate that the per-operator backward rules need (the gate h(x) of
 * f = x h(x): sigmoid(x) for Swish, i.e. v1 of the paper's example) to `scratch`
 * in the storage type; the second reads grad_out, x and that intermediate and
 * walks the rules of Eqs. 1-2: grad_in = g h + g x h'.
 *   scratch [scratch] at least nfad_cmp_recompute_scratch_bytes(kind, dtype, n)
 *           bytes of device memory, 16-byte aligned; contents undefined after.
 * Accuracy is that of operator-by-operator back-propagation through a stored
 * intermediate (1 - h is formed by subtraction), not that of the nested path.
 * grad_in may equal grad_out; it must not overlap x or scratch.
 */
NFAD_API int nfad_cmp_recompute_backward(int kind, int dtype, const void* grad_out, const void* x, void* scratch,
                                size_t scratch_bytes, void* grad_in, size_t n, nfad_stream_t stream);

/*
 * The recomputation comparator for callers that cannot hand over scratch memory.
 * (The paper has no counterpart: this is a convenience of this library.)
 *
 * Some users of this code have no way to allocate device memory at the point
 * where they call it: a plug-in running under a host application that hands out
 * all device memory up front and forbids cudaMalloc afterwards, a serving loop in
 * which an allocation's implicit device-wide synchronisation would stall every
 * other stream, or a component that is simply not given an allocator.  For them
 * this entry point does what nfad_cmp_recompute_backward does, bit for bit, but
 * takes its scratch from a fixed array of NFAD_NOALLOC_SCRATCH_BYTES that is part
 * of the library image (every GPU that loads the library holds those bytes
 * until the process exits).  It calls no allocation routine of any kind.
 *
 *   grad_out, x [in], grad_in [out]: n elements each, same rules as above;
 *   grad_in may equal grad_out and must not overlap x.
 *   n * element size must not exceed NFAD_NOALLOC_SCRATCH_BYTES (2 097 152 fp32 or
 *   4 194 304 bf16/fp16 elements); larger calls return NFAD_E_TOO_LARGE and launch
 *   nothing -- use nfad_cmp_recompute_backward with your own scratch instead.
 *
 * The first call on each device looks up the array's device address (a one-time
 * set-up with that device current); make that first call outside any stream
 * capture.  All calls on a device share the one array: it still holds whatever
 * the previous call left there (nothing in it needs to start at zero -- the first
 * kernel overwrites every byte the second one reads), and two calls whose
 * kernels may overlap on the GPU (different streams without an ordering between
 * them) race on it.  Serialise such calls, or give them their own scratch through
 * nfad_cmp_recompute_backward.
 */
#define NFAD_NOALLOC_SCRATCH_BYTES 8388608
NFAD_API int nfad_cmp_recompute_backward_noalloc(int kind, int dtype, const void* grad_out, const void* x,
                                                 void* grad_in, size_t n, nfad_stream_t stream);

/* Bytes of scratch the recomputation comparator needs for n elements; 0 on a bad kind or dtype. */
NFAD_API size_t nfad_cmp_recompute_scratch_bytes(int kind, int dtype, size_t n);

/*
 * Bytes per element that a layout keeps alive between the forward and the
 * backward pass.  Nested, conventional and recomputation keep one tensor;
 * operator-by-operator back-propagation keeps every tensor its rules need
 * (for Swish the paper's own count, x and sigmoid(x), Section II-C approach 1;
 * for the other kinds the count under the usual per-operator rules).
 * Returns a negative nfad_status on a bad argument.
 */
NFAD_API int nfad_saved_bytes_per_element(int kind, int dtype, int layout);

/*
 * FAD sequences composed at run time.
 *
 * The paper's method is not tied to four activations: any run of FAD-compatible
 * primitive operations (Section III-A: unary operations, binary operations whose
 * two inputs come from the same source, binary operations with one constant)
 * with one source and M >= 1 results (R^1 -> R^M, Section II-D "Computation
 * efficiency" and the state sequence NY, YY.., YN of Section IV) can be nested in
 * back-propagation the same way.  A sequence is a straight-line program over 12
 * dual registers; register 0 holds the source (x, tangent 1).  Each instruction
 * applies one primitive to register a (and b for ADD / MUL, which merge two
 * branches of the same source) and writes register dst; NFAD_OP_OUT copies
 * register a to result slot dst (0 <= dst < m).  SCALE and ADD_CONST take their
 * constant from c.
 *
 *   program [host] n_ops <= 32 instructions.  Malformed programs (unknown opcode, register
 *           out of range, a register read before it is written, a result slot out of
 *           range or never written) give NFAD_E_PROGRAM.
 *   x       [in]   n elements.
 *   y, dfdx [host arrays of m device pointers, m <= 4] y[k][i] = k-th result, dfdx[k][i] its
 *           derivative with respect to x[i]: per result, the one tensor to keep.
 * One kernel runs the whole sequence per element on dual numbers; no intermediate reaches
 * memory.  Arithmetic: fp32 primitives for the 16-bit storage types (a few fp32 ulp where the
 * composed function is well conditioned), fp64 primitives good to 2^-45 for fp32 storage (results
 * within a few fp32 ulp of the exact ones wherever the program itself does not cancel).  The
 * constants of a program are fp32 (`c` below).  The four activations of Table I have dedicated
 * entry points above.  Outputs must not overlap each other or x.
 */
typedef enum {
    NFAD_OP_ADD = 0, NFAD_OP_MUL = 1, NFAD_OP_SCALE = 2, NFAD_OP_ADD_CONST = 3, NFAD_OP_EXP = 4, NFAD_OP_LOG1P = 5,
    NFAD_OP_TANH = 6, NFAD_OP_ERF = 7, NFAD_OP_SOFTPLUS = 8, NFAD_OP_SIGMOID = 9, NFAD_OP_HALF_ONE_PLUS_TANH = 10,
    NFAD_OP_HALF_ONE_PLUS_ERF = 11, NFAD_OP_OUT = 12
} nfad_opcode;

typedef struct { int op; int a; int b; int dst; float c; } nfad_seq_op;

NFAD_API int nfad_seq_forward(const nfad_seq_op* program, int n_ops, int dtype, const void* x, void* const* y,
                              void* const* dfdx, int m, size_t n, nfad_stream_t stream);

/*
 * Two executors run a sequence.  The COMPILED one turns the program into straight-line device code
 * over the same dual primitives, compiles it for the device at hand with NVRTC on first use (about a
 * second per new (program, dtype, m); cached afterwards) and launches it as one kernel with every
 * dual number in hardware registers, like the dedicated activation kernels.  The INTERPRETER runs any
 * program at once with its registers in local memory and is several times slower.  Mode 0 (the
 * default): compiled when NVRTC, the driver library and this library's headers (the csrc directory
 * beside the library, or NFAD_JIT_INCLUDE) are available, otherwise interpreted; 1: always
 * interpreted; 2: compiled or fail (NFAD_E_CUDA with cudaErrorNotSupported or the compiler's error,
 * whose text nfad_seq_compile_log() returns).  The two executors run the same primitives, but the
 * compiler may contract across instruction boundaries: results can differ in the last bits.
 * nfad_seq_last_executor(): 1 = interpreter, 2 = compiled, for the calling thread's last sequence.
 * The first compiled call of a program must not be made inside a stream capture.
 */
NFAD_API int nfad_seq_set_executor(int mode);
NFAD_API int nfad_seq_last_executor(void);
NFAD_API const char* nfad_seq_compile_log(void);
/* The CUDA source the compiled executor builds for a sequence (valid until the calling thread's next call of this
 * function); NULL for a malformed program or a bad dtype.  Needs no device: for inspection and for testing the
 * generator where no GPU is present. */
NFAD_API const char* nfad_seq_compiled_source(const nfad_seq_op* program, int n_ops, int dtype, int m);

/*
 * Backward of a sequence with m results (Section II-E; for a binary merge "the post-process
 * will merge (accumulate) FAD results", Section IV): grad_in[i] = sum_k grad_out[k][i] * dfdx[k][i],
 * accumulated in fp32 in the order k = 0..m-1 with fused multiply-adds and rounded once.
 * For m == 1 this is nfad_act_backward.  grad_out, dfdx: host arrays of m device pointers.
 */
NFAD_API int nfad_seq_backward(int dtype, const void* const* grad_out, const void* const* dfdx, int m, void* grad_in,
                               size_t n, nfad_stream_t stream);

/*
 * One primitive as its own kernel, the way a framework runs it when every operator is a node
 * of the graph (Section II-C approach 1); used to MEASURE operator-by-operator back-propagation.
 *   forward  (backward == 0): out0 = op(in0 [, in1]) for ADD / MUL, op(in0) otherwise.
 *   backward (backward != 0): in0 = upstream gradient; in1 (, in2) = what the operator's rule kept:
 *       MUL: both operands (out0 = g * in2 is the gradient of the first operand, out1 = g * in1 of the second);
 *       EXP, TANH, SIGMOID, HALF_ONE_PLUS_TANH: the forward output;
 *       LOG1P, ERF, SOFTPLUS, HALF_ONE_PLUS_ERF: the forward input;  SCALE: nothing.
 *       ADD and ADD_CONST pass the gradient through and need no kernel.
 * Unused pointers are NULL.  Exact in-place use allowed.
 */
NFAD_API int nfad_ew_op(int op, int backward, float c, int dtype, const void* in0, const void* in1, const void* in2,
                        void* out0, void* out1, size_t n, nfad_stream_t stream);

/*
 * The pass fused with its producer's bias.
 *
 * A linear layer hands over x[rows, cols] (row-major, contiguous) and bias[cols]; the
 * activation sees z = x + bias.  From x's side the addition is a binary operation with
 * one constant input, which the method treats as unary (Section III-A), and dz/dx = 1:
 * the forward pass still emits y = f(z) and the one saved tensor f'(z), and the backward
 * pass is still the multiplication of Eq. 4.  From the bias's side dz/dbias = 1 on every
 * row, so its gradient is the column sum of that same product.  The paper only notes
 * that frameworks fuse such element-wise chains by hand (Section III); these two entry
 * points are that fusion for this library, and save one write and one read of the
 * pre-activation tensor forward and one read of grad_in backward.
 *
 * Forward:  z = x[r, c] + bias[c], formed by ONE fp32 addition (for every storage type);
 *           y[r, c] = f(z), dfdx[r, c] = f'(z), arithmetic and rounding as nfad_act_forward.
 *   x [in] rows*cols elements; bias [in] cols elements; y, dfdx [out] rows*cols elements.
 *   y may equal x; dfdx may equal x; bias must not overlap an output.
 *
 * Backward: grad_in[r, c] = round(grad_out[r, c] * dfdx[r, c]) exactly as nfad_act_backward, and
 *           grad_bias[c] = sum over r of the STORED (rounded) grad_in[r, c], accumulated in fp32
 *           in a fixed order (so the result is reproducible run to run and does not depend on
 *           pointer alignment): the rows are cut into chunks of consecutive rows, each chunk is
 *           summed in row order, then the chunks' sums are added in a fixed order (32 runs of
 *           consecutive chunks, then the runs).  grad_bias is always fp32.
 *   grad_out, dfdx [in], grad_in [out] rows*cols elements (grad_in may equal grad_out or dfdx);
 *   grad_bias [out] cols floats (4-byte aligned); scratch: device memory of at least
 *   nfad_bias_act_backward_scratch_bytes() bytes, 4-byte aligned, contents irrelevant before
 *   and after; may be NULL when that size is 0.  Too small a scratch gives NFAD_E_SCRATCH.
 *   rows == 0 gives grad_bias = 0.
 *
 * The 128-bit path needs cols to be a multiple of the packet (8 elements for the 16-bit
 * types, 4 for fp32) and 16-byte aligned tensors; otherwise every element is handled one
 * by one with identical results.  cols must be below 2^31 (NFAD_E_TOO_LARGE otherwise).
 * The scratch size depends on the current device (its SM count decides how the rows are
 * cut into chunks): ask for it with the device current that will run the call.
 */
NFAD_API int nfad_bias_act_forward(int kind, int dtype, const void* x, const void* bias, void* y, void* dfdx, size_t rows,
                                   size_t cols, nfad_stream_t stream);
/* The value-only form (a pass that will not be differentiated): y = f(x + bias), bit-identical to the y of
 * nfad_bias_act_forward; no dfdx. */
NFAD_API int nfad_bias_act_forward_infer(int kind, int dtype, const void* x, const void* bias, void* y, size_t rows,
                                         size_t cols, nfad_stream_t stream);
NFAD_API int nfad_bias_act_backward(int kind, int dtype, const void* grad_out, const void* dfdx, void* grad_in,
                                    float* grad_bias, void* scratch, size_t scratch_bytes, size_t rows, size_t cols,
                                    nfad_stream_t stream);
/* Bytes of scratch nfad_bias_act_backward needs on the current device; 0 on a bad dtype or when none is needed. */
NFAD_API size_t nfad_bias_act_backward_scratch_bytes(int dtype, size_t rows, size_t cols);

/*
 * The whole pass for tensors that live in HOST memory (no counterpart in the paper: a service entry
 * point for callers whose activations are kept off the device, and the end-to-end form of the pass
 * that the benchmark times).  Forward and backward of one batch:
 *   x_host, grad_out_host [in, host]   n elements each
 *   y_host, grad_in_host  [out, host]  n elements each: y = f(x), grad_in = round(grad_out * f'(x))
 *   dfdx_host             [out, host]  n elements or NULL: the saved tensor, if the caller wants it
 * with exactly the arithmetic of nfad_act_forward followed by nfad_act_backward (bit-identical
 * results).  The batch is cut into chunks that move through a three-stage pipeline -- host-to-device
 * copies on one internal stream, the two kernels on `stream`, device-to-host copies on a second
 * internal stream, chained by events -- so that both directions of the host link are busy at once.
 *   workspace [scratch, device] at least nfad_host_step_workspace_bytes(dtype, n) bytes for full speed,
 *             16-byte aligned; any size that holds one chunk of 2048 elements per slot works
 *             (NFAD_E_SCRATCH below that).  Contents undefined afterwards.
 * Host buffers should be page-locked (cudaHostAlloc / cudaHostRegister): pageable memory works but
 * the copies then block the calling thread and do not overlap.  Host buffers must not overlap one
 * another.  Completion is stream-ordered on `stream`: work enqueued on `stream` after the call, and a
 * synchronisation on it, see every result in host memory.  flags = 0: the inputs are read in stream
 * order too (the copies start when `stream` reaches the call).  flags = NFAD_HOST_INPUTS_READY: the
 * caller guarantees that x_host and grad_out_host hold their final contents when the call is made
 * and that no work pending on `stream` writes them; the input copies may then start at once, so
 * that consecutive calls keep both directions of the link busy across the call boundary.  Calls on
 * one device share the pipeline, whatever stream they name: the copies of a later call run after
 * those of an earlier one, and with either flag value a call whose workspace or chunk size differs
 * from the previous call's first waits until that call has finished with its workspace, so two
 * callers on different streams may not corrupt each other's slots (they do take turns).
 * Any other flag bit gives NFAD_E_LAYOUT.  State: two streams and a few events per
 * device, created on the first call on that device (make that call outside a stream capture; the
 * call itself cannot be captured into a graph) and kept until the process exits; enqueueing is
 * serialised by a mutex.
 */
#define NFAD_HOST_INPUTS_READY 1
NFAD_API int nfad_host_step(int kind, int dtype, const void* x_host, const void* grad_out_host, void* y_host, void* dfdx_host,
                            void* grad_in_host, size_t n, void* workspace, size_t workspace_bytes, int flags,
                            nfad_stream_t stream);
NFAD_API size_t nfad_host_step_workspace_bytes(int dtype, size_t n);

/*
 * Traffic probe (a measurement aid with no counterpart in the paper): moves
 * n_words 32-bit words per tensor through the same streaming kernel as the
 * activation pass, with a read/write mix of 1:1 (o0 = a), 1:2 (o0 = a, o1 = ~a)
 * or 2:1 (o0 = a ^ b), so that the bandwidth a given mix can reach on the device
 * is known beside the activation kernels' numbers.  Unused tensors may be NULL.
 * Two one-sided mixes measure the read and the write ceiling alone: 1:0 reads a and
 * writes nothing (o0 is a one-word sink that is only written if a checksum of the data
 * matches a fixed constant), 0:1 writes a fixed pattern to o0; both need a 16-byte
 * aligned tensor of a multiple of 4 words (NFAD_E_ALIGN otherwise).
 * Any other mix gives NFAD_E_LAYOUT.  Same pointer, aliasing and stream rules as above.
 */
NFAD_API int nfad_probe_stream(int reads, int writes, const void* a, const void* b, void* o0, void* o1, size_t n_words,
                               nfad_stream_t stream);

/* The cudaError_t (as an int) behind the calling thread's last NFAD_E_CUDA; 0 if none. */
NFAD_API int nfad_last_cuda_error(void);

/* A static, human-readable name for a status. */
NFAD_API const char* nfad_status_string(int status);

/* Library version, "major.minor.patch". */
NFAD_API const char* nfad_version(void);

#ifdef __cplusplus
}
#endif

#endif /* NFAD_H_ */
