// nfad_dispatch.cuh -- (op, kind) -> template instance, shared by both kernel
// translation units.
#pragma once

#include "nfad_internal.h"
#include "nfad_ops.cuh"
#include "nfad_stream.cuh"

namespace nfad {

template <class S, class P, class K>
cudaError_t dispatch_op(OpCode op, const void* const* in, void* const* out, size_t n, cudaStream_t st)
{
    switch (op) {
    case kOpForward:      return launch_stream<S, ForwardTrainOp<K, P>>(in, out, n, st);
    case kOpForwardInfer: return launch_stream<S, ForwardInferOp<K, P>>(in, out, n, st);
    case kOpBackward:     return launch_stream<S, BackwardOp>(in, out, n, st);
    case kOpConvBackward: return launch_stream<S, ConvBackwardOp<K, P>>(in, out, n, st);
    case kOpRecompute1:   return launch_stream<S, RecomputePhase1Op<K, P>>(in, out, n, st);
    case kOpRecompute2:   return launch_stream<S, RecomputePhase2Op<K, P>>(in, out, n, st);
    default: break;
    }
    return cudaErrorInvalidValue;
}

template <class S, class P>
cudaError_t dispatch_kind(OpCode op, int kind, const void* const* in, void* const* out, size_t n, cudaStream_t st)
{
    switch (kind) {
    case kGeluErf:  return dispatch_op<S, P, GeluErf>(op, in, out, n, st);
    case kGeluTanh: return dispatch_op<S, P, GeluTanh>(op, in, out, n, st);
    case kSwish:    return dispatch_op<S, P, Swish>(op, in, out, n, st);
    case kMish:     return dispatch_op<S, P, Mish>(op, in, out, n, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace nfad
