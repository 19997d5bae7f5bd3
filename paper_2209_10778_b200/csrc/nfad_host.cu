// nfad_host.cu -- the whole pass for tensors that live in HOST memory.
//
// forward + backward of one batch (x, grad_out in host memory -> y, grad_in, optionally f' in host
// memory) as a three-stage pipeline over chunks: host-to-device copies on one internal stream, the two
// kernels on the caller's stream, device-to-host copies on a second internal stream, chained by
// events.  PCIe is full duplex and the kernels are ~100x faster than the copies, so the pass runs at
// the speed of the slower copy direction instead of the sum of both.  The saved tensor f' never leaves
// the device unless the caller asks for it.
//
// State: two streams and 3 * kSlots events per device, created on the first call on that device and
// kept until the process exits.  Enqueueing is serialised by a mutex (it is quick: a few hundred
// microseconds of host time).  Consecutive calls on one stream run one after the other: a call's copies
// start when the caller's stream reaches the call and the stream continues when its last result is out.
#include <stdint.h>

#include <mutex>

#include "../../include/nfad.h"
#include "nfad_internal.h"

namespace {

constexpr int kSlots = 4;                      // chunks in flight: one per pipeline stage and one of slack
constexpr int kMaxDevices = 64;
constexpr size_t kChunkAlign = 8 * 256;        // elements: whole tiles of the streaming kernels
// Per tensor and slot.  Measured on a 25 MB-per-tensor batch over PCIe 5 x16 (two calls per step, inputs ready):
// 1 MB chunks reach 6.7, 2 MB 8.4, 4 MB 10.2, 8 MB 11.2 and 16 MB 9.3 G elements/s -- every copy pays a fixed
// set-up cost, and too few chunks leave nothing to overlap.
constexpr size_t kPreferredChunkBytes = size_t(8) << 20;

struct DeviceState {
    bool ready = false;
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t in[kSlots], done[kSlots], out[kSlots], start, finish;
    // layout of the previous call's slots: a call with the same layout may run ahead into slots as they
    // free up; any other call first waits for the previous call to finish altogether
    const void* last_workspace = nullptr;
    size_t last_slot_bytes = 0;
};

std::mutex g_mutex;
DeviceState g_state[kMaxDevices];

size_t elem_size(int dtype) { return dtype == NFAD_F32 ? 4 : 2; }

cudaError_t device_state(DeviceState** out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    DeviceState& s = g_state[dev];
    if (!s.ready) {
        if ((e = cudaStreamCreateWithFlags(&s.h2d, cudaStreamNonBlocking)) != cudaSuccess) return e;
        if ((e = cudaStreamCreateWithFlags(&s.d2h, cudaStreamNonBlocking)) != cudaSuccess) return e;
        for (int i = 0; i < kSlots; ++i) {
            if ((e = cudaEventCreateWithFlags(&s.in[i], cudaEventDisableTiming)) != cudaSuccess) return e;
            if ((e = cudaEventCreateWithFlags(&s.done[i], cudaEventDisableTiming)) != cudaSuccess) return e;
            if ((e = cudaEventCreateWithFlags(&s.out[i], cudaEventDisableTiming)) != cudaSuccess) return e;
        }
        if ((e = cudaEventCreateWithFlags(&s.start, cudaEventDisableTiming)) != cudaSuccess) return e;
        if ((e = cudaEventCreateWithFlags(&s.finish, cudaEventDisableTiming)) != cudaSuccess) return e;
        s.ready = true;
    }
    *out = &s;
    return cudaSuccess;
}

// Elements per chunk that a workspace of `bytes` allows: 5 device tensors (x, g, y, f', grad_in) per slot.
size_t chunk_elements(int dtype, size_t n, size_t bytes)
{
    const size_t es = elem_size(dtype);
    size_t c = bytes / (size_t(kSlots) * 5 * es);
    const size_t want = kPreferredChunkBytes / es;
    if (c > want) c = want;
    c = c / kChunkAlign * kChunkAlign;
    if (c > n) c = (n + kChunkAlign - 1) / kChunkAlign * kChunkAlign;
    return c;
}

}  // namespace

extern "C" {

size_t nfad_host_step_workspace_bytes(int dtype, size_t n)
{
    if (dtype < 0 || dtype > 2 || n == 0) return 0;
    const size_t es = elem_size(dtype);
    size_t c = kPreferredChunkBytes / es;
    const size_t n_up = (n + kChunkAlign - 1) / kChunkAlign * kChunkAlign;
    if (c > n_up) c = n_up;
    return size_t(kSlots) * 5 * c * es;
}

int nfad_host_step(int kind, int dtype, const void* x_host, const void* grad_out_host, void* y_host, void* dfdx_host,
                   void* grad_in_host, size_t n, void* workspace, size_t workspace_bytes, int flags, nfad_stream_t stream)
{
    if (flags & ~NFAD_HOST_INPUTS_READY) return NFAD_E_LAYOUT;
    if (kind < 0 || kind > 3) return NFAD_E_KIND;
    if (dtype < 0 || dtype > 2) return NFAD_E_DTYPE;
    if (n == 0) return NFAD_OK;
    if (!x_host || !grad_out_host || !y_host || !grad_in_host || !workspace) return NFAD_E_NULL;
    const size_t es = elem_size(dtype);
    if (reinterpret_cast<uintptr_t>(workspace) & 15u) return NFAD_E_ALIGN;
    const size_t chunk = chunk_elements(dtype, n, workspace_bytes);
    if (chunk == 0) return NFAD_E_SCRATCH;

    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState* s = nullptr;
    cudaError_t e = device_state(&s);
    cudaStream_t compute = static_cast<cudaStream_t>(stream);
    auto fail = [&](cudaError_t err) {
        nfad::note_cuda_error(err);
        return NFAD_E_CUDA;
    };
    if (e != cudaSuccess) return fail(e);

    char* ws = static_cast<char*>(workspace);
    const size_t slot_bytes = 5 * chunk * es;
    const bool same_layout = s->last_workspace == workspace && s->last_slot_bytes == slot_bytes;
    if (!(flags & NFAD_HOST_INPUTS_READY)) {
        // fully stream-ordered: the input copies start after whatever the caller's stream holds at this point
        if ((e = cudaEventRecord(s->start, compute)) != cudaSuccess) return fail(e);
        if ((e = cudaStreamWaitEvent(s->h2d, s->start, 0)) != cudaSuccess) return fail(e);
    }
    if (!same_layout) {
        // the previous call on this device (from whatever stream) cut the workspace differently, or used another one that
        // may overlap this one: its slots are not this call's slots, so the per-slot events do not protect them.  Wait
        // until it has finished with all of them (a no-op when nothing is in flight).
        if ((e = cudaStreamWaitEvent(s->h2d, s->finish, 0)) != cudaSuccess) return fail(e);
    }
    s->last_workspace = workspace;
    s->last_slot_bytes = slot_bytes;
    size_t c_index = 0;
    for (size_t off = 0; off < n; off += chunk, ++c_index) {
        const int slot = int(c_index % kSlots);
        const size_t m = n - off < chunk ? n - off : chunk;
        const size_t bytes = m * es;
        char* base = ws + size_t(slot) * slot_bytes;
        void* dx = base;
        void* dg = base + chunk * es;
        void* dy = base + 2 * chunk * es;
        void* dd = base + 3 * chunk * es;
        void* dgin = base + 4 * chunk * es;
        const char* hx = static_cast<const char*>(x_host) + off * es;
        const char* hg = static_cast<const char*>(grad_out_host) + off * es;

        // stage 1: inputs in, once the slot's previous outputs (this call's, or the previous call's when it used the
        // same slots) have left; waiting on an event that was never recorded is a no-op
        if ((c_index >= size_t(kSlots) || same_layout) && (e = cudaStreamWaitEvent(s->h2d, s->out[slot], 0)) != cudaSuccess)
            return fail(e);
        if ((e = cudaMemcpyAsync(dx, hx, bytes, cudaMemcpyHostToDevice, s->h2d)) != cudaSuccess) return fail(e);
        if ((e = cudaMemcpyAsync(dg, hg, bytes, cudaMemcpyHostToDevice, s->h2d)) != cudaSuccess) return fail(e);
        if ((e = cudaEventRecord(s->in[slot], s->h2d)) != cudaSuccess) return fail(e);

        // stage 2: the two kernels on the caller's stream
        if ((e = cudaStreamWaitEvent(compute, s->in[slot], 0)) != cudaSuccess) return fail(e);
        int rc = nfad_act_forward(kind, dtype, dx, dy, dd, m, stream);
        if (rc == NFAD_OK) rc = nfad_act_backward(kind, dtype, dg, dd, dgin, m, stream);
        if (rc != NFAD_OK) return rc;
        if ((e = cudaEventRecord(s->done[slot], compute)) != cudaSuccess) return fail(e);

        // stage 3: results out
        if ((e = cudaStreamWaitEvent(s->d2h, s->done[slot], 0)) != cudaSuccess) return fail(e);
        if ((e = cudaMemcpyAsync(static_cast<char*>(y_host) + off * es, dy, bytes, cudaMemcpyDeviceToHost, s->d2h)) != cudaSuccess)
            return fail(e);
        if ((e = cudaMemcpyAsync(static_cast<char*>(grad_in_host) + off * es, dgin, bytes, cudaMemcpyDeviceToHost, s->d2h)) != cudaSuccess)
            return fail(e);
        if (dfdx_host &&
            (e = cudaMemcpyAsync(static_cast<char*>(dfdx_host) + off * es, dd, bytes, cudaMemcpyDeviceToHost, s->d2h)) != cudaSuccess)
            return fail(e);
        if ((e = cudaEventRecord(s->out[slot], s->d2h)) != cudaSuccess) return fail(e);
    }
    // the caller's stream completes only when every result is in host memory, and the next call's input
    // copies (ordered after s->start of that call) cannot overtake this call's kernels
    if ((e = cudaEventRecord(s->finish, s->d2h)) != cudaSuccess) return fail(e);
    if ((e = cudaStreamWaitEvent(compute, s->finish, 0)) != cudaSuccess) return fail(e);
    return NFAD_OK;
}

}  // extern "C"
