// nfad_jit.cu -- FAD sequences compiled at run time.
//
// A sequence is turned into straight-line CUDA over the dual primitives (one line per instruction,
// registers become named values), compiled for the device at hand with NVRTC around the fixed skeleton
// of nfad_jit_kernel.cuh, loaded through the driver API and cached per (program, storage type, result
// count, device).  The first call with a new sequence pays the compilation (about a second); later
// calls launch the cached kernel.  NVRTC and the driver library are opened with dlopen on first use, so
// the library itself has no link-time dependency on either and loads on machines without a GPU.
#include <cuda.h>
#include <dlfcn.h>
#include <nvrtc.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <unistd.h>

#include <map>
#include <mutex>
#include <string>
#include <vector>

#include "nfad_internal.h"
#include "nfad_jit_kernel.cuh"

namespace nfad {

namespace {

struct Api {
    bool tried = false, ok = false;
    std::string why;
    decltype(&nvrtcCreateProgram) create = nullptr;
    decltype(&nvrtcCompileProgram) compile = nullptr;
    decltype(&nvrtcGetProgramLogSize) log_size = nullptr;
    decltype(&nvrtcGetProgramLog) log = nullptr;
    decltype(&nvrtcGetCUBINSize) cubin_size = nullptr;
    decltype(&nvrtcGetCUBIN) cubin = nullptr;
    decltype(&nvrtcDestroyProgram) destroy = nullptr;
    CUresult (*module_load)(CUmodule*, const void*) = nullptr;
    CUresult (*module_get)(CUfunction*, CUmodule, const char*) = nullptr;
    CUresult (*launch)(CUfunction, unsigned, unsigned, unsigned, unsigned, unsigned, unsigned, unsigned, CUstream, void**, void**) = nullptr;
    std::string cuda_include, own_include;
};

std::mutex g_mutex;
Api g_api;
std::map<std::string, CUfunction> g_cache;
std::string g_log;
int g_mode = 0;          // 0 auto, 1 interpreter only, 2 compiled only
thread_local int g_last_executor = 0;   // 1 interpreter, 2 compiled

std::string dir_of(const std::string& path)
{
    size_t k = path.find_last_of('/');
    return k == std::string::npos ? std::string(".") : path.substr(0, k);
}

template <class F> bool sym(void* h, const char* name, F* out)
{
    *out = reinterpret_cast<F>(dlsym(h, name));
    return *out != nullptr;
}

void open_api()
{
    Api& a = g_api;
    a.tried = true;
    void* rtc = nullptr;
    for (const char* name : {"libnvrtc.so.12", "libnvrtc.so", "/usr/local/cuda/lib64/libnvrtc.so.12", "/usr/local/cuda/lib64/libnvrtc.so"}) {
        rtc = dlopen(name, RTLD_NOW | RTLD_LOCAL);
        if (rtc) break;
    }
    if (!rtc) { a.why = "libnvrtc not found"; return; }
    void* drv = dlopen("libcuda.so.1", RTLD_NOW | RTLD_LOCAL);
    if (!drv) { a.why = "libcuda.so.1 not found"; return; }
    bool ok = sym(rtc, "nvrtcCreateProgram", &a.create) && sym(rtc, "nvrtcCompileProgram", &a.compile) &&
              sym(rtc, "nvrtcGetProgramLogSize", &a.log_size) && sym(rtc, "nvrtcGetProgramLog", &a.log) &&
              sym(rtc, "nvrtcGetCUBINSize", &a.cubin_size) && sym(rtc, "nvrtcGetCUBIN", &a.cubin) &&
              sym(rtc, "nvrtcDestroyProgram", &a.destroy) && sym(drv, "cuModuleLoadData", &a.module_load) &&
              sym(drv, "cuModuleGetFunction", &a.module_get) && sym(drv, "cuLaunchKernel", &a.launch);
    if (!ok) { a.why = "a symbol of libnvrtc / libcuda is missing"; return; }
    // this library's own headers: next to it, in csrc/
    Dl_info info;
    if (const char* env = getenv("NFAD_JIT_INCLUDE")) a.own_include = env;
    else if (dladdr(reinterpret_cast<void*>(&open_api), &info) && info.dli_fname) a.own_include = dir_of(info.dli_fname) + "/csrc";
    // the toolkit's headers (cuda_bf16.h, cuda_fp16.h): the first of $CUDA_HOME/include, the include directory
    // beside the NVRTC that was loaded, /usr/local/cuda/include that really holds them
    std::vector<std::string> candidates;
    if (const char* env = getenv("CUDA_HOME")) candidates.push_back(std::string(env) + "/include");
    if (dladdr(reinterpret_cast<void*>(a.create), &info) && info.dli_fname) {
        char real[4096];
        std::string lib = realpath(info.dli_fname, real) ? std::string(real) : std::string(info.dli_fname);
        candidates.push_back(dir_of(dir_of(lib)) + "/include");
    }
    candidates.push_back("/usr/local/cuda/include");
    a.cuda_include = candidates.back();
    for (const std::string& c : candidates) {
        if (access((c + "/cuda_bf16.h").c_str(), R_OK) == 0) {
            a.cuda_include = c;
            break;
        }
    }
    a.ok = true;
}

const char* kOpExpr[] = {
    /* add */ "dual_add(%s, %s)", /* mul */ "dual_mul(%s, %s)", /* scale */ nullptr, /* add_const */ nullptr,
    /* exp */ "dual_exp(%s)", /* log1p */ "dual_log1p(%s)", /* tanh */ "dual_tanh(%s)", /* erf */ "dual_erf(%s)",
    /* softplus */ "dual_softplus(%s)", /* sigmoid */ "as_dual(dual_sigmoid(%s))",
    /* (1+tanh)/2 */ "as_dual(dual_half_one_plus_tanh(%s))", /* (1+erf)/2 */ "as_dual(dual_half_one_plus_erf(%s))"};

std::string generate(const SeqProgramHost& p, int m, const char* store)
{
    // fp32 tensors run under the double-precision policy, 16-bit tensors under the fp32 one (as the interpreter does)
    const bool wide = strcmp(store, "StoreF32") == 0;
    const char* pol = wide ? "Wide" : "Fast";
    char buf[512];
    std::string s = "#include \"nfad_jit_kernel.cuh\"\nnamespace nfad {\n";
    snprintf(buf, sizeof buf, "template <> __device__ __forceinline__ void jit_element<%d>(float x, float (&yv)[%d], float (&yt)[%d])\n{\n", m, m, m);
    s += buf;
    snprintf(buf, sizeof buf, wide ? "    const Dual<%s> v_src{double(x), 1.0};\n" : "    const Dual<%s> v_src{x, 1.0f};\n", pol);
    s += buf;
    std::string reg[12];
    reg[0] = "v_src";
    for (int i = 0; i < p.n_ops; ++i) {
        const std::string a = reg[p.a[i]], b = reg[p.b[i]];
        if (p.op[i] == 12) {                       // OUT
            snprintf(buf, sizeof buf, "    yv[%d] = dual_value(%s); yt[%d] = dual_tangent(%s);\n", p.dst[i], a.c_str(), p.dst[i], a.c_str());
            s += buf;
            continue;
        }
        unsigned bits;
        float c = p.c[i];
        memcpy(&bits, &c, 4);
        char cst[64], expr[256];
        snprintf(cst, sizeof cst, wide ? "double(__int_as_float(0x%08x))" : "__int_as_float(0x%08x)", bits);
        if (p.op[i] == 2) snprintf(expr, sizeof expr, "dual_scale(%s, %s)", cst, a.c_str());
        else if (p.op[i] == 3) snprintf(expr, sizeof expr, "dual_add_const(%s, %s)", cst, a.c_str());
        else if (p.op[i] < 2) snprintf(expr, sizeof expr, kOpExpr[p.op[i]], a.c_str(), b.c_str());
        else snprintf(expr, sizeof expr, kOpExpr[p.op[i]], a.c_str());
        snprintf(buf, sizeof buf, "    const Dual<%s> v%d = %s;\n", pol, i, expr);
        s += buf;
        snprintf(buf, sizeof buf, "v%d", i);
        reg[p.dst[i]] = buf;
    }
    s += "}\n}  // namespace nfad\n";
    snprintf(buf, sizeof buf, "extern \"C\" __global__ void __launch_bounds__(256, 4) nfad_seq_compiled(const nfad::JitArgs a)\n{\n    nfad::jit_forward<nfad::%s, %d>(a);\n}\n", store, m);
    s += buf;
    return s;
}

cudaError_t build(const std::string& src, int dev, CUfunction* out)
{
    Api& a = g_api;
    int major = 0, minor = 0;
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev);
    char arch[64];
    snprintf(arch, sizeof arch, (major == 10 && minor == 0) ? "--gpu-architecture=sm_100a" : "--gpu-architecture=sm_%d%d", major, minor);
    const std::string inc1 = "-I" + a.own_include, inc2 = "-I" + a.cuda_include;
    const char* opts[] = {arch, "--std=c++17", "--fmad=true", inc1.c_str(), inc2.c_str()};
    nvrtcProgram prog;
    if (a.create(&prog, src.c_str(), "nfad_seq_compiled.cu", 0, nullptr, nullptr) != NVRTC_SUCCESS) {
        g_log = "nvrtcCreateProgram failed";
        return cudaErrorUnknown;
    }
    nvrtcResult r = a.compile(prog, int(sizeof opts / sizeof opts[0]), opts);
    size_t ls = 0;
    a.log_size(prog, &ls);
    g_log.assign(ls ? ls - 1 : 0, '\0');
    if (ls > 1) a.log(prog, &g_log[0]);
    if (r != NVRTC_SUCCESS) {
        a.destroy(&prog);
        return cudaErrorUnknown;
    }
    size_t cs = 0;
    a.cubin_size(prog, &cs);
    std::vector<char> image(cs);
    a.cubin(prog, image.data());
    a.destroy(&prog);
    cudaFree(nullptr);                             // makes sure the primary context exists and is current
    CUmodule mod;
    if (a.module_load(&mod, image.data()) != CUDA_SUCCESS) { g_log += "\ncuModuleLoadData failed"; return cudaErrorUnknown; }
    if (a.module_get(out, mod, "nfad_seq_compiled") != CUDA_SUCCESS) { g_log += "\ncuModuleGetFunction failed"; return cudaErrorUnknown; }
    return cudaSuccess;
}

}  // namespace

std::string seq_generate_source(const SeqProgramHost& p, int dtype, int m)
{
    return generate(p, m, dtype == kF32 ? "StoreF32" : dtype == kBF16 ? "StoreBF16" : "StoreF16");
}

int seq_executor_mode() { return g_mode; }
void seq_set_executor_mode(int mode) { std::lock_guard<std::mutex> lock(g_mutex); g_mode = mode; }
int seq_last_executor() { return g_last_executor; }
void seq_note_executor(int which) { g_last_executor = which; }
const char* seq_jit_log()
{
    std::lock_guard<std::mutex> lock(g_mutex);
    static thread_local std::string copy;
    copy = g_api.tried && !g_api.ok ? g_api.why : g_log;
    return copy.c_str();
}

// cudaSuccess: launched.  cudaErrorNotSupported: the compiled executor is not available here (the caller may
// interpret instead).  Anything else: a real failure.
cudaError_t launch_seq_forward_compiled(const SeqProgramHost& p, int dtype, const void* x, void* const* y, void* const* d, int m,
                                        size_t n, cudaStream_t st)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    CUfunction f = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!g_api.tried) open_api();
        if (!g_api.ok) return cudaErrorNotSupported;
        std::string key(reinterpret_cast<const char*>(&p), sizeof p);
        key.push_back(char(dtype));
        key.push_back(char(m));
        key.push_back(char(dev));
        auto it = g_cache.find(key);
        if (it == g_cache.end()) {
            const char* store = dtype == kF32 ? "StoreF32" : dtype == kBF16 ? "StoreBF16" : "StoreF16";
            CUfunction built = nullptr;
            e = build(generate(p, m, store), dev, &built);
            g_cache[key] = e == cudaSuccess ? built : nullptr;      // a failed build is remembered, not retried
            f = g_cache[key];
        } else {
            f = it->second;
        }
    }
    if (!f) return cudaErrorNotSupported;
    JitArgs a;
    a.x = x;
    const size_t esz = dtype == kF32 ? 4 : 2, vec = 16 / esz;
    uintptr_t mis = reinterpret_cast<uintptr_t>(x) & 15u;
    bool congruent = true;
    for (int k = 0; k < kJitMaxOut; ++k) {
        a.y[k] = k < m ? y[k] : nullptr;
        a.d[k] = k < m ? d[k] : nullptr;
        if (k < m)
            congruent = congruent && ((reinterpret_cast<uintptr_t>(y[k]) & 15u) == mis) && ((reinterpret_cast<uintptr_t>(d[k]) & 15u) == mis);
    }
    a.n = n;
    if (congruent) {
        size_t head = ((16u - mis) & 15u) / esz;
        a.head = head > n ? n : head;
        a.packets = (n - a.head) / vec;
    } else {
        a.head = n;
        a.packets = 0;
    }
    const size_t tile = size_t(256) * kJitUnroll;
    size_t blocks = (a.packets + tile - 1) / tile;
    if (!congruent) blocks = edge_grid_blocks(n, 256);      // every element goes through the element-wise path: fill the device
    if (blocks == 0) blocks = 1;
    if (blocks > 0x7fffffffull) blocks = 0x7fffffffull;
    void* params[1] = {&a};
    CUresult r = g_api.launch(f, (unsigned)blocks, 1, 1, 256, 1, 1, 0, reinterpret_cast<CUstream>(st), params, nullptr);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorLaunchFailure;
}

}  // namespace nfad
