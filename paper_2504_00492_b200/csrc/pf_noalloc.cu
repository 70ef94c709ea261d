// pf_deltanet_fwd_f32_static: the fp32 forward pass for callers that must not allocate device memory.
//
// Some callers cannot call cudaMalloc (or anything that allocates) at the point where they need this
// operation: code running while a stream is being captured, real-time loops that forbid allocation
// after start-up, hosts embedding the library under a fixed device-memory budget, or processes whose
// allocator is owned by another runtime.  The other entry points take their per-chunk scratch from
// the stream-ordered allocator or from a caller buffer; this one keeps it in a fixed array that is
// part of the library image, so it allocates nothing.  The price: the array (PF_STATIC_SCRATCH_BYTES)
// is resident on every GPU that loads the library until the process exits, and problems whose scratch
// would not fit are refused.
#include <mutex>

#include "pf_common.cuh"

namespace pf {
namespace {

constexpr size_t kStaticScratchBytes = 8u << 20;   // 8 MiB; keep in step with PF_STATIC_SCRATCH_BYTES

// Scratch of the four SIMT kernels (T', W, Uh, P per chunk).  In HOST code this name is only a handle
// for cudaGetSymbolAddress -- it is not a device address and must never be passed to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device, once resolved

// Resolves the array's device address for the CURRENT device (once per device).
int static_scratch(void** out) {
    int dev = 0;
    PF_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return PF_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
        void* ptr = nullptr;
        PF_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        if (!ptr) return record_cuda_error(cudaErrorInvalidSymbol, "cudaGetSymbolAddress(g_static_scratch)");
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return PF_OK;
}

}  // namespace
}  // namespace pf

extern "C" size_t pf_static_scratch_bytes(void) { return pf::kStaticScratchBytes; }

extern "C" size_t pf_static_scratch_need(int B, int H, int L, int d_k, int d_v, int r, int chunk) {
    pf::Problem p{};
    p.B = B; p.H = H; p.L = L; p.d_k = d_k; p.d_v = d_v; p.r = r; p.chunk = chunk;
    p.in_dtype = PF_DTYPE_F32;
    return pf::simt_workspace_bytes(p);
}

extern "C" int pf_deltanet_fwd_f32_static(const float* q, const float* k, const float* v, const float* beta,
                                          const float* S0, int B, int H, int L, int d_k, int d_v, int r, int chunk,
                                          float* O, float* S_final, void* stream) {
    using namespace pf;
    // the same checks as the allocating entry point (shape, pointers, alignment, O not overlapping an input, device)
    pf_params a{};
    a.q = q; a.k = k; a.v = v; a.beta = beta; a.S0 = S0;
    a.B = B; a.H = H; a.L = L; a.d_k = d_k; a.d_v = d_v; a.r = r; a.chunk = chunk;
    a.O = O; a.S_final = S_final;
    a.in_dtype = PF_DTYPE_F32;
    a.impl = PF_IMPL_SIMT;
    a.stream = stream;
    int st = check_call(&a);
    if (st != PF_OK) return st;

    Problem p{};
    p.q = q; p.k = k; p.v = v; p.beta = beta; p.S0 = S0;
    p.B = B; p.H = H; p.L = L; p.d_k = d_k; p.d_v = d_v; p.r = r; p.chunk = chunk;
    p.O = O; p.S_final = S_final;
    p.in_dtype = PF_DTYPE_F32;
    p.stream = (cudaStream_t)stream;
    if (simt_workspace_bytes(p) > kStaticScratchBytes) return PF_ERR_WORKSPACE;   // too large for the fixed array

    void* scratch = nullptr;
    st = static_scratch(&scratch);
    if (st != PF_OK) return st;
    // Every word of the scratch that the kernels read is written earlier in the same call (gram writes
    // all of T and P, solve rewrites T, wu writes all of W and Uh), so nothing has to be cleared.
    begin_call();
    st = simt_forward(p, scratch);
    if (st == PF_OK) end_call();
    return st;
}
