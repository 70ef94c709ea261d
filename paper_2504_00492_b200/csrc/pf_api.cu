// extern "C" entry points: argument checks, implementation choice, scratch memory, dispatch.
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "pf_common.cuh"
#include "pf_tc.cuh"
#include "pf_tc_prims.cuh"

namespace pf {

static thread_local char g_err[512] = "";
static thread_local int g_launches = 0;
static thread_local int g_wait_code = 0;
static thread_local int g_launch_accum = 0;

int record_cuda_error(cudaError_t e, const char* where) {
    snprintf(g_err, sizeof(g_err), "%s: %s (%s)", where, cudaGetErrorName(e), cudaGetErrorString(e));
    return PF_ERR_CUDA;
}

void count_launch(int n) { g_launch_accum += n; }

// ---- optional per-kernel timing ---------------------------------------------------------------
struct ProfEntry {
    char name[48];
    cudaEvent_t e0, e1;
};
static bool g_prof_on = false;
static ProfEntry g_prof[64];
static int g_prof_n = 0;       // entries of the current call
static int g_prof_made = 0;    // events created so far

void prof_begin(const char* name, cudaStream_t stream) {
    if (!g_prof_on || g_prof_n >= 64) return;
    ProfEntry& e = g_prof[g_prof_n];
    if (g_prof_n >= g_prof_made) {
        if (cudaEventCreate(&e.e0) != cudaSuccess || cudaEventCreate(&e.e1) != cudaSuccess) return;
        g_prof_made = g_prof_n + 1;
    }
    snprintf(e.name, sizeof(e.name), "%s", name);
    cudaEventRecord(e.e0, stream);
}

void prof_end(cudaStream_t stream) {
    if (!g_prof_on || g_prof_n >= 64 || g_prof_n >= g_prof_made) return;
    cudaEventRecord(g_prof[g_prof_n].e1, stream);
    ++g_prof_n;
}

namespace {

// The library's own status word (one per device that loads the library).  In host code the name is only a handle
// for cudaGetSymbolAddress; its device address is looked up once per device.
static __device__ int g_status_word;
constexpr int kMaxDevices = 64;
std::mutex g_status_mu;
int* g_status_ptr[kMaxDevices] = {};

int library_status_word(int** out) {
    int dev = 0;
    PF_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return PF_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_status_mu);
    if (!g_status_ptr[dev]) {
        void* ptr = nullptr;
        PF_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_status_word));
        g_status_ptr[dev] = (int*)ptr;
    }
    *out = g_status_ptr[dev];
    return PF_OK;
}

// One warp waits for a flag that nothing sets, with the bounded-wait routine of the kernels and a short limit.
__global__ void wait_selftest_kernel(int* status, const int* flag, long long limit_cycles) {
    if (threadIdx.x == 0) tc::flag_wait_ge_limit(flag, 1, status, 900, limit_cycles);
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

int check_shape(int B, int H, int L, int d_k, int d_v, int r, int chunk) {
    if (B < 1 || H < 1 || L < 0) return PF_ERR_INVALID;
    if (!(d_k == 64 || d_k == 128) || !(d_v == 64 || d_v == 128)) return PF_ERR_UNSUPPORTED;
    if (r < 1 || r > 4) return PF_ERR_UNSUPPORTED;
    if (!(chunk == 16 || chunk == 32 || chunk == 64)) return PF_ERR_UNSUPPORTED;
    return PF_OK;
}

Problem as_problem(int B, int H, int L, int d_k, int d_v, int r, int chunk, int in_dtype) {
    Problem p{};
    p.B = B; p.H = H; p.L = L; p.d_k = d_k; p.d_v = d_v; p.r = r; p.chunk = chunk;
    p.in_dtype = in_dtype;
    return p;
}

// option fields of pf_params: 0 = default
int check_options(const pf_params* a) {
    if (a->segments < 0 || a->segments > 64) return PF_ERR_INVALID;
    if (a->wu_builder != 0 && a->wu_builder != 1) return PF_ERR_INVALID;
    if (a->ring_depth != 0 && (a->ring_depth < 3 || a->ring_depth > 64)) return PF_ERR_INVALID;
    if (a->status && ((uintptr_t)a->status & 3u)) return PF_ERR_ALIGNMENT;
    return PF_OK;
}
Problem as_problem(const pf_params* a) {
    Problem p = as_problem(a->B, a->H, a->L, a->d_k, a->d_v, a->r, a->chunk, a->in_dtype);
    p.mode = a->mode;
    p.wu_builder = a->wu_builder;
    p.ring_depth = a->ring_depth;
    return p;
}

// Picks the kernels.  The tensor-core kernels take up to 128 rows per chunk (tiles of 64 or 128).  A chunk with more
// rows (r = 4 with chunk 64 has 256, r = 3 with chunk 64 has 192) is evaluated as consecutive blocks of whole tokens
// with at most 128 rows each: block forward substitution of the chunk's triangular system (the block-triangular case
// of the Proposition after Theorem 3.2), in which the coupling of a block to the blocks before it, A_21 [Uh_1 | W_1],
// is carried by the state, because flows compose exactly (Proposition 2.1).  In effect p.chunk becomes the block
// length; pf_select_chunk reports it.  PF_IMPL_AUTO also moves to a longer chunk when the caller's gives fewer than
// 64 rows (the result does not depend on the chunk length beyond rounding); explicit implementations never lengthen it.
int select_impl(Problem& p, int impl) {
    if (p.in_dtype != PF_DTYPE_BF16 && p.in_dtype != PF_DTYPE_F32) return PF_ERR_UNSUPPORTED;
    p.auto_impl = impl == PF_IMPL_AUTO;
    const bool tc_family = impl == PF_IMPL_AUTO || impl == PF_IMPL_TC || impl == PF_IMPL_TC_SPLIT;
    if (tc_family && !tc_supported(p)) {
        // (42 tokens of r = 3 rows are 126 of a tile's 128 rows: the longest block of rank 3 that fits)
        for (int c : {64, 42, 32, 16}) {
            if (impl != PF_IMPL_AUTO && c >= p.chunk) continue;
            Problem t = p;
            t.chunk = c;
            if ((c != 42 || (p.r == 3 && p.chunk > 42)) && tc_supported(t)) {
                p.chunk = c;
                break;
            }
        }
    }
    switch (impl) {
        case PF_IMPL_SIMT: return PF_IMPL_SIMT;
        case PF_IMPL_TC: return tc_supported(p) ? (int)PF_IMPL_TC : (int)PF_ERR_UNSUPPORTED;
        case PF_IMPL_AUTO: return tc_supported(p) ? PF_IMPL_TC : PF_IMPL_SIMT;
        case PF_IMPL_TC_SPLIT: return tc_supported(p) ? (int)PF_IMPL_TC_SPLIT : (int)PF_ERR_UNSUPPORTED;
        case PF_IMPL_TC_REFFLOW: return tc_scan_supported(p) ? (int)PF_IMPL_TC_REFFLOW : (int)PF_ERR_UNSUPPORTED;
        default: return PF_ERR_UNSUPPORTED;
    }
}

// PF_IMPL_TC: the single launch where it supports the shape; under PF_IMPL_AUTO only where it is also the faster of
// the two tensor-core forms (an explicit PF_IMPL_TC takes it whenever it can run).
bool use_fused(const Problem& p) { return fused_supported(p) && (!p.auto_impl || fused_preferred(p)); }

// what the kernels of `impl` carve up (the fp32 step sizes of PF_STEP_EXACT follow it)
size_t kernel_workspace_need(const Problem& p, int impl) {
    if (impl == PF_IMPL_TC) return use_fused(p) ? fused_workspace_bytes(p) : tc_workspace_bytes(p);
    if (impl == PF_IMPL_TC_SPLIT) return tc_workspace_bytes(p);
    if (impl == PF_IMPL_TC_REFFLOW) return tc_refflow_workspace_bytes(p);
    return simt_workspace_bytes(p);
}
size_t workspace_need(const Problem& p, int impl) {
    return align_up(kernel_workspace_need(p, impl), 256) + beta32_bytes(p);
}

// PF_STEP_EXACT: beta'[m] = (1 - e^{-beta_m |k_m|^2}) / |k_m|^2 for every factor m (a row of k); beta_m where k_m = 0.
// One warp per row.
template <class Tin>
__global__ void __launch_bounds__(256) exact_steps_kernel(const Tin* __restrict__ k, const Tin* __restrict__ beta,
                                                          float* __restrict__ out, long long rows, int d_k) {
    const long long m = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (m >= rows) return;
    const int lane = threadIdx.x & 31;
    float s = 0.f;
    for (int i = lane; i < d_k; i += 32) {
        const float x = (float)k[m * d_k + i];
        s = fmaf(x, x, s);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) {
        const float b = (float)beta[m];
        out[m] = s > 0.f ? -expm1f(-b * s) / s : b;
    }
}

bool overlaps(const void* a, size_t an, const void* b, size_t bn) {
    if (!a || !b || an == 0 || bn == 0) return false;
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + bn && b0 < a0 + an;
}

}  // namespace

// Checks that every entry point makes before anything is launched: shape, mode and step, pointers, alignment, O not
// overlapping an input, device architecture.
int check_call(const pf_params* a) {
    if (!a) return PF_ERR_INVALID;
    int st = check_shape(a->B, a->H, a->L, a->d_k, a->d_v, a->r, a->chunk);
    if (st != PF_OK) return st;
    if (a->in_dtype != PF_DTYPE_BF16 && a->in_dtype != PF_DTYPE_F32) return PF_ERR_UNSUPPORTED;
    if (a->mode != PF_MODE_SUM && a->mode != PF_MODE_PRODUCT) return PF_ERR_INVALID;
    if (a->step != PF_STEP_EULER && a->step != PF_STEP_EXACT) return PF_ERR_INVALID;
    if (a->step == PF_STEP_EXACT && a->mode == PF_MODE_SUM && a->r != 1) return PF_ERR_UNSUPPORTED;   // rank-1 factors only
    st = check_options(a);
    if (st != PF_OK) return st;
    if (a->L > 0 && (!a->q || !a->k || !a->v || !a->beta || !a->O)) return PF_ERR_INVALID;
    if (!aligned16(a->q) || !aligned16(a->k) || !aligned16(a->v) || !aligned16(a->beta) || !aligned16(a->O) ||
        !aligned16(a->S0) || !aligned16(a->S_final))
        return PF_ERR_ALIGNMENT;
    const size_t es = a->in_dtype == PF_DTYPE_F32 ? 4 : 2;
    const size_t th = (size_t)a->B * a->H * a->L;
    const size_t o_bytes = th * a->d_v * 4;
    if (overlaps(a->O, o_bytes, a->q, th * a->d_k * es) || overlaps(a->O, o_bytes, a->k, th * a->r * a->d_k * es) ||
        overlaps(a->O, o_bytes, a->v, th * a->r * a->d_v * es) || overlaps(a->O, o_bytes, a->beta, th * a->r * es))
        return PF_ERR_INVALID;
    int dev = 0;
    PF_CUDA_TRY(cudaGetDevice(&dev));
    int major = 0;
    PF_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    if (major != 10) return PF_ERR_ARCH;
    return PF_OK;
}

// A new top-level call begins: the launch count and the profile list start over.
void begin_call() {
    g_launch_accum = 0;
    g_prof_n = 0;
}
void end_call() { g_launches = g_launch_accum; }

namespace {

// One forward call on the problem as given.  `top`: this is the caller's call itself (it resets and publishes the
// launch count and the profile list); false for the passes of a segmented call.
int forward_one(const pf_params* a, bool top) {
    int st = check_call(a);
    if (st != PF_OK) return st;
    Problem p = as_problem(a);
    const int impl = select_impl(p, a->impl);
    if (impl < 0) return impl;

    p.q = a->q; p.k = a->k; p.v = a->v; p.beta = a->beta; p.S0 = a->S0;
    p.O = a->O; p.S_final = a->S_final;
    p.stream = (cudaStream_t)a->stream;

    const size_t need = workspace_need(p, impl);
    void* ws = a->workspace;
    bool own = false;
    if (ws) {
        if (a->workspace_bytes < need || ((uintptr_t)ws & 255u)) return PF_ERR_WORKSPACE;
    } else if (need > 0) {
        PF_CUDA_TRY(cudaMallocAsync(&ws, need, p.stream));
        own = true;
    }
    if (top) begin_call();
    // the status word of this call: the caller's, else word 0 of the caller's workspace, else the library's own
    if (a->status) p.status = a->status;
    else if (a->workspace) p.status = (int*)ws;
    else {
        st = library_status_word(&p.status);
        if (st != PF_OK) {
            if (own) cudaFreeAsync(ws, p.stream);
            return st;
        }
    }
    if (top) {      // (the passes of a segmented call share the word: the first expired wait of any of them stays)
        cudaError_t e = cudaMemsetAsync(p.status, 0, sizeof(int), p.stream);
        if (e != cudaSuccess) {
            if (own) cudaFreeAsync(ws, p.stream);
            return record_cuda_error(e, "cudaMemsetAsync(status)");
        }
    }
    const long long rows = (long long)p.B * p.H * p.L * p.r;
    if (a->step == PF_STEP_EXACT && rows > 0) {
        float* b32 = (float*)((uint8_t*)ws + align_up(kernel_workspace_need(p, impl), 256));
        const unsigned grid = (unsigned)((rows + 7) / 8);
        prof_begin("exact_steps", p.stream);
        if (p.in_dtype == PF_DTYPE_F32)
            exact_steps_kernel<float><<<grid, 256, 0, p.stream>>>((const float*)p.k, (const float*)p.beta, b32, rows, p.d_k);
        else
            exact_steps_kernel<__nv_bfloat16><<<grid, 256, 0, p.stream>>>((const __nv_bfloat16*)p.k,
                                                                          (const __nv_bfloat16*)p.beta, b32, rows, p.d_k);
        prof_end(p.stream);
        count_launch();
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) {
            if (own) cudaFreeAsync(ws, p.stream);
            return record_cuda_error(e, "exact_steps_kernel");
        }
        p.beta32 = b32;
    }
    if (impl == PF_IMPL_TC) st = use_fused(p) ? fused_forward(p, ws) : tc_forward(p, ws);
    else if (impl == PF_IMPL_TC_SPLIT) st = tc_forward(p, ws);
    else if (impl == PF_IMPL_TC_REFFLOW) st = tc_forward_refflow(p, ws);
    else st = simt_forward(p, ws);
    if (own) {
        cudaError_t e = cudaFreeAsync(ws, p.stream);
        if (e != cudaSuccess && st == PF_OK) st = record_cuda_error(e, "cudaFreeAsync");
    }
    if (st == PF_OK && top) end_call();
    return st;
}

// ---- segmented evaluation: the flows of S segments of every sequence in parallel, then their composition --------
// Section 3, step 3 ("Scan"): the flow of an interval is the pair (P, Xi) with S_end = S_start P + Xi (Proposition 2.1),
// and flows of consecutive intervals compose.  A sequence of L tokens is cut into S segments of L/S tokens, which the
// kernels see as S independent sequences (the layout [B,H,L,...] makes that a change of H and L, not a copy).  The
// whole pass is linear in (S_start, v), so a segment's output splits into the part its own tokens write and the part
// its start state contributes:
//   pass A: every segment from the zero state, the caller's v   -> O_zero (into O),  S_final = Xi_seg
//   pass R: every segment from the identity (d_v = d_k), v = 0  -> R[t][i] = (P_t q_t)[i], the query as the start state
//           sees it (an O-shaped scratch),                         S_final = P_seg   (row j of the state carries e_j P)
//   compose (one small kernel, serial over the S segments of a sequence, parallel over sequences and rows):
//           start(0) = S0,  start(s+1) = start(s) P_s + Xi_s;  the last one is S_final
//   apply:  O[t][:] += start(s)^T-contracted R[t][:]   (one GEMM per segment, no serial dependence)
// Two passes instead of one, each S times more parallel, and no pass waits for the composition: worth it when B*H is
// far below the SM count.
struct SegArrays {
    float* xi;      // [B*H*S][d_k][d_v]  pass A's S_final
    float* pb;      // same, pass R's
    float* start;   // same, start state of every segment
    float* ident;   // same, identity in every slot (the S0 of pass R)
};
size_t seg_array_bytes(const pf_params* a, int S) {
    return align_up((size_t)a->B * a->H * S * a->d_k * a->d_v * sizeof(float), 256);
}
size_t seg_response_bytes(const pf_params* a) {      // R: one fp32 d_k-vector per token-head
    return align_up((size_t)a->B * a->H * a->L * a->d_k * sizeof(float), 256);
}
size_t seg_zero_v_bytes(const pf_params* a) {
    const size_t es = a->in_dtype == PF_DTYPE_F32 ? 4 : 2;
    return align_up((size_t)a->B * a->H * a->L * a->r * a->d_v * es, 256);
}

__global__ void seg_identity_kernel(float* __restrict__ out, long long slots, int d) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= slots * d * d) return;
    const int r = (int)((e / d) % d), c = (int)(e % d);
    out[e] = r == c ? 1.f : 0.f;
}

// grid (B*H, d/16), 256 threads; thread (jj, tx): row j = 16*blockIdx.y + jj of the state, columns i = tx, tx + 16, ...
// Arrays are in the API layout X[i][j] = S[j][i].  The steps are serial, so each step's P and Xi are fetched into
// registers while the step before is being computed.
template <int D>
__global__ void __launch_bounds__(256) seg_compose_kernel(const float* __restrict__ S0, SegArrays arr,
                                                          float* __restrict__ S_final, int S) {
    constexpr int d = D;
    extern __shared__ float sm[];
    constexpr int ld = d + 4;       // (padded: the threads of a warp read 16 consecutive rows of Ps, 16 bytes each, without bank conflicts)
    float* Ps = sm;                 // [d][ld]  Ps[i][i'] = P[i'][i], as pass R's S_final stores it
    float* cur = sm + d * ld;       // [16][d]  rows of the current state
    const long long bh = blockIdx.x;
    const int j0 = blockIdx.y * 16;
    const int jj = threadIdx.x >> 4, tx = threadIdx.x & 15;
    constexpr int per = d / 16;     // columns per thread: 8 (d = 128) or 4 (d = 64)
    constexpr int NV = d * d / 4 / 256;     // 16-byte pieces of P per thread: 16 or 4
    for (int e = threadIdx.x; e < 16 * d; e += 256) {
        const int r = e / d, i = e % d;
        cur[e] = S0 ? S0[(bh * d + i) * d + j0 + r] : 0.f;
    }
    float4 pv[NV];
    float xv[per];
    auto fetch = [&](int s) {
        const long long slot = bh * S + s;
        const float4* pb = (const float4*)(arr.pb + slot * d * d);
        const float* xi = arr.xi + slot * d * d;
#pragma unroll
        for (int u = 0; u < NV; ++u) pv[u] = pb[u * 256 + threadIdx.x];
#pragma unroll
        for (int c = 0; c < per; ++c) xv[c] = xi[(long long)(tx + 16 * c) * d + j0 + jj];
    };
    fetch(0);
    __syncthreads();
    for (int s = 0; s < S; ++s) {
        const long long slot = bh * S + s;
        float* st = arr.start + slot * d * d;
        for (int e = threadIdx.x; e < 16 * d; e += 256) {
            const int r = e % 16, i = e / 16;
            st[(long long)i * d + j0 + r] = cur[r * d + i];
        }
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int e = (u * 256 + threadIdx.x) * 4;
            *(float4*)(Ps + (e / d) * ld + (e % d)) = pv[u];
        }
        float acc[per];     // (indexed by unrolled loops only, so that it stays in registers)
#pragma unroll
        for (int c = 0; c < per; ++c) acc[c] = xv[c];
        __syncthreads();
        if (s + 1 < S) fetch(s + 1);
        // (column i of the new row is a dot product along i', which is contiguous in both operands)
#pragma unroll 2
        for (int ip = 0; ip < d; ip += 4) {
            const float4 a = *(const float4*)(cur + jj * d + ip);
#pragma unroll
            for (int c = 0; c < per; ++c) {
                const float4 pq = *(const float4*)(Ps + (tx + 16 * c) * ld + ip);
                acc[c] = fmaf(a.x, pq.x, fmaf(a.y, pq.y, fmaf(a.z, pq.z, fmaf(a.w, pq.w, acc[c]))));
            }
        }
        __syncthreads();
#pragma unroll
        for (int c = 0; c < per; ++c) cur[jj * d + tx + 16 * c] = acc[c];
        __syncthreads();
    }
    if (S_final)
        for (int e = threadIdx.x; e < 16 * d; e += 256) {
            const int r = e % 16, i = e / 16;
            S_final[(bh * d + i) * d + j0 + r] = cur[r * d + i];
        }
}

// O[slot][t][j] += sum_i R[slot][t][i] start[slot][i][j]: grid (ceil(Lseg / 64), slots), 256 threads; a CTA takes 64
// tokens of one segment, thread (ty, tx) the 4 tokens 4 ty .. 4 ty + 3 and the D/16 columns j = (D/16) tx ...
template <int D>
__global__ void __launch_bounds__(256) seg_apply_kernel(const float* __restrict__ R, const float* __restrict__ start,
                                                        float* __restrict__ O, int Lseg) {
    extern __shared__ float sm[];
    float* Ss = sm;                 // [D][D]    start[i][j]
    float* Rs = sm + D * D;         // [D][64]   R[t][i] transposed: the 4 tokens of a thread are one 16-byte load
    constexpr int PER = D / 16;
    const long long slot = blockIdx.y;
    const int t0 = blockIdx.x * 64;
    const float* st = start + slot * D * D;
    for (int e = threadIdx.x; e < D * D / 4; e += 256) ((float4*)Ss)[e] = ((const float4*)st)[e];
    const float* Rg = R + (slot * Lseg + t0) * (long long)D;
    for (int e = threadIdx.x; e < 64 * D; e += 256) {
        const int t = e / D, i = e % D;
        Rs[i * 64 + t] = (t0 + t < Lseg) ? Rg[(long long)t * D + i] : 0.f;
    }
    __syncthreads();
    const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
    float acc[4][PER];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < PER; ++c) acc[a][c] = 0.f;
#pragma unroll 4
    for (int i = 0; i < D; ++i) {
        const float4 rv = *(const float4*)(Rs + i * 64 + 4 * ty);
        float b[PER];
#pragma unroll
        for (int c4 = 0; c4 < PER / 4; ++c4) {
            const float4 bv = *(const float4*)(Ss + i * D + PER * tx + 4 * c4);
            b[4 * c4] = bv.x; b[4 * c4 + 1] = bv.y; b[4 * c4 + 2] = bv.z; b[4 * c4 + 3] = bv.w;
        }
#pragma unroll
        for (int c = 0; c < PER; ++c) {
            acc[0][c] = fmaf(rv.x, b[c], acc[0][c]);
            acc[1][c] = fmaf(rv.y, b[c], acc[1][c]);
            acc[2][c] = fmaf(rv.z, b[c], acc[2][c]);
            acc[3][c] = fmaf(rv.w, b[c], acc[3][c]);
        }
    }
    float* Og = O + (slot * Lseg + t0) * (long long)D;
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int t = 4 * ty + a;
        if (t0 + t >= Lseg) continue;
        float4* row = (float4*)(Og + (long long)t * D + PER * tx);
#pragma unroll
        for (int c4 = 0; c4 < PER / 4; ++c4) {
            float4 o = row[c4];
            o.x += acc[a][4 * c4]; o.y += acc[a][4 * c4 + 1]; o.z += acc[a][4 * c4 + 2]; o.w += acc[a][4 * c4 + 3];
            row[c4] = o;
        }
    }
}

// The same product with fp16 operands on mma.sync.m16n8k16 (fp32 accumulation), for the bf16 entry points, whose
// kernels round the state and the queries to fp16 as well: grid (ceil(Lseg / 128), slots), 256 threads; warp w takes the
// 16 tokens 16 w .. 16 w + 15 and all D columns.  Both operands sit in shared memory with their contraction index
// contiguous and rows padded by 16 bytes, so that every fragment register is one conflict-free 32-bit load.
template <int D>
__global__ void __launch_bounds__(256) seg_apply_mma_kernel(const float* __restrict__ R, const float* __restrict__ start,
                                                            float* __restrict__ O, int Lseg) {
    extern __shared__ __align__(16) uint8_t smraw[];
    constexpr int LD = D + 8;                       // halves per row
    __half* As = (__half*)smraw;                    // [128 tokens][LD]   R[t][i]
    __half* Bs = As + 128 * LD;                     // [D columns j][LD]  start[i][j] transposed
    const long long slot = blockIdx.y;
    const int t0 = blockIdx.x * 128;
    const float* Rg = R + (slot * Lseg + t0) * (long long)D;
    for (int e = threadIdx.x; e < 128 * D / 4; e += 256) {
        const int t = e / (D / 4), i4 = (e % (D / 4)) * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (t0 + t < Lseg) v = *(const float4*)(Rg + (long long)t * D + i4);
        *(uint2*)(As + t * LD + i4) = make_uint2(tc::pack_h2(v.x, v.y), tc::pack_h2(v.z, v.w));
    }
    const float* st = start + slot * D * D;
    for (int e = threadIdx.x; e < D * D; e += 256) {
        const int i = e / D, j = e % D;
        Bs[j * LD + i] = __float2half_rn(st[e]);
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gid = lane >> 2, tig = lane & 3;
    float acc[D / 8][4];
#pragma unroll
    for (int nt = 0; nt < D / 8; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    const __half* arow = As + (16 * warp + gid) * LD + 2 * tig;
#pragma unroll
    for (int k0 = 0; k0 < D; k0 += 16) {
        uint32_t a[4];
        a[0] = *(const uint32_t*)(arow + k0);
        a[1] = *(const uint32_t*)(arow + 8 * LD + k0);
        a[2] = *(const uint32_t*)(arow + k0 + 8);
        a[3] = *(const uint32_t*)(arow + 8 * LD + k0 + 8);
#pragma unroll
        for (int nt = 0; nt < D / 8; ++nt) {
            const __half* brow = Bs + (8 * nt + gid) * LD + k0 + 2 * tig;
            tc::mma_16816(acc[nt], a, *(const uint32_t*)brow, *(const uint32_t*)(brow + 8));
        }
    }
    float* Og = O + (slot * Lseg + t0) * (long long)D;
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        const int t = 16 * warp + gid + 8 * hh;
        if (t0 + t >= Lseg) continue;
#pragma unroll
        for (int nt = 0; nt < D / 8; ++nt) {
            float2* o = (float2*)(Og + (long long)t * D + 8 * nt + 2 * tig);
            float2 v = *o;
            v.x += acc[nt][2 * hh];
            v.y += acc[nt][2 * hh + 1];
            *o = v;
        }
    }
}

bool seg_applicable(const pf_params* a, int S) {
    return S > 1 && a->d_k == a->d_v && a->L > 0 && a->L % S == 0;
}
pf_params seg_subproblem(const pf_params* a, int S) {
    pf_params b = *a;
    b.H = a->H * S;
    b.L = a->L / S;
    b.segments = 0;
    return b;
}
size_t seg_tail_bytes(const pf_params* a, int S) {
    return 4 * seg_array_bytes(a, S) + seg_response_bytes(a) + seg_zero_v_bytes(a);
}
size_t seg_workspace_need(const pf_params* a, int S) {
    const pf_params b = seg_subproblem(a, S);
    Problem p = as_problem(&b);
    const int impl = select_impl(p, b.impl);
    if (impl < 0) return 0;
    return align_up(workspace_need(p, impl), 256) + seg_tail_bytes(a, S);
}

int forward_segmented(const pf_params* a, int S) {
    int st = check_call(a);
    if (st != PF_OK) return st;
    if (!seg_applicable(a, S)) return PF_ERR_UNSUPPORTED;
    pf_params sub = seg_subproblem(a, S);
    const size_t need = seg_workspace_need(a, S);
    if (need == 0) return PF_ERR_UNSUPPORTED;
    cudaStream_t stream = (cudaStream_t)a->stream;
    void* ws = a->workspace;
    bool own = false;
    if (ws) {
        if (a->workspace_bytes < need || ((uintptr_t)ws & 255u)) return PF_ERR_WORKSPACE;
    } else {
        PF_CUDA_TRY(cudaMallocAsync(&ws, need, stream));
        own = true;
    }
    const size_t ab = seg_array_bytes(a, S);
    uint8_t* tail = (uint8_t*)ws + (need - seg_tail_bytes(a, S));
    SegArrays arr{(float*)tail, (float*)(tail + ab), (float*)(tail + 2 * ab), (float*)(tail + 3 * ab)};
    float* resp = (float*)(tail + 4 * ab);
    void* zero_v = (uint8_t*)resp + seg_response_bytes(a);
    sub.workspace = ws;
    sub.workspace_bytes = need - seg_tail_bytes(a, S);
    begin_call();
    // one status word for both passes: the caller's, else word 0 of the workspace (as for an unsegmented call
    // with a workspace), else the library's own; cleared once, so the first expired wait of either pass stays in it
    if (!sub.status) {
        if (a->workspace) sub.status = (int*)ws;
        else {
            st = library_status_word(&sub.status);
            if (st != PF_OK) {
                if (own) cudaFreeAsync(ws, stream);
                return st;
            }
        }
    }
    auto finish = [&](int code) {
        if (own) cudaFreeAsync(ws, stream);
        return code;
    };
    {
        cudaError_t e = cudaMemsetAsync(sub.status, 0, sizeof(int), stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(zero_v, 0, seg_zero_v_bytes(a), stream);
        if (e != cudaSuccess) return finish(record_cuda_error(e, "cudaMemsetAsync(status, zero v)"));
    }
    const int d = a->d_k;
    const long long slots = (long long)a->B * a->H * S;
    // pass A: zero start, the caller's v
    sub.S0 = nullptr;
    sub.S_final = arr.xi;
    st = forward_one(&sub, false);
    if (st != PF_OK) return finish(st);
    // pass R: identity start, v = 0; its "output" is the response of every token to the start state
    {
        const long long total = slots * d * d;
        prof_begin("seg_identity", stream);
        seg_identity_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(arr.ident, slots, d);
        prof_end(stream);
        count_launch();
    }
    sub.S0 = arr.ident;
    sub.v = zero_v;
    sub.O = resp;
    sub.S_final = arr.pb;
    st = forward_one(&sub, false);
    if (st != PF_OK) return finish(st);
    // composition of the S flows of every sequence
    {
        const int smem = (d * (d + 4) + 16 * d) * (int)sizeof(float);
        const void* fn = d == 128 ? (const void*)seg_compose_kernel<128> : (const void*)seg_compose_kernel<64>;
        cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return finish(record_cuda_error(e, "seg_compose_kernel attribute"));
        const float* s0 = a->S0;
        float* sf = a->S_final;
        int nseg = S;
        void* args[] = {(void*)&s0, (void*)&arr, (void*)&sf, (void*)&nseg};
        prof_begin("seg_compose", stream);
        e = cudaLaunchKernel(fn, dim3((unsigned)(a->B * a->H), (unsigned)(d / 16)), dim3(256), args, (size_t)smem, stream);
        prof_end(stream);
        count_launch();
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) return finish(record_cuda_error(e, "seg_compose_kernel"));
    }
    // every segment's start state applied to its responses
    {
        const int Lseg = a->L / S;
        const bool half_ops = a->in_dtype == PF_DTYPE_BF16;      // (the fp32 entry points keep fp32 throughout)
        const int smem = half_ops ? (128 + d) * (d + 8) * 2 : (d * d + 64 * d) * (int)sizeof(float);
        const void* fn = half_ops ? (d == 128 ? (const void*)seg_apply_mma_kernel<128> : (const void*)seg_apply_mma_kernel<64>)
                                  : (d == 128 ? (const void*)seg_apply_kernel<128> : (const void*)seg_apply_kernel<64>);
        cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return finish(record_cuda_error(e, "seg_apply_kernel attribute"));
        const int rows = half_ops ? 128 : 64;
        const dim3 grid((unsigned)((Lseg + rows - 1) / rows), (unsigned)slots);
        const float* rp = resp;
        const float* sp = arr.start;
        float* op = a->O;
        int lseg = Lseg;
        void* args[] = {(void*)&rp, (void*)&sp, (void*)&op, (void*)&lseg};
        prof_begin("seg_apply", stream);
        e = cudaLaunchKernel(fn, grid, dim3(256), args, (size_t)smem, stream);
        prof_end(stream);
        count_launch();
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) return finish(record_cuda_error(e, "seg_apply_kernel"));
    }
    if (own) {
        cudaError_t e = cudaFreeAsync(ws, stream);
        if (e != cudaSuccess) return record_cuda_error(e, "cudaFreeAsync");
    }
    end_call();
    return PF_OK;
}

int forward(const pf_params* a) {
    if (!a) return PF_ERR_INVALID;
    if (a->segments > 1) return forward_segmented(a, a->segments);
    return forward_one(a, true);
}

}  // namespace
}  // namespace pf

extern "C" {

int pf_deltanet_fwd_ex(const pf_params* p) { return pf::forward(p); }

int pf_deltanet_fwd(const void* q, const void* k, const void* v, const void* beta, const float* S0, int B, int H,
                    int L, int d_k, int d_v, int r, int chunk, float* O, float* S_final, void* stream) {
    pf_params a;
    memset(&a, 0, sizeof(a));
    a.q = q; a.k = k; a.v = v; a.beta = beta; a.S0 = S0;
    a.B = B; a.H = H; a.L = L; a.d_k = d_k; a.d_v = d_v; a.r = r; a.chunk = chunk;
    a.O = O; a.S_final = S_final;
    a.in_dtype = PF_DTYPE_BF16;
    a.impl = PF_IMPL_AUTO;
    a.stream = stream;
    return pf::forward(&a);
}

int pf_deltanet_fwd_f32(const float* q, const float* k, const float* v, const float* beta, const float* S0, int B,
                        int H, int L, int d_k, int d_v, int r, int chunk, float* O, float* S_final, void* stream) {
    pf_params a;
    memset(&a, 0, sizeof(a));
    a.q = q; a.k = k; a.v = v; a.beta = beta; a.S0 = S0;
    a.B = B; a.H = H; a.L = L; a.d_k = d_k; a.d_v = d_v; a.r = r; a.chunk = chunk;
    a.O = O; a.S_final = S_final;
    a.in_dtype = PF_DTYPE_F32;
    a.impl = PF_IMPL_AUTO;
    a.stream = stream;
    return pf::forward(&a);
}

size_t pf_workspace_bytes_ex(const pf_params* a) {
    if (!a || pf::check_shape(a->B, a->H, a->L, a->d_k, a->d_v, a->r, a->chunk) != PF_OK || pf::check_options(a) != PF_OK) return 0;
    if (a->mode != PF_MODE_SUM && a->mode != PF_MODE_PRODUCT) return 0;
    if (a->segments > 1) return pf::seg_applicable(a, a->segments) ? pf::seg_workspace_need(a, a->segments) : 0;
    pf::Problem p = pf::as_problem(a);
    const int sel = pf::select_impl(p, a->impl);
    if (sel < 0) return 0;
    return pf::workspace_need(p, sel);
}

size_t pf_workspace_bytes(int B, int H, int L, int d_k, int d_v, int r, int chunk, int in_dtype, int impl) {
    pf_params a;
    memset(&a, 0, sizeof(a));
    a.B = B; a.H = H; a.L = L; a.d_k = d_k; a.d_v = d_v; a.r = r; a.chunk = chunk;
    a.in_dtype = in_dtype; a.impl = impl;
    return pf_workspace_bytes_ex(&a);
}

int pf_select_impl(int B, int H, int L, int d_k, int d_v, int r, int chunk, int in_dtype, int impl) {
    const int st = pf::check_shape(B, H, L, d_k, d_v, r, chunk);
    if (st != PF_OK) return st;
    pf::Problem p = pf::as_problem(B, H, L, d_k, d_v, r, chunk, in_dtype);
    return pf::select_impl(p, impl);
}

int pf_select_chunk(int B, int H, int L, int d_k, int d_v, int r, int chunk, int in_dtype, int impl) {
    const int st = pf::check_shape(B, H, L, d_k, d_v, r, chunk);
    if (st != PF_OK) return st;
    pf::Problem p = pf::as_problem(B, H, L, d_k, d_v, r, chunk, in_dtype);
    const int sel = pf::select_impl(p, impl);
    return sel < 0 ? sel : p.chunk;
}

int pf_read_status(const void* word, void* stream) {
    int* w = (int*)word;
    if (!w) {
        const int st = pf::library_status_word(&w);
        if (st != PF_OK) return st;
    }
    int code = 0;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaMemcpy(&code, w, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return pf::record_cuda_error(e, "pf_read_status");
    pf::g_wait_code = code;
    return code == 0 ? PF_OK : PF_ERR_TIMEOUT;
}

int pf_last_wait_code(void) { return pf::g_wait_code; }

int pf_wait_selftest(int* status, int limit_us, void* stream) {
    if (limit_us < 1 || limit_us > 1000000) return PF_ERR_INVALID;
    if (status && ((uintptr_t)status & 3u)) return PF_ERR_ALIGNMENT;
    int* lib_word = nullptr;
    int st = pf::library_status_word(&lib_word);
    if (st != PF_OK) return st;
    int* w = status ? status : lib_word;
    int dev = 0, khz = 0;
    PF_CUDA_TRY(cudaGetDevice(&dev));
    PF_CUDA_TRY(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev));
    PF_CUDA_TRY(cudaMemsetAsync(w, 0, sizeof(int), (cudaStream_t)stream));
    // the flag that nothing sets: a zeroed word in device memory, allocated on first use (this is a test helper)
    static int* zero_flag[pf::kMaxDevices] = {};
    if (!zero_flag[dev]) {
        PF_CUDA_TRY(cudaMalloc((void**)&zero_flag[dev], 256));
        PF_CUDA_TRY(cudaMemset(zero_flag[dev], 0, 256));
    }
    pf::wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(w, zero_flag[dev], (long long)limit_us * (khz / 1000));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return pf::record_cuda_error(e, "wait_selftest_kernel");
    return PF_OK;
}

int pf_last_launch_count(void) { return pf::g_launches; }

void pf_profile_enable(int on) { pf::g_prof_on = on != 0; }

int pf_profile_count(void) { return pf::g_prof_n; }

int pf_profile_read(int idx, char* name, int name_cap, float* ms) {
    if (idx < 0 || idx >= pf::g_prof_n || !ms) return PF_ERR_INVALID;
    pf::ProfEntry& e = pf::g_prof[idx];
    cudaError_t err = cudaEventSynchronize(e.e1);
    if (err == cudaSuccess) err = cudaEventElapsedTime(ms, e.e0, e.e1);
    if (err != cudaSuccess) return pf::record_cuda_error(err, "pf_profile_read");
    if (name && name_cap > 0) snprintf(name, (size_t)name_cap, "%s", e.name);
    return PF_OK;
}

const char* pf_status_string(int s) {
    switch (s) {
        case PF_OK: return "ok";
        case PF_ERR_INVALID: return "invalid argument";
        case PF_ERR_UNSUPPORTED: return "unsupported shape, dtype or implementation";
        case PF_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case PF_ERR_ARCH: return "device is not compute capability 10.x";
        case PF_ERR_CUDA: return "CUDA error";
        case PF_ERR_WORKSPACE: return "workspace too small or misaligned";
        case PF_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

const char* pf_last_error_string(void) { return pf::g_err; }

int pf_version(void) { return 100; }

}  // extern "C"
