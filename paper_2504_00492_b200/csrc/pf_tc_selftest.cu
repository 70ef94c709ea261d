// Diagnostic: one tcgen05 GEMM D[128 x N] = (+-A) * B^T from slab-stored fp16 operands in every
// operand-major combination the tensor-core path uses.  It checks the shared-memory descriptors,
// the swizzle function, the instruction descriptor and the TMEM read-back against a host GEMM.
#include "pf_common.cuh"
#include "pf_tc_prims.cuh"

namespace pf {
namespace {

using namespace tc;

__global__ void __launch_bounds__(128) tc_selftest_kernel(int variant, const __half* __restrict__ A,
                                                          const __half* __restrict__ B, float* __restrict__ D, int N,
                                                          int* err) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;                 // 32 KB
    uint8_t* sB = smem + 32768;         // up to 64 KB
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_base;
    const bool a_mn = variant & 1, b_mn = variant & 2, neg = variant & 4;
    const bool a_ns = variant & 8, b_ns = variant & 16;      // operand stored unswizzled (column groups of 8)
    const bool a_tm = variant & 32;                          // A (K-major) in tensor memory instead of shared memory
    const int tid = threadIdx.x, warp = tid >> 5;

    // A is given row-major as [128][128] in both cases: K-major -> A[m][k]; MN-major -> A[k][m].
    for (int e = tid; e < 128 * 128; e += 128) {
        const int row = e >> 7, col = e & 127;
        *(__half*)(sA + (a_ns ? ns_off(row, col, 128) : slab_off(row, col, 128))) = A[e];
    }
    if (!b_mn) {   // B[n][k]: N rows, 128 cols
        for (int e = tid; e < N * 128; e += 128) {
            const int row = e >> 7, col = e & 127;
            *(__half*)(sB + (b_ns ? ns_off(row, col, N) : slab_off(row, col, N))) = B[e];
        }
    } else {       // B[k][n]: 128 rows, N cols
        for (int e = tid; e < 128 * N; e += 128) {
            const int row = e / N, col = e % N;
            *(__half*)(sB + (b_ns ? ns_off(row, col, 128) : slab_off(row, col, 128))) = B[e];
        }
    }
    if (tid == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(&tmem_base, 512);
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = tmem_base;

    if (a_tm) {
        // row m of A as 64 packed words into tensor memory columns [256, 320)   (the accumulator uses [0, N))
        for (int half = 0; half < 2; ++half) {
            uint32_t w[32];
            for (int c = 0; c < 32; ++c) {
                const __half2 h2 = __halves2half2(A[tid * 128 + 64 * half + 2 * c], A[tid * 128 + 64 * half + 2 * c + 1]);
                w[c] = *reinterpret_cast<const uint32_t*>(&h2);
            }
            tmem_st32(tb + 256 + 32 * half + ((uint32_t)(warp * 32) << 16), w);
        }
        tmem_st_wait();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }
    if (tid == 0) {
        const uint32_t a_base = smem_u32(sA), b_base = smem_u32(sB);
        const int b_rows = b_mn ? 128 : N;
        if (a_tm) {
            const uint32_t idesc = make_idesc(N, false, b_mn, neg);
            for (int kk = 0; kk < 8; ++kk) {
                uint64_t bd;
                if (b_ns) bd = b_mn ? desc_ns_mnmajor(b_base + kk * ns_kstep_mnmajor(), b_rows) : desc_ns_kmajor(b_base + kk * ns_kstep_kmajor(b_rows), b_rows);
                else bd = b_mn ? desc_mnmajor(b_base + kk * 2048u, (uint32_t)b_rows * 128u) : desc_kmajor(b_base + (kk >> 2) * (uint32_t)b_rows * 128u + (kk & 3) * 32u);
                mma_f16_ta(tb, tb + 256 + 8 * kk, bd, idesc, kk > 0);
            }
        } else if (a_ns || b_ns) {
            const uint32_t idesc = make_idesc(N, a_mn, b_mn, neg);
            for (int kk = 0; kk < 8; ++kk) {
                uint64_t ad, bd;
                if (a_ns) ad = a_mn ? desc_ns_mnmajor(a_base + kk * ns_kstep_mnmajor(), 128) : desc_ns_kmajor(a_base + kk * ns_kstep_kmajor(128), 128);
                else ad = a_mn ? desc_mnmajor(a_base + kk * 2048u, 128u * 128u) : desc_kmajor(a_base + (kk >> 2) * 128u * 128u + (kk & 3) * 32u);
                if (b_ns) bd = b_mn ? desc_ns_mnmajor(b_base + kk * ns_kstep_mnmajor(), b_rows) : desc_ns_kmajor(b_base + kk * ns_kstep_kmajor(b_rows), b_rows);
                else bd = b_mn ? desc_mnmajor(b_base + kk * 2048u, (uint32_t)b_rows * 128u) : desc_kmajor(b_base + (kk >> 2) * (uint32_t)b_rows * 128u + (kk & 3) * 32u);
                mma_f16(tb, ad, bd, idesc, kk > 0);
            }
        } else if (a_mn && b_mn) gemm_issue<true, true>(tb, a_base, 128, b_base, b_rows, N, 128, neg, false);
        else if (a_mn) gemm_issue<true, false>(tb, a_base, 128, b_base, b_rows, N, 128, neg, false);
        else if (b_mn) gemm_issue<false, true>(tb, a_base, 128, b_base, b_rows, N, 128, neg, false);
        else gemm_issue<false, false>(tb, a_base, 128, b_base, b_rows, N, 128, neg, false);
        mma_commit(&bar);
    }
    const bool ok = mbar_wait(&bar, 0, err, 1);
    tc_fence_after();
    if (ok) {
        for (int c0 = 0; c0 < N; c0 += 32) {
            uint32_t r[32];
            tmem_ld32(tb + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, r);
            tmem_ld_wait();
            for (int j = 0; j < 32; ++j)
                if (c0 + j < N) D[(size_t)tid * N + c0 + j] = __uint_as_float(r[j]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tb, 512);
}

}  // namespace
}  // namespace pf

extern "C" int pf_tc_selftest(int variant, const void* A, const void* B, float* D, int N, void* stream) {
    using namespace pf;
    if (!A || !B || !D) return PF_ERR_INVALID;
    if (variant < 0 || variant > 63 || ((variant & 32) && (variant & 9))) return PF_ERR_INVALID;
    if (N < 16 || N > 256 || (N % 16)) return PF_ERR_UNSUPPORTED;
    int dev = 0, major = 0;
    PF_CUDA_TRY(cudaGetDevice(&dev));
    PF_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    if (major != 10) return PF_ERR_ARCH;
    int* err = nullptr;
    PF_CUDA_TRY(cudaMalloc(&err, sizeof(int)));
    PF_CUDA_TRY(cudaMemsetAsync(err, 0, sizeof(int), (cudaStream_t)stream));
    const int smem = 1024 + 32768 + 65536;
    PF_CUDA_TRY(cudaFuncSetAttribute(tc_selftest_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    tc_selftest_kernel<<<1, 128, smem, (cudaStream_t)stream>>>(variant, (const __half*)A, (const __half*)B, D, N, err);
    cudaError_t e = cudaGetLastError();
    int h = 0;
    if (e == cudaSuccess) e = cudaMemcpyAsync(&h, err, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    cudaFree(err);
    if (e != cudaSuccess) return record_cuda_error(e, "pf_tc_selftest");
    return h ? PF_ERR_TIMEOUT : PF_OK;
}
