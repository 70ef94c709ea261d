// Shared host/device definitions of the pf library (internal; the public ABI is include/pf.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "pf.h"

namespace pf {

// One forward problem as the launchers see it.
struct Problem {
    const void* q;
    const void* k;
    const void* v;
    const void* beta;
    const float* S0;
    int B, H, L, d_k, d_v, r, chunk;
    float* O;
    float* S_final;
    int in_dtype;
    int mode;           // PF_MODE_SUM (0) or PF_MODE_PRODUCT
    const float* beta32;    // null, or fp32 step sizes [B,H,L,r] (device) that the kernels use in place of beta
    bool auto_impl;         // the caller left the choice of kernels to the library (PF_IMPL_AUTO)
    int wu_builder;         // fp32 SIMT path: 0 = triangular inverse then W = T'K, Uh = T'V; 1 = the wavefront system of
                            // Theorem 3.3 (pf_params.wu_builder)
    int ring_depth;         // single-launch path: slots per sequence of the hand-off ring, 0 = default (pf_params.ring_depth)
    int* status;            // device word that receives the code of the first bounded wait that expires (never null
                            // when a tensor-core kernel is launched)
    cudaStream_t stream;

    __host__ __device__ int n() const { return chunk * r; }            // rows per chunk
    // Rows of the tile the tensor-core kernels give a chunk (0: none fits).  A chunk whose n is not a tile size (r = 3)
    // sits in the next larger tile: the rows past n are given beta = 0, which makes their rows of W and Uh exactly
    // zero, so whatever finite keys and values the tile holds there contribute nothing.
    __host__ __device__ int tile_rows() const {
        const int nn = n();
        if (nn == 64 || nn == 128) return nn;
        if (r == 3 && nn <= 128) return nn <= 64 ? 64 : 128;
        return 0;
    }
    // Rows m' < m of a chunk interact (the strict mask of Theorem 3.2) when they lie in different groups of this
    // many consecutive rows: r for the sum form (different tokens), 1 for the product form (any earlier row).
    __host__ __device__ int mask_group() const { return mode == PF_MODE_PRODUCT ? 1 : r; }
    __host__ __device__ int chunks_per_seq() const { return (L + chunk - 1) / chunk; }
    __host__ __device__ long long total_chunks() const { return (long long)B * H * chunks_per_seq(); }
};

// Records a CUDA error for pf_last_error_string(); returns PF_ERR_CUDA.
int record_cuda_error(cudaError_t e, const char* where);
void count_launch(int n = 1);

#define PF_CUDA_TRY(expr)                                             \
    do {                                                              \
        cudaError_t _e = (expr);                                      \
        if (_e != cudaSuccess) return ::pf::record_cuda_error(_e, #expr); \
    } while (0)

// Entry points share these (pf_api.cu): the checks made before anything is launched, and the bookkeeping of a
// top-level call (launch count, profile list).
int check_call(const pf_params* a);
void begin_call();
void end_call();

// Optional per-kernel timing (pf_profile_*): when enabled, prof_begin/prof_end bracket a launch
// with CUDA events on its stream; otherwise they do nothing.
void prof_begin(const char* name, cudaStream_t stream);
void prof_end(cudaStream_t stream);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
// room at the end of every workspace for the fp32 step sizes of PF_STEP_EXACT
inline size_t beta32_bytes(const Problem& p) { return align_up((size_t)p.B * p.H * p.L * p.r * 4, 256); }

// fp32 SIMT path (pf_simt.cu)
size_t simt_workspace_bytes(const Problem& p);
int simt_forward(const Problem& p, void* workspace);

// tcgen05 path (pf_tc.cu)
bool tc_supported(const Problem& p);
bool tc_scan_supported(const Problem& p);
size_t tc_workspace_bytes(const Problem& p);
int tc_forward(const Problem& p, void* workspace);

}  // namespace pf
