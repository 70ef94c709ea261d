// Internal interfaces of the tensor-core path (shared by pf_tc.cu and pf_tc_flow.cu).
#pragma once

#include "pf_common.cuh"

namespace pf {

struct TcGeo {
    int L, d_k, d_v, r, C, n, NC;          // NC = chunks per sequence
    int rm;                                // strict-mask group size (Problem::mask_group)
    const float* b32;                      // null, or fp32 step sizes used in place of beta (Problem::beta32)
    uint32_t e_bytes, q_bytes, xi_bytes;   // per-chunk workspace record sizes
};

struct TcWs {
    int* err;       // device status word: 0, or the code of the first bounded wait that expired
    uint8_t* E;     // [G][e_bytes]
    uint8_t* Qt;    // [G][q_bytes]
    uint8_t* Xi;    // [G][xi_bytes]
};

TcGeo tc_geo(const Problem& p);
size_t tc_ws_carve(const Problem& p, void* base, TcWs* out);

// pf_tc_flow.cu
bool tc_flow_available();
int tc_flow_launch(const Problem& p, const TcWs& ws, int dvs);

// pf_tc.cu
int tc_scan_launch(const Problem& p, const TcWs& ws);
int tc_forward_refflow(const Problem& p, void* workspace);
size_t tc_refflow_workspace_bytes(const Problem& p);

// pf_fused.cu: flow builders and state scan in one cooperative launch
bool fused_supported(const Problem& p);
bool fused_preferred(const Problem& p);     // enough SMs are left for building flows that the single launch wins
size_t fused_workspace_bytes(const Problem& p);
int fused_forward(const Problem& p, void* workspace);

// pf_simt.cu: runs the gram/solve/wu kernels only and returns where W, Uh and P were left.
int simt_prepare(const Problem& p, void* workspace, float** W, float** U, float** P);

}  // namespace pf
