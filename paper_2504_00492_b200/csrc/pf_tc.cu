// tcgen05 tensor-core path (bf16 inputs, fp16 on-chip operands, fp32 accumulation).
//
// The paper's pipeline (Section 3): Chunk -> Parallel Compute (per-chunk flow) -> Scan.
//
//   tc_flow  (parallel over all chunks; kernel in pf_tc_flow.cu)
//       builds, for every chunk, its flow in compact form from Theorem 3.2:
//           T' = (I + Mstrict (.) diag(beta) K K^T)^{-1} diag(beta),  W = T' K,  Uh = T' V,
//           E  = -K^T W        (d_k x d_k;  I + E^T is the chunk propagator  P_chunk = I - W^T K)
//           Xi = K^T Uh        (d_k x d_v;  the chunk's integrated drive, transposed)
//       and the state-independent parts of the readout,
//           Qt = Q - P W  (stored transposed),   O_intra = P Uh  (written into O),
//           P  = (Q K^T) (.) Mincl.
//   tc_scan  (this file; one CTA per (sequence, d_v slice), serial over chunks)
//       carries the state:   S^T <- S^T + E S^T + Xi,     O = O_intra + Qt S^T,
//       i.e. S_1 = S_0 P_chunk + Uh^T K  and  O = Q S_0^T + P (Uh - W S_0^T).
//   flow_pack_ref  (this file) builds the same per-chunk flow from the fp32 SIMT intermediates; it exists
//       so that each tensor-core kernel can be checked on its own.
//
// Per-chunk workspace (g = global chunk index):
//   E  image: fp16, slab layout [d_k rows i][d_k cols i']        (K-major A operand of the scan)
//   Qt image: fp16, one slab     [d_k rows i][64 cols t]         (MN-major A operand of the scan)
//   Xi      : fp16, [d_v/DVS slices][d_k rows i][DVS cols j]     (added to the state in registers)
#include "pf_common.cuh"
#include "pf_tc.cuh"
#include "pf_tc_prims.cuh"

namespace pf {

using namespace tc;

// ======================================================================================================
// tc_scan
// ======================================================================================================
namespace {

constexpr int SCAN_STAGES = 3;
constexpr int SCAN_THREADS = 256;

// Dynamic shared memory of tc_scan (bytes from a 1024-aligned base), sized by d_k so that the d_k = 64 shapes fit two
// CTAs per SM (64 KB each; at d_k = 128 it is 176 KB):
//   SCAN_STAGES stages of [E image (d_k x d_k fp16) | Qt image (d_k x 64 fp16)], then two fp16 copies of the state
//   slice (d_k rows of 128 bytes).
struct ScanSmem {
    __host__ __device__ static int stage_bytes(int d_k) { return d_k * d_k * 2 + d_k * 128; }
    __host__ __device__ static int qt_off(int d_k) { return d_k * d_k * 2; }
    __host__ __device__ static int sb_off(int d_k) { return SCAN_STAGES * stage_bytes(d_k); }
    __host__ __device__ static int sb_bytes(int d_k) { return d_k * 128; }
    __host__ __device__ static int total(int d_k) { return sb_off(d_k) + 2 * sb_bytes(d_k); }
};

template <int DVS>
__global__ void __launch_bounds__(SCAN_THREADS, 1)
tc_scan(TcGeo g, TcWs ws, const float* __restrict__ S0, float* __restrict__ O, float* __restrict__ S_final) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t full_bar[SCAN_STAGES], empty_bar[SCAN_STAGES];
    __shared__ uint64_t s_ready[2], o_done[2], o_free[2], delta_done;
    __shared__ uint32_t tmem_base_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slices = g.d_v / DVS;
    const long long seq = blockIdx.x / slices;
    const int slice = (int)(blockIdx.x % slices);
    const int j0 = slice * DVS;
    const int d_k = g.d_k, d_v = g.d_v, NC = g.NC;
    constexpr uint32_t TM_COLS = (3 * DVS <= 128) ? 128 : 256;

    if (tid == 0) {
        for (int s = 0; s < SCAN_STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&s_ready[b], 128); mbar_init(&o_done[b], 1); mbar_init(&o_free[b], 64); }
        mbar_init(&delta_done, 1);
        mbar_fence_init();
    }
    if (warp == 7) tmem_alloc(&tmem_base_s, TM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = tmem_base_s;
    const uint32_t t_delta = tb, t_o0 = tb + DVS;     // O buffers at tb + DVS and tb + 2*DVS
    const uint32_t e_bytes = (uint32_t)d_k * d_k * 2, q_bytes = (uint32_t)d_k * 128;
    int* err = ws.err;

    if (warp < 4) {
        // ---------------- chain: the state lives here, row i of S^T per thread ----------------------
        const int i = tid;
        const bool active = i < d_k;
        float S[DVS];
#pragma unroll
        for (int j = 0; j < DVS; ++j) S[j] = (active && S0) ? S0[(seq * d_k + i) * (long long)d_v + j0 + j] : 0.f;
        uint4 xi_next[DVS / 8];
        const uint8_t* xi_base = ws.Xi + (size_t)seq * NC * g.xi_bytes + (size_t)slice * d_k * DVS * 2 + (size_t)i * DVS * 2;
        auto load_xi = [&](int c) {
#pragma unroll
            for (int qd = 0; qd < DVS / 8; ++qd)
                xi_next[qd] = active ? __ldg((const uint4*)(xi_base + (size_t)c * g.xi_bytes) + qd) : make_uint4(0, 0, 0, 0);
        };
        if (NC > 0) load_xi(0);
        bool ok = true;
        for (int c = 0; c < NC && ok; ++c) {
            uint8_t* sb = smem + ScanSmem::sb_off(d_k) + (c & 1) * ScanSmem::sb_bytes(d_k);
            // fp16 copy of the state as the B operand of both MMAs: row i, DVS columns (the buffer has d_k rows)
#pragma unroll
            for (int qd = 0; active && qd < DVS / 8; ++qd) {
                uint4 pk;
                pk.x = pack_h2(S[8 * qd + 0], S[8 * qd + 1]);
                pk.y = pack_h2(S[8 * qd + 2], S[8 * qd + 3]);
                pk.z = pack_h2(S[8 * qd + 4], S[8 * qd + 5]);
                pk.w = pack_h2(S[8 * qd + 6], S[8 * qd + 7]);
                *(uint4*)(sb + i * 128 + ((qd ^ (i & 7)) << 4)) = pk;
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(&s_ready[c & 1]);
            uint4 xi[DVS / 8];
#pragma unroll
            for (int qd = 0; qd < DVS / 8; ++qd) xi[qd] = xi_next[qd];
            if (c + 1 < NC) load_xi(c + 1);
            ok = mbar_wait(&delta_done, c & 1, err, 11);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int c0 = 0; c0 < DVS; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(t_delta + ((uint32_t)(warp * 32) << 16) + c0, r);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const uint32_t w = ((const uint32_t*)&xi[(c0 + j) / 8])[((c0 + j) % 8) / 2];
                    const float2 x = __half22float2(*reinterpret_cast<const __half2*>(&w));
                    S[c0 + j] += __uint_as_float(r[j]) + x.x;
                    S[c0 + j + 1] += __uint_as_float(r[j + 1]) + x.y;
                }
            }
        }
        if (ok && active && S_final)
#pragma unroll
            for (int j = 0; j < DVS; ++j) S_final[(seq * d_k + i) * (long long)d_v + j0 + j] = S[j];
    } else if (warp < 6) {
        // ---------------- output epilogue: O[t, j0..] = O_intra + Qt S^T ---------------------------
        const int t = (warp - 4) * 32 + lane;
        for (int c = 0; c < NC; ++c) {
            const int b = c & 1;
            if (!mbar_wait(&o_done[b], (c >> 1) & 1, err, 12)) break;
            tc_fence_after();
            const int Cv = min(g.C, g.L - c * g.C);
            float* orow = O + (seq * g.L + (long long)c * g.C + t) * d_v + j0;
#pragma unroll
            for (int c0 = 0; c0 < DVS; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(t_o0 + b * DVS + ((uint32_t)((warp - 4) * 32) << 16) + c0, r);
                tmem_ld_wait();
                if (t < Cv) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        float4 o = *(const float4*)(orow + c0 + j);
                        o.x += __uint_as_float(r[j]);
                        o.y += __uint_as_float(r[j + 1]);
                        o.z += __uint_as_float(r[j + 2]);
                        o.w += __uint_as_float(r[j + 3]);
                        *(float4*)(orow + c0 + j) = o;
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(&o_free[b]);
        }
    } else if (warp == 6) {
        // ---------------- producer: bulk copies of the chunk's E and Qt images ----------------------
        // (the whole warp walks the loop so that it stays converged; lane 0 does the work)
        for (int c = 0; c < NC; ++c) {
            int ok = 1;
            if (lane == 0) {
                const int s = c % SCAN_STAGES;
                if (c >= SCAN_STAGES) ok = mbar_wait(&empty_bar[s], ((c / SCAN_STAGES) - 1) & 1, err, 13);
                if (ok) {
                    const size_t gc = (size_t)seq * NC + c;
                    uint8_t* st = smem + s * ScanSmem::stage_bytes(d_k);
                    mbar_expect_tx(&full_bar[s], e_bytes + q_bytes);
                    bulk_load(st, ws.E + gc * g.e_bytes, e_bytes, &full_bar[s]);
                    bulk_load(st + ScanSmem::qt_off(d_k), ws.Qt + gc * g.q_bytes, q_bytes, &full_bar[s]);
                }
            }
            if (!__shfl_sync(0xffffffffu, ok, 0)) break;
        }
    } else {
        // ---------------- MMA issue (lane 0 of warp 7) -------------------------------------------------
        for (int c = 0; c < NC; ++c) {
            int ok = 1;
            if (lane == 0) {
                const int s = c % SCAN_STAGES, b = c & 1;
                ok = mbar_wait(&full_bar[s], (c / SCAN_STAGES) & 1, err, 14) && mbar_wait(&s_ready[b], (c >> 1) & 1, err, 15);
                if (ok) {
                    tc_fence_after();
                    const uint32_t e_base = smem_u32(smem + s * ScanSmem::stage_bytes(d_k));
                    const uint32_t q_base = e_base + ScanSmem::qt_off(d_k);
                    const uint32_t s_base = smem_u32(smem + ScanSmem::sb_off(d_k) + b * ScanSmem::sb_bytes(d_k));
                    // Delta^T[i, j] = sum_i' E[i, i'] S[j, i']
                    gemm_issue<false, true>(t_delta, e_base, d_k, s_base, 128, DVS, d_k, false, false);
                    mma_commit(&delta_done);
                    if (c >= 2) ok = mbar_wait(&o_free[b], ((c >> 1) - 1) & 1, err, 16);
                    if (ok) {
                        tc_fence_after();
                        // O[t, j] = sum_i Qt^T[i, t] S[j, i]
                        gemm_issue<true, true>(t_o0 + b * DVS, q_base, d_k, s_base, 128, DVS, d_k, false, false);
                        mma_commit(&o_done[b]);
                        mma_commit(&empty_bar[s]);
                    }
                }
            }
            if (!__shfl_sync(0xffffffffu, ok, 0)) break;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 7) tmem_dealloc(tb, TM_COLS);
}

// ======================================================================================================
// flow_pack_ref: per-chunk flow from the fp32 SIMT intermediates (W, Uh, P), one CTA per chunk.
// Plain loops; used to test tc_scan in isolation and as the reference for tc_flow's outputs.
// ======================================================================================================
template <class Tin>
__device__ __forceinline__ float ldin(const Tin* p);
template <>
__device__ __forceinline__ float ldin<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

__global__ void __launch_bounds__(256)
flow_pack_ref(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k, const float* __restrict__ Wf,
              const float* __restrict__ Uf, const float* __restrict__ Pf, TcGeo g, TcWs ws, float* __restrict__ O, int dvs) {
    const long long gc = blockIdx.x;
    const long long seq = gc / g.NC;
    const int c = (int)(gc % g.NC);
    const int t0 = c * g.C;
    const int Cv = min(g.C, g.L - t0);
    const int nv = Cv * g.r;
    const int n = g.n, d_k = g.d_k, d_v = g.d_v;
    const __nv_bfloat16* Kc = k + ((seq * g.L + t0) * g.r) * (long long)d_k;
    const __nv_bfloat16* Qc = q + (seq * g.L + t0) * (long long)d_k;
    const float* W = Wf + gc * (long long)n * d_k;
    const float* U = Uf + gc * (long long)n * d_v;
    const float* P = Pf + gc * (long long)g.C * n;
    uint8_t* Eo = ws.E + (size_t)gc * g.e_bytes;
    uint8_t* Qo = ws.Qt + (size_t)gc * g.q_bytes;
    uint8_t* Xo = ws.Xi + (size_t)gc * g.xi_bytes;

    for (int e = threadIdx.x; e < d_k * d_k; e += blockDim.x) {       // E[i][i'] = -sum_m K[m][i] W[m][i']
        const int i = e / d_k, ip = e % d_k;
        float acc = 0.f;
        for (int m = 0; m < nv; ++m) acc += ldin(Kc + (long long)m * d_k + i) * W[(long long)m * d_k + ip];
        *(__half*)(Eo + slab_off(i, ip, d_k)) = __float2half_rn(-acc);
    }
    for (int e = threadIdx.x; e < d_k * d_v; e += blockDim.x) {       // Xi[i][j] = sum_m K[m][i] Uh[m][j]
        const int i = e / d_v, j = e % d_v;
        float acc = 0.f;
        for (int m = 0; m < nv; ++m) acc += ldin(Kc + (long long)m * d_k + i) * U[(long long)m * d_v + j];
        *(__half*)(Xo + ((size_t)(j / dvs) * d_k * dvs + (size_t)i * dvs + (j % dvs)) * 2) = __float2half_rn(acc);
    }
    for (int e = threadIdx.x; e < d_k * 64; e += blockDim.x) {        // Qt^T[i][t] = Q[t][i] - sum_m W[m][i] P[t][m]
        const int i = e / 64, t = e % 64;
        float acc = 0.f;
        if (t < Cv) {
            acc = ldin(Qc + (long long)t * d_k + i);
            for (int m = 0; m < nv; ++m) acc -= W[(long long)m * d_k + i] * P[(long long)t * n + m];
        }
        *(__half*)(Qo + slab_off(i, t, d_k)) = __float2half_rn(acc);
    }
    for (int e = threadIdx.x; e < Cv * d_v; e += blockDim.x) {        // O_intra[t][j] = sum_m P[t][m] Uh[m][j]
        const int t = e / d_v, j = e % d_v;
        float acc = 0.f;
        for (int m = 0; m < nv; ++m) acc += P[(long long)t * n + m] * U[(long long)m * d_v + j];
        O[(seq * g.L + t0 + t) * (long long)d_v + j] = acc;
    }
}

int pick_dvs(const Problem& p) {
    // narrower slices = more CTAs and a shorter serial step; 32 is the narrowest the layout supports
    (void)p;
    return 32;
}

}  // namespace

TcGeo tc_geo(const Problem& p) {
    TcGeo g{};
    g.L = p.L; g.d_k = p.d_k; g.d_v = p.d_v; g.r = p.r; g.C = p.chunk; g.n = p.n(); g.NC = p.chunks_per_seq(); g.rm = p.mask_group(); g.b32 = p.beta32;
    g.e_bytes = (uint32_t)p.d_k * p.d_k * 2;
    g.q_bytes = (uint32_t)p.d_k * 128;
    g.xi_bytes = (uint32_t)p.d_k * p.d_v * 2;
    return g;
}

size_t tc_ws_carve(const Problem& p, void* base, TcWs* out) {
    const TcGeo g = tc_geo(p);
    const size_t G = (size_t)p.total_chunks();
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes, 1024); return o; };
    const size_t o_err = take(1024);
    const size_t o_e = take(G * g.e_bytes);
    const size_t o_q = take(G * g.q_bytes);
    const size_t o_x = take(G * g.xi_bytes);
    if (out && base) {
        uint8_t* b = (uint8_t*)base;
        out->err = p.status;     // (the first 1 KB of the workspace is reserved: its word 0 is the status word of callers that pass a workspace and no status pointer)
        (void)o_err;
        out->E = b + o_e;
        out->Qt = b + o_q;
        out->Xi = b + o_x;
    }
    return off;
}

bool tc_scan_supported(const Problem& p) { return p.in_dtype == PF_DTYPE_BF16 && p.chunk <= 64; }

bool tc_supported(const Problem& p) {
    if (!tc_scan_supported(p)) return false;
    if (p.tile_rows() == 0) return false;
    return tc_flow_available();
}

size_t tc_workspace_bytes(const Problem& p) { return tc_ws_carve(p, nullptr, nullptr) + 1024; }

int tc_scan_launch(const Problem& p, const TcWs& ws) {
    const TcGeo g = tc_geo(p);
    const int dvs = pick_dvs(p);
    const long long nseq = (long long)p.B * p.H;
    const int smem = ScanSmem::total(p.d_k) + 1024;
    const unsigned grid = (unsigned)(nseq * (p.d_v / dvs));
    prof_begin("tc_scan", p.stream);
    if (dvs == 32) {
        PF_CUDA_TRY(cudaFuncSetAttribute(tc_scan<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        tc_scan<32><<<grid, SCAN_THREADS, smem, p.stream>>>(g, ws, p.S0, p.O, p.S_final);
    } else {
        PF_CUDA_TRY(cudaFuncSetAttribute(tc_scan<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        tc_scan<64><<<grid, SCAN_THREADS, smem, p.stream>>>(g, ws, p.S0, p.O, p.S_final);
    }
    prof_end(p.stream);
    PF_CUDA_TRY(cudaGetLastError());
    count_launch(1);
    return PF_OK;
}

int tc_scan_dvs(const Problem& p) { return pick_dvs(p); }

// Debug pipeline: SIMT gram/solve/wu -> flow_pack_ref -> tc_scan.  `workspace` must hold the tc
// workspace followed by the SIMT workspace.
int tc_forward_refflow(const Problem& p, void* workspace) {
    TcWs ws;
    const size_t tc_bytes = align_up(tc_ws_carve(p, workspace, &ws), 1024);
    void* simt_ws = (uint8_t*)workspace + tc_bytes;
    float *Wf, *Uf, *Pf;
    int st = simt_prepare(p, simt_ws, &Wf, &Uf, &Pf);
    if (st != PF_OK) return st;
    const TcGeo g = tc_geo(p);
    const long long G = p.total_chunks();
    if (G > 0) {
        prof_begin("flow_pack_ref", p.stream);
        flow_pack_ref<<<(unsigned)G, 256, 0, p.stream>>>((const __nv_bfloat16*)p.q, (const __nv_bfloat16*)p.k, Wf, Uf, Pf, g,
                                                          ws, p.O, pick_dvs(p));
        prof_end(p.stream);
        PF_CUDA_TRY(cudaGetLastError());
        count_launch(1);
    }
    return tc_scan_launch(p, ws);
}

size_t tc_refflow_workspace_bytes(const Problem& p) {
    return align_up(tc_ws_carve(p, nullptr, nullptr), 1024) + simt_workspace_bytes(p) + 1024;
}

int tc_forward(const Problem& p, void* workspace) {
    TcWs ws;
    tc_ws_carve(p, workspace, &ws);
    int st = tc_flow_launch(p, ws, pick_dvs(p));
    if (st != PF_OK) return st;
    return tc_scan_launch(p, ws);
}

}  // namespace pf
