// tc_flow: the per-chunk flow builder on tcgen05 (the "Parallel Compute" step of Section 3).
//
// One persistent CTA per SM walks over chunks.  For a chunk with rows m = t*r + j (n = C*r rows):
//
//   load     K [n x d_k], Q [C x d_k], V [n x d_v] by TMA (bf16, 128B swizzle), convert to fp16 in place
//   MMA1     [G | P0^T] = K [K;Q]^T                               (tcgen05, accumulators in TMEM)
//   epi1     A = Mstrict (.) diag(beta) G  -> fp16 into the X buffer (+ fp32 copies of the 16x16 diagonal
//            blocks);  P^T = P0^T (.) Mincl -> fp16
//   solve    X = (I + A)^{-1}: 16x16 diagonal blocks by forward substitution in registers (fp32), then
//            log2(n/16) levels of  X_hi,lo = -X_hi,hi A_hi,lo X_lo,lo  with warp-level mma.sync
//            (the block-triangular inverse of the Proposition after Theorem 3.2, by recursive doubling);
//            T' = X diag(beta)
//   MMA2     W = T' K,  Uh = T' V                                  (Theorem 3.2)
//   epi2     W, Uh -> fp16 operands
//   MMA3     E = -K^T W,  Xi = K^T Uh                               (the chunk's flow, transposed)
//   MMA4     Qt^T = Q^T - W^T P^T,   O_intra^T = Uh^T P^T
//   epi3     E, Xi, Qt^T -> workspace (fp16, in the layouts tc_scan consumes);  O_intra -> O (fp32)
//
// All MMAs run with M = 128; operands with fewer rows read past their tile inside this CTA's shared
// memory, which only produces accumulator lanes that are never read.
#include "pf_common.cuh"
#include "pf_tc.cuh"
#include "pf_tc_prims.cuh"

namespace pf {

using namespace tc;

namespace {

constexpr int FLOW_THREADS = 128;

template <int N, int DK, int DV>
struct FlowSmem {
    static constexpr int kq_rows = N + 64;                        // K rows then Q rows in every d-half slab
    static constexpr int kq_bytes = (DK / 64) * kq_rows * 128;
    static constexpr int v_bytes = (DV / 64) * N * 128;           // V, later Uh
    static constexpr int x_bytes = (N / 64) * N * 128;            // A -> X -> T'
    static constexpr int w_bytes = (DK / 64) * N * 128;
    static constexpr int pt_bytes = N * 128;                      // P^T: [n rows m][64 cols t]
    static constexpr int id_bytes = 64 * 128;                     // 64 x 64 identity
    // Two regions are borrowed instead of owned: the identity lives in the X region, which is dead once the W / Uh
    // product has read X (it is rewritten there for every chunk), and the fp32 diagonal blocks of the inverse live
    // in the W region, which is written only after the inverse is complete.  With d_k = d_v = 64 that brings a CTA
    // under half an SM's shared memory, and with the 256 tensor-memory columns those shapes need, two CTAs share an SM.
    static constexpr bool two_per_sm = (DK + DV <= 128) && (N + 64 <= 256);
    static constexpr int tmem_cols = two_per_sm ? 256 : 512;
    static constexpr int kq_off = 0;
    static constexpr int v_off = kq_off + kq_bytes;
    static constexpr int x_off = v_off + v_bytes;
    static constexpr int w_off = x_off + x_bytes;
    static constexpr int pt_off = w_off + w_bytes;
    static constexpr int id_off = x_off;                          // (borrowed, see above)
    static constexpr int diag_off = w_off;                        // fp32 [N/16][16][16] (borrowed)
    static constexpr int diag_bytes = (N / 16) * 256 * 4;
    static_assert(id_bytes <= x_bytes && diag_bytes <= w_bytes, "borrowed regions fit");
    static constexpr int beta_off = pt_off + pt_bytes;            // fp16 beta[N] (column scaling)
    static constexpr int total = beta_off + 1024;
};

struct FlowMaps {
    CUtensorMap q, k, v;
};

// Brings a tile into the L2 ahead of the load that will land it in shared memory (no completion to wait for).
__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap* map, int x, int y, int z) {
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(map), "r"(x), "r"(y), "r"(z) : "memory");
}


template <int N, int DK, int DV>
__global__ void __launch_bounds__(FLOW_THREADS, (FlowSmem<N, DK, DV>::two_per_sm ? 2 : 1))
tc_flow(const __grid_constant__ FlowMaps maps, TcGeo g, TcWs ws, const __nv_bfloat16* __restrict__ beta,
        float* __restrict__ O, long long G, int dvs) {
    using SM = FlowSmem<N, DK, DV>;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t tma_bar, mma_bar;
    __shared__ uint32_t tmem_base_s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int r = g.r, C = g.C;
    const int dvs_shift = (dvs == 64) ? 6 : 5;
    int* err = ws.err;

    uint8_t* sKQ = smem + SM::kq_off;
    uint8_t* sV = smem + SM::v_off;
    uint8_t* sX = smem + SM::x_off;
    uint8_t* sW = smem + SM::w_off;
    uint8_t* sPT = smem + SM::pt_off;
    uint8_t* sI = smem + SM::id_off;
    float* sDiag = (float*)(smem + SM::diag_off);
    __half* sBeta = (__half*)(smem + SM::beta_off);
    const uint32_t kq_b = smem_u32(sKQ), v_b = smem_u32(sV), x_b = smem_u32(sX), w_b = smem_u32(sW),
                   pt_b = smem_u32(sPT), id_b = smem_u32(sI);

    if (tid == 0) {
        mbar_init(&tma_bar, 1);
        mbar_init(&mma_bar, 1);
        mbar_fence_init();
        prefetch_tmap(&maps.q);
        prefetch_tmap(&maps.k);
        prefetch_tmap(&maps.v);
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(&tmem_base_s, SM::tmem_cols);
    // (the Q rows of the KQ slabs start defined: stale rows are read)
    for (int e = tid; e < SM::kq_bytes / 16; e += FLOW_THREADS) ((uint4*)sKQ)[e] = make_uint4(0, 0, 0, 0);
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = tmem_base_s;
    // [G | P0^T] (N + 64 columns), then [W | Uh], then [E | Xi] next to [Qt^T | O_intra^T]; each is drained before the
    // next product that reuses its columns is issued
    const uint32_t t_d1 = tb, t_d2 = SM::two_per_sm ? tb : tb + 256, t_d3 = SM::two_per_sm ? tb + 128 : tb,
                   t_d4 = SM::two_per_sm ? tb : tb + 256;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    uint32_t tma_phase = 0, mma_phase = 0;
    bool ok = true;
    for (long long gc = blockIdx.x; gc < G && ok; gc += gridDim.x) {
        const long long seq = gc / g.NC;
        const int c = (int)(gc % g.NC);
        const int t0 = c * C;
        const int Cv = min(C, g.L - t0);
        const int nv = Cv * r;

        // ---- load ---------------------------------------------------------------------------------
        if (tid == 0) {
            constexpr uint32_t bytes_k = N * 128, bytes_v = N * 128;
            const uint32_t bytes_q = (uint32_t)C * 128;
            mbar_expect_tx(&tma_bar, (DK / 64) * (bytes_k + bytes_q) + (DV / 64) * bytes_v);
            for (int h = 0; h < DK / 64; ++h) {
                tma_load_3d(sKQ + h * SM::kq_rows * 128, &maps.k, 64 * h, t0 * r, (int)seq, &tma_bar);
                tma_load_3d(sKQ + h * SM::kq_rows * 128 + N * 128, &maps.q, 64 * h, t0, (int)seq, &tma_bar);
            }
            for (int h = 0; h < DV / 64; ++h) tma_load_3d(sV + h * N * 128, &maps.v, 64 * h, t0 * r, (int)seq, &tma_bar);
            // the tiles of this CTA's next chunk into the L2: their load proper is issued only when this chunk is done
            // with the buffers, and then finds them there
            const long long gn = gc + gridDim.x;
            if (gn < G) {
                const int sn = (int)(gn / g.NC), tn = (int)(gn % g.NC) * C;
                for (int h = 0; h < DK / 64; ++h) {
                    tma_prefetch_3d(&maps.k, 64 * h, tn * r, sn);
                    tma_prefetch_3d(&maps.q, 64 * h, tn, sn);
                }
                for (int h = 0; h < DV / 64; ++h) tma_prefetch_3d(&maps.v, 64 * h, tn * r, sn);
            }
        }
        const int m = tid;
        float beta_m = 0.f;
        if (m < nv) {
            const long long bi = (seq * g.L + t0) * (long long)r + m;
            beta_m = g.b32 ? g.b32[bi] : __bfloat162float(beta[bi]);
        }
        if (m < N) sBeta[m] = __float2half_rn(beta_m);
        ok = mbar_wait(&tma_bar, tma_phase, err, 21);
        tma_phase ^= 1;
        if (!ok) break;
        // ---- bf16 -> fp16 in place (elementwise, so the swizzled layout is untouched) --------------------
        {
            constexpr int chunks = (SM::kq_bytes + SM::v_bytes) / 16;   // the two regions are contiguous
            uint4* p = (uint4*)sKQ;
            for (int e = tid; e < chunks; e += FLOW_THREADS) {
                uint4 val = p[e];
                uint32_t* w = (uint32_t*)&val;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
                    w[i] = pack_h2(lo, hi);
                }
                p[e] = val;
            }
        }
        fence_async_smem();
        __syncthreads();
        // ---- MMA1: [G | P0^T] = K [K;Q]^T ---------------------------------------------------------
        if (tid == 0) {
            tc_fence_after();
            gemm_issue<false, false>(t_d1, kq_b, SM::kq_rows, kq_b, SM::kq_rows, N + 64, DK, false, false);
            mma_commit(&mma_bar);
        }
        ok = mbar_wait(&mma_bar, mma_phase, err, 22);
        mma_phase ^= 1;
        if (!ok) break;
        tc_fence_after();
        // ---- epilogue 1: A -> X buffer (fp16) + fp32 diagonal blocks; P^T -> fp16 -------------------------
        {
            const int tokm = m / r;
            const int row_lim = (m / g.rm) * g.rm;   // rows m' < row_lim: earlier tokens (sum form) / earlier rows (product form)
#pragma unroll
            for (int c0 = 0; c0 < N; c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(t_d1 + lane_base + c0, rr);
                tmem_ld_wait();
                if (m < N) {
#pragma unroll
                    for (int j8 = 0; j8 < 32; j8 += 8) {
                        float a[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const int mp = c0 + j8 + j;
                            a[j] = (mp < row_lim) ? beta_m * __uint_as_float(rr[j8 + j]) : 0.f;
                        }
                        uint4 pk = make_uint4(pack_h2(a[0], a[1]), pack_h2(a[2], a[3]), pack_h2(a[4], a[5]), pack_h2(a[6], a[7]));
                        *(uint4*)(sX + slab_off(m, c0 + j8, N)) = pk;
                        if (((c0 + j8) >> 4) == (m >> 4)) {   // inside this row's 16x16 diagonal block
                            float* dst = sDiag + (m >> 4) * 256 + (m & 15) * 16 + ((c0 + j8) & 15);
#pragma unroll
                            for (int j = 0; j < 8; ++j) dst[j] = a[j];
                        }
                    }
                }
            }
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(t_d1 + lane_base + N + c0, rr);
                tmem_ld_wait();
                if (m < N) {
#pragma unroll
                    for (int j8 = 0; j8 < 32; j8 += 8) {
                        float a[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const int t = c0 + j8 + j;
                            a[j] = (tokm <= t && t < Cv && m < nv) ? __uint_as_float(rr[j8 + j]) : 0.f;
                        }
                        uint4 pk = make_uint4(pack_h2(a[0], a[1]), pack_h2(a[2], a[3]), pack_h2(a[4], a[5]), pack_h2(a[6], a[7]));
                        *(uint4*)(sPT + m * 128 + ((((c0 + j8) >> 3) ^ (m & 7)) << 4)) = pk;
                    }
                }
            }
        }
        tc_fence_before();
        __syncthreads();
        // ---- solve: 16x16 diagonal blocks by forward substitution (thread = one column of one block) ------
        if (tid < N) {
            const int b = tid >> 4, cc = tid & 15;
            const float* Ab = sDiag + b * 256;
            float x[16];
#pragma unroll
            for (int mm = 0; mm < 16; ++mm) {
                float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
                for (int mp = 0; mp < mm; ++mp) {
                    if (mp & 1) acc1 = fmaf(Ab[mm * 16 + mp], x[mp], acc1);
                    else acc0 = fmaf(Ab[mm * 16 + mp], x[mp], acc0);
                }
                x[mm] = ((mm == cc) ? 1.f : 0.f) - (acc0 + acc1);
            }
#pragma unroll
            for (int mm = 0; mm < 16; ++mm)
                *(__half*)(sX + slab_off(16 * b + mm, 16 * b + cc, N)) = __float2half_rn(x[mm]);
        }
        __syncthreads();
        merge_level<N, 16, 0>(x_b, sX, warp, lane);
        merge_level<N, 32, 0>(x_b, sX, warp, lane);
        if (N == 128) merge_level<N, 64, 0>(x_b, sX, warp, lane);
        // ---- T' = X diag(beta): the row owner scales its row by the column betas -----------------------------
        if (m < N) {
#pragma unroll
            for (int ch = 0; ch < N / 8; ++ch) {
                uint4* px = (uint4*)(sX + slab_off(m, 8 * ch, N));
                uint4 xv = *px;
                const uint4 bv = *(const uint4*)(sBeta + 8 * ch);
                __half2* xh = (__half2*)&xv;
                const __half2* bh = (const __half2*)&bv;
#pragma unroll
                for (int i = 0; i < 4; ++i) xh[i] = __hmul2(xh[i], bh[i]);
                *px = xv;
            }
        }
        fence_async_smem();
        __syncthreads();
        // ---- MMA2: W = T' K,  Uh = T' V -------------------------------------------------------------
        if (tid == 0) {
            tc_fence_after();
            gemm_issue<false, true>(t_d2, x_b, N, kq_b, SM::kq_rows, DK, N, false, false);
            gemm_issue<false, true>(t_d2 + DK, x_b, N, v_b, N, DV, N, false, false);
            mma_commit(&mma_bar);
        }
        ok = mbar_wait(&mma_bar, mma_phase, err, 23);
        mma_phase ^= 1;
        if (!ok) break;
        tc_fence_after();
        // 64 x 64 identity, fp16, slab layout, into the (now dead) X region: B operand of the "+ Q^T" product below
        for (int e = tid; e < 64 * 8; e += FLOW_THREADS) {
            const int row = e >> 3, ch = e & 7;
            uint4 val = make_uint4(0, 0, 0, 0);
            if ((row >> 3) == ch) ((uint16_t*)&val)[row & 7] = 0x3C00;   // 1.0 in fp16
            *(uint4*)(sI + row * 128 + ((ch ^ (row & 7)) << 4)) = val;
        }
        // ---- epilogue 2: W and Uh as fp16 operands (Uh overwrites V) ----------------------------------
#pragma unroll 1
        for (int c0 = 0; c0 < DK + DV; c0 += 32) {
            uint32_t rr[32];
            tmem_ld32(t_d2 + lane_base + c0, rr);
            tmem_ld_wait();
            if (m < N) {
                uint8_t* dst = (c0 < DK) ? sW : sV;
                const int col0 = (c0 < DK) ? c0 : c0 - DK;
#pragma unroll
                for (int j8 = 0; j8 < 32; j8 += 8) {
                    uint4 pk = make_uint4(pack_h2(__uint_as_float(rr[j8]), __uint_as_float(rr[j8 + 1])),
                                          pack_h2(__uint_as_float(rr[j8 + 2]), __uint_as_float(rr[j8 + 3])),
                                          pack_h2(__uint_as_float(rr[j8 + 4]), __uint_as_float(rr[j8 + 5])),
                                          pack_h2(__uint_as_float(rr[j8 + 6]), __uint_as_float(rr[j8 + 7])));
                    *(uint4*)(dst + slab_off(m, col0 + j8, N)) = pk;
                }
            }
        }
        fence_async_smem();
        tc_fence_before();
        __syncthreads();
        // ---- MMA3: E = -K^T W, Xi = K^T Uh;  MMA4: Qt^T = Q^T - W^T P^T, O_intra^T = Uh^T P^T ---------------
        if (tid == 0) {
            tc_fence_after();
            gemm_issue<true, true>(t_d3, kq_b, SM::kq_rows, w_b, N, DK, N, true, false);
            gemm_issue<true, true>(t_d3 + DK, kq_b, SM::kq_rows, v_b, N, DV, N, false, false);
            gemm_issue<true, true>(t_d4, w_b, N, pt_b, N, 64, N, true, false);
            gemm_issue<true, true>(t_d4, kq_b + N * 128, SM::kq_rows, id_b, 64, 64, 64, false, true);
            gemm_issue<true, true>(t_d4 + 64, v_b, N, pt_b, N, 64, N, false, false);
            mma_commit(&mma_bar);
        }
        ok = mbar_wait(&mma_bar, mma_phase, err, 24);
        mma_phase ^= 1;
        if (!ok) break;
        tc_fence_after();
        // ---- epilogue 3: the chunk's flow -> workspace; O_intra -> O -----------------------------------
        {
            const int i = tid;   // accumulator lane: a d_k index (E, Xi, Qt^T) or a d_v index (O_intra^T)
            uint8_t* Eo = ws.E + (size_t)gc * g.e_bytes;
            uint8_t* Qo = ws.Qt + (size_t)gc * g.q_bytes;
            uint8_t* Xo = ws.Xi + (size_t)gc * g.xi_bytes;
#pragma unroll 1
            for (int c0 = 0; c0 < DK + DV; c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(t_d3 + lane_base + c0, rr);
                tmem_ld_wait();
                if (i < DK) {
#pragma unroll
                    for (int j8 = 0; j8 < 32; j8 += 8) {
                        uint4 pk = make_uint4(pack_h2(__uint_as_float(rr[j8]), __uint_as_float(rr[j8 + 1])),
                                              pack_h2(__uint_as_float(rr[j8 + 2]), __uint_as_float(rr[j8 + 3])),
                                              pack_h2(__uint_as_float(rr[j8 + 4]), __uint_as_float(rr[j8 + 5])),
                                              pack_h2(__uint_as_float(rr[j8 + 6]), __uint_as_float(rr[j8 + 7])));
                        if (c0 < DK) {
                            *(uint4*)(Eo + slab_off(i, c0 + j8, DK)) = pk;
                        } else {
                            const int j = c0 - DK + j8;
                            const int sl = j >> dvs_shift, jj = j & (dvs - 1);
                            *(uint4*)(Xo + ((size_t)sl * DK * dvs + (size_t)i * dvs + jj) * 2) = pk;
                        }
                    }
                }
            }
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(t_d4 + lane_base + c0, rr);
                tmem_ld_wait();
                if (i < DK) {
#pragma unroll
                    for (int j8 = 0; j8 < 32; j8 += 8) {
                        uint4 pk = make_uint4(pack_h2(__uint_as_float(rr[j8]), __uint_as_float(rr[j8 + 1])),
                                              pack_h2(__uint_as_float(rr[j8 + 2]), __uint_as_float(rr[j8 + 3])),
                                              pack_h2(__uint_as_float(rr[j8 + 4]), __uint_as_float(rr[j8 + 5])),
                                              pack_h2(__uint_as_float(rr[j8 + 6]), __uint_as_float(rr[j8 + 7])));
                        *(uint4*)(Qo + i * 128 + ((((c0 + j8) >> 3) ^ (i & 7)) << 4)) = pk;
                    }
                }
            }
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(t_d4 + lane_base + 64 + c0, rr);
                tmem_ld_wait();
                if (i < DV) {
                    float* ocol = O + (seq * g.L + t0) * (long long)DV + i;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (c0 + j < Cv) ocol[(long long)(c0 + j) * DV] = __uint_as_float(rr[j]);
                }
            }
        }
        tc_fence_before();
        __syncthreads();   // shared and tensor memory are reused by the next chunk
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tb, SM::tmem_cols);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// bf16 tensor [seqs][rows][cols], box = 64 cols x box_rows rows x 1, 128B swizzle, zero fill out of bounds
bool make_map(CUtensorMap* m, const void* base, uint64_t seqs, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {cols, rows, seqs};
    cuuint64_t strides[2] = {cols * 2, rows * cols * 2};
    cuuint32_t box[3] = {64, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int N, int DK, int DV>
int launch(const Problem& p, const TcWs& ws, int dvs, const FlowMaps& maps) {
    using SM = FlowSmem<N, DK, DV>;
    const int smem = SM::total + 1024;
    static_assert(SM::total + 1024 <= 227 * 1024, "shared memory budget");
    PF_CUDA_TRY(cudaFuncSetAttribute(tc_flow<N, DK, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    int dev = 0, sms = 148;
    PF_CUDA_TRY(cudaGetDevice(&dev));
    PF_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const long long G = p.total_chunks();
    const long long slots = (long long)sms * (SM::two_per_sm ? 2 : 1);
    const unsigned grid = (unsigned)(G < slots ? G : slots);
    prof_begin("tc_flow", p.stream);
    tc_flow<N, DK, DV><<<grid, FLOW_THREADS, smem, p.stream>>>(maps, tc_geo(p), ws, (const __nv_bfloat16*)p.beta, p.O, G, dvs);
    prof_end(p.stream);
    PF_CUDA_TRY(cudaGetLastError());
    count_launch(1);
    return PF_OK;
}

}  // namespace

bool tc_flow_available() { return true; }

int tc_flow_launch(const Problem& p, const TcWs& ws, int dvs) {
    if (p.total_chunks() == 0) return PF_OK;
    const int n = p.tile_rows();       // box rows: the whole tile, rows past the chunk's own included (they get beta = 0)
    const uint64_t seqs = (uint64_t)p.B * p.H;
    FlowMaps maps;
    if (!make_map(&maps.k, p.k, seqs, (uint64_t)p.L * p.r, p.d_k, n) ||
        !make_map(&maps.q, p.q, seqs, (uint64_t)p.L, p.d_k, p.chunk) ||
        !make_map(&maps.v, p.v, seqs, (uint64_t)p.L * p.r, p.d_v, n))
        return record_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
#define PF_FLOW_CASE(NN, KK, VV) \
    if (n == NN && p.d_k == KK && p.d_v == VV) return launch<NN, KK, VV>(p, ws, dvs, maps);
    PF_FLOW_CASE(128, 128, 128)
    PF_FLOW_CASE(128, 128, 64)
    PF_FLOW_CASE(128, 64, 128)
    PF_FLOW_CASE(128, 64, 64)
    PF_FLOW_CASE(64, 128, 128)
    PF_FLOW_CASE(64, 128, 64)
    PF_FLOW_CASE(64, 64, 128)
    PF_FLOW_CASE(64, 64, 64)
#undef PF_FLOW_CASE
    return PF_ERR_UNSUPPORTED;
}

}  // namespace pf
