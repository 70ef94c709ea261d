// fused: the whole tensor-core path in ONE cooperative launch (d_k = d_v = 128, n = C*r in {64, 128}).
//
// The paper's pipeline (Section 3) is Chunk -> Parallel Compute -> Scan.  Here both stages run at the same
// time on disjoint sets of SMs and hand each chunk's flow over through a small ring that stays in L2:
//
//   flow CTAs (one per SM that is not a scan SM) walk over the chunks in time-major order
//       (chunk 0 of every sequence, then chunk 1, ...) and build for each chunk, from Theorem 3.2,
//           X  = (I + Mstrict (.) (K K^T diag(beta)))^{-1}          (so that T' = diag(beta) X)
//           W  = diag(beta) X K,   Uh = diag(beta) X V
//           E  = -K^T W,  Xi = K^T Uh                                (the chunk flow of Proposition 2.1)
//           Qt = Q - P W (stored transposed),  OI = P Uh,            P = (Q K^T) (.) Mincl
//       and store (E, Qt, Xi, OI) into slot (chunk mod R) of the sequence's ring;
//   scan CTAs (one per sequence) carry the state over the chunks,
//           O^T = OI^T + S Qt^T,      S^T <- S^T + E S^T + Xi,
//       reading each slot as soon as its flag is set and freeing it for the flow CTAs afterwards.
//
// The ring (R slots of 112 KB per sequence) is rewritten in place, so the hand-off never has to reach HBM:
// the only compulsory HBM traffic is one read of q, k, v, beta and one write of O.
//
// A flow CTA is software-pipelined over two chunks with five kinds of warps (14 warps):
//   warps 0-3  "solve"  epilogue of G = K K^T (mask, column scaling, fp16) and the triangular inverse
//   warps 4-7  "mid"    bf16 -> fp16 conversion of K, V, Q; epilogue of P^T; epilogue of [W | Uh]
//   warps 8-11 "out"    epilogue of [E | Xi] and [Qt^T | OI^T], staging and bulk stores into the ring
//   warp 12             TMA loads (K and V double-buffered, Q single)
//   warp 13             tcgen05.mma issue
// Tensor memory: RA = columns [0,256) holds [W | Uh] and then [E | Xi]; RB = [256,384) holds G of the NEXT
// chunk and then [Qt^T | OI^T] of the current one; RC = [384,448) holds P0^T.
//
// A scan CTA: warps 0-7 own the state (row i of S^T per thread, d_v split in two halves of 64 columns),
// warps 8-11 add OI and write O, warp 12 streams E/Qt images in with bulk copies, warp 13 issues the MMAs.
//
// Every wait is bounded (about a second of cycles) and reports a code in the status word.
#include "pf_common.cuh"
#include "pf_tc.cuh"
#include "pf_tc_prims.cuh"

namespace pf {

using namespace tc;

namespace {

constexpr int FT = 448;                 // threads per CTA
constexpr int DK = 128, DV = 128;
constexpr int SCAN_STAGES = 3;

// ---- ring slot layout (bytes) ---------------------------------------------------------------------------
constexpr uint32_t SLOT_E = 0;                          // E image : fp16 [2 slabs][128 rows i][128 B]   (K-major A)
constexpr uint32_t SLOT_QT = SLOT_E + DK * DK * 2;      // Qt image: fp16 [128 rows i][128 B = 64 t]     (MN-major B)
constexpr uint32_t SLOT_XI = SLOT_QT + DK * 128;        // Xi image: fp16 [2 slabs (j half)][128 rows i][128 B]
constexpr uint32_t SLOT_OI = SLOT_XI + DK * DV * 2;     // OI      : fp32 [64 rows t][128 cols j]
constexpr uint32_t SLOT_BYTES = SLOT_OI + 64 * DV * 4;  // 114688

struct FusedGeo {
    int L, r, C, NC, nseq, R;
    int n_scan, n_flow;
    int items;          // nseq * NC
};

struct FusedWs {
    int* status;        // word 0: first expired wait (0 = none)
    int* ready;         // [nseq][R]: chunk index + 1 once the slot holds that chunk
    int* consumed;      // [nseq]: number of leading chunks the scan no longer needs
    uint8_t* ring;      // [nseq][R][SLOT_BYTES]
};

struct FusedMaps {
    CUtensorMap q, k, v;
};

// ---- shared memory ----------------------------------------------------------------------------------------
// flow role
constexpr int F_K = 0;                          // 2 x 32 KB  K (fp16 after conversion)
constexpr int F_V = F_K + 2 * 32768;            // 2 x 32 KB  V -> Uh -> Xi staging
constexpr int F_X = F_V + 2 * 32768;            // 2 x 32 KB  A -> X -> W -> E staging
constexpr int F_Q = F_X + 2 * 32768;            // 16 KB      Q
constexpr int F_PT = F_Q + 16384;               // 16 KB      P^T -> Qt staging
constexpr int F_BETA = F_PT + 16384;            // 2 x 128 fp32
constexpr int F_BAR = F_BETA + 1024;
constexpr int SMEM_BYTES = F_BAR + 512;         // 230912
// scan role
constexpr int S_STAGE = 0;                      // 3 x (32 KB E + 16 KB Qt)
constexpr int S_STAGE_BYTES = 32768 + 16384;
constexpr int S_S16 = S_STAGE + SCAN_STAGES * S_STAGE_BYTES;   // 2 x 32 KB fp16 copy of the state
static_assert(S_S16 + 2 * 32768 <= F_BAR, "scan role fits below the barrier block");
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");

// barriers (indices into the uint64_t block at F_BAR)
enum {
    // flow role
    B_KFULL = 0,      // [2] TMA: K landed
    B_VFULL = 2,      // [2]
    B_QFULL = 4,
    B_K16 = 5,        // [2] mid: K converted
    B_V16 = 7,        // [2]
    B_Q16 = 9,
    B_GDONE = 10,     // mma: G complete
    B_GFREE = 11,     // solve: G drained from tensor memory
    B_XREADY = 12,    // [2] solve: X complete
    B_D2DONE = 14,    // mma: [W | Uh] complete
    B_WUREADY = 15,   // mid: W, Uh in shared memory (RA drained)
    B_P0DONE = 16,    // mma: P0^T complete
    B_PTREADY = 17,   // mid: P^T in shared memory (RC drained)
    B_D34DONE = 18,   // mma: [E | Xi] and [Qt^T | OI^T] complete
    B_D4FREE = 19,    // out: RB drained, Q no longer needed
    B_RAFREE = 20,    // out: RA drained
    B_XFREE = 21,     // [2] out: bulk store finished reading the E staging
    B_VFREE = 23,     // [2] out: ... the Xi staging
    B_PTFREE = 25,    // out: ... the Qt staging
    // scan role
    B_FULL = 32,      // [3] producer: E, Qt landed (and the slot's Xi, OI are visible)
    B_EMPTY = 35,     // [3] everyone is done with the stage's chunk
    B_SREADY = 38,    // [2 buffers][2 halves]
    B_DDONE = 42,     // [2 halves]
    B_ODONE = 44,     // [2]
    B_OFREE = 46,     // [2]
    B_COUNT = 48
};

__device__ __forceinline__ uint4 pack8(const uint32_t* r, float scale) {
    return make_uint4(pack_h2(__uint_as_float(r[0]) * scale, __uint_as_float(r[1]) * scale),
                      pack_h2(__uint_as_float(r[2]) * scale, __uint_as_float(r[3]) * scale),
                      pack_h2(__uint_as_float(r[4]) * scale, __uint_as_float(r[5]) * scale),
                      pack_h2(__uint_as_float(r[6]) * scale, __uint_as_float(r[7]) * scale));
}

// bf16 -> fp16 in place, elementwise (so the swizzled layout is untouched); 128 threads
__device__ __forceinline__ void cvt_region(uint8_t* base, int bytes, int t128) {
    uint4* p = (uint4*)base;
    const int chunks = bytes >> 4;
#pragma unroll 4
    for (int e = t128; e < chunks; e += 128) {
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

// One level of the recursive-doubling inverse (Proposition on block-triangular inversion): diagonal blocks of
// size S are merged into blocks of size 2S,  X_hi,lo = -X_hi,hi A_hi,lo X_lo,lo.  Task = (merge, 16-row
// strip): N/32 tasks, one warp each; the four solve warps synchronise on named barrier 1.
template <int N, int S>
__device__ __forceinline__ void merge_level(uint32_t xb, uint8_t* xg, int warp, int lane) {
    constexpr int TASKS = N / 32;
    constexpr int STRIPS = S / 16;
    constexpr int NT = S / 8;
    float z[NT][4];
    const bool has_task = warp < TASKS;
    const int q = warp / STRIPS, strip = warp % STRIPS;
    const int lo0 = 2 * S * q, hi0 = lo0 + S, R0 = hi0 + 16 * strip;
    if (has_task) {
        float u[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) u[nt][e] = 0.f;
#pragma unroll
        for (int kk = 0; kk < S / 16; ++kk) {
            if (kk > strip) continue;   // X_hi,hi is lower triangular
            uint32_t a[4];
            ldmatrix_x4(a, xb + slab_off(R0 + (lane & 15), hi0 + 16 * kk + ((lane >> 4) << 3), N));
#pragma unroll
            for (int np = 0; np < S / 16; ++np) {
                uint32_t b[4];
                const int id = lane >> 3;
                ldmatrix_x4_trans(b, xb + slab_off(hi0 + 16 * kk + (lane & 7) + ((id & 1) << 3),
                                                   lo0 + 16 * np + ((id >> 1) << 3), N));
                mma_16816(u[2 * np], a, b[0], b[1]);
                mma_16816(u[2 * np + 1], a, b[2], b[3]);
            }
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) z[nt][e] = 0.f;
#pragma unroll
        for (int kk = 0; kk < S / 16; ++kk) {
            uint32_t a[4];
            a[0] = pack_h2(u[2 * kk][0], u[2 * kk][1]);
            a[1] = pack_h2(u[2 * kk][2], u[2 * kk][3]);
            a[2] = pack_h2(u[2 * kk + 1][0], u[2 * kk + 1][1]);
            a[3] = pack_h2(u[2 * kk + 1][2], u[2 * kk + 1][3]);
#pragma unroll
            for (int np = 0; np < S / 16; ++np) {
                if (np > kk) continue;  // X_lo,lo is lower triangular
                uint32_t b[4];
                const int id = lane >> 3;
                ldmatrix_x4_trans(b, xb + slab_off(lo0 + 16 * kk + (lane & 7) + ((id & 1) << 3),
                                                   lo0 + 16 * np + ((id >> 1) << 3), N));
                mma_16816(z[2 * np], a, b[0], b[1]);
                mma_16816(z[2 * np + 1], a, b[2], b[3]);
            }
        }
    }
    named_bar(1, 128);   // every strip has read A_hi,lo before anyone overwrites it
    if (has_task) {
        const int gq = lane >> 2, t4 = lane & 3;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int col = lo0 + 8 * nt + 2 * t4;
            *(uint32_t*)(xg + slab_off(R0 + gq, col, N)) = pack_h2(-z[nt][0], -z[nt][1]);
            *(uint32_t*)(xg + slab_off(R0 + gq + 8, col, N)) = pack_h2(-z[nt][2], -z[nt][3]);
        }
    }
    named_bar(1, 128);
}

// =============================================================================================================
// flow role
// =============================================================================================================
template <int N>
__device__ void flow_role(const FusedMaps& maps, const FusedGeo& g, const FusedWs& ws,
                          const __nv_bfloat16* __restrict__ beta, uint8_t* smem, uint64_t* bar, uint32_t tb,
                          int fid) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int r = g.r, C = g.C, nseq = g.nseq;
    int* err = ws.status;
    const int nk = fid < g.items ? (g.items - fid + g.n_flow - 1) / g.n_flow : 0;
    const uint32_t RA = tb, RB = tb + 256, RC = tb + 384;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    constexpr uint32_t KV_SLAB = N * 128;                 // bytes of one 64-column slab of K / V / W / Uh
    constexpr uint32_t K_BYTES = N * 256;

    auto item = [&](int k, int& seq, int& c) {
        const int q = fid + k * g.n_flow;
        c = q / nseq;
        seq = q - c * nseq;
    };

    if (warp < 4) {
        // ------------------------------------------------ solve: G epilogue + triangular inverse -------------
        const int m = tid;
        const int tokm = m / r, row_lim = tokm * r;       // rows m' < row_lim belong to earlier tokens
        float* sBeta = (float*)(smem + F_BETA);
        float beta_next = 0.f;
        if (nk > 0) {
            int seq, c;
            item(0, seq, c);
            const int nv = min(C, g.L - c * C) * r;
            if (m < nv) beta_next = __bfloat162float(beta[((long long)seq * g.L + (long long)c * C) * r + m]);
        }
        for (int k = 0; k < nk; ++k) {
            const int b = k & 1;
            uint8_t* sX = smem + F_X + b * 32768;
            const uint32_t x_b = smem_u32(sX);
            float* sB = sBeta + b * 128;
            const float bm = beta_next;
            beta_next = 0.f;
            if (k + 1 < nk) {
                int seq, c;
                item(k + 1, seq, c);
                const int nv = min(C, g.L - c * C) * r;
                if (m < nv) beta_next = __bfloat162float(beta[((long long)seq * g.L + (long long)c * C) * r + m]);
            }
            // A failed wait must not strand the other threads at a named barrier: the first barrier after the
            // waits carries the outcome, and the whole warpgroup leaves together.
            bool ok = true;
            if (k >= 2) ok = mbar_wait_clk(&bar[B_XFREE + b], ((k >> 1) - 1) & 1, err, 101);
            sB[m] = bm;     // the readers of this half (chunk k-2) are done: X of chunk k-2 has been released
            ok = ok && mbar_wait_clk(&bar[B_GDONE], k & 1, err, 102);
            tc_fence_after();
            if (!named_bar_and(1, 128, ok)) return;
            // A = Mstrict (.) (G diag(beta)) as fp16 into X
#pragma unroll
            for (int c0 = 0; c0 < N; c0 += 32) {
                if (c0 < 32 * (warp + 1)) {
                    uint32_t rr[32];
                    tmem_ld32(RB + lane_base + c0, rr);
                    tmem_ld_wait();
                    if (m < N) {
#pragma unroll
                        for (int j8 = 0; j8 < 32; j8 += 8) {
                            float a[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const int mp = c0 + j8 + j;
                                a[j] = (mp < row_lim) ? sB[mp] * __uint_as_float(rr[j8 + j]) : 0.f;
                            }
                            *(uint4*)(sX + slab_off(m, c0 + j8, N)) =
                                make_uint4(pack_h2(a[0], a[1]), pack_h2(a[2], a[3]), pack_h2(a[4], a[5]), pack_h2(a[6], a[7]));
                        }
                    }
                } else if (m < N) {
#pragma unroll
                    for (int j8 = 0; j8 < 32; j8 += 8) *(uint4*)(sX + slab_off(m, c0 + j8, N)) = make_uint4(0, 0, 0, 0);
                }
            }
            tc_fence_before();
            mbar_arrive(&bar[B_GFREE]);
            named_bar(1, 128);
            // 16x16 diagonal blocks: forward substitution, one thread per column of one block (fp32)
            float x[16];
            const int bk = tid >> 4, cc = tid & 15;
            if (tid < N) {
#pragma unroll
                for (int mm = 0; mm < 16; ++mm) {
                    const uint4 lo = *(const uint4*)(sX + slab_off(16 * bk + mm, 16 * bk, N));
                    const uint4 hi = *(const uint4*)(sX + slab_off(16 * bk + mm, 16 * bk + 8, N));
                    const __half2* hl = (const __half2*)&lo;
                    const __half2* hh = (const __half2*)&hi;
                    float a[16];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f0 = __half22float2(hl[e]), f1 = __half22float2(hh[e]);
                        a[2 * e] = f0.x; a[2 * e + 1] = f0.y; a[8 + 2 * e] = f1.x; a[9 + 2 * e] = f1.y;
                    }
                    float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
                    for (int mp = 0; mp < mm; ++mp) {
                        if (mp & 1) acc1 = fmaf(a[mp], x[mp], acc1);
                        else acc0 = fmaf(a[mp], x[mp], acc0);
                    }
                    x[mm] = ((mm == cc) ? 1.f : 0.f) - (acc0 + acc1);
                }
            }
            named_bar(1, 128);
            if (tid < N) {
#pragma unroll
                for (int mm = 0; mm < 16; ++mm)
                    *(__half*)(sX + slab_off(16 * bk + mm, 16 * bk + cc, N)) = __float2half_rn(x[mm]);
            }
            named_bar(1, 128);
            merge_level<N, 16>(x_b, sX, warp, lane);
            merge_level<N, 32>(x_b, sX, warp, lane);
            if (N == 128) merge_level<N, 64>(x_b, sX, warp, lane);
            fence_async_smem();
            mbar_arrive(&bar[B_XREADY + b]);
        }
    } else if (warp < 8) {
        // ------------------------------------------------ mid: conversions, P^T and [W | Uh] epilogues --------
        const int m = tid - 128;
        const int tokm = m / r;
        const float* sBeta = (const float*)(smem + F_BETA);
        uint8_t* sPT = smem + F_PT;
        if (nk > 0) {
            if (!mbar_wait_clk(&bar[B_KFULL + 0], 0, err, 111)) return;
            cvt_region(smem + F_K, K_BYTES, m);
            fence_async_smem();
            mbar_arrive(&bar[B_K16 + 0]);
            if (!mbar_wait_clk(&bar[B_VFULL + 0], 0, err, 112)) return;
            cvt_region(smem + F_V, K_BYTES, m);
            fence_async_smem();
            mbar_arrive(&bar[B_V16 + 0]);
        }
        for (int k = 0; k < nk; ++k) {
            const int b = k & 1, b1 = b ^ 1;
            int seq, c;
            item(k, seq, c);
            const int Cv = min(C, g.L - c * C), nv = Cv * r;
            if (k + 1 < nk) {
                if (!mbar_wait_clk(&bar[B_KFULL + b1], ((k + 1) >> 1) & 1, err, 113)) return;
                cvt_region(smem + F_K + b1 * 32768, K_BYTES, m);
                fence_async_smem();
                mbar_arrive(&bar[B_K16 + b1]);
            }
            if (!mbar_wait_clk(&bar[B_QFULL], k & 1, err, 114)) return;
            cvt_region(smem + F_Q, 16384, m);
            fence_async_smem();
            mbar_arrive(&bar[B_Q16]);
            if (k + 1 < nk) {
                if (!mbar_wait_clk(&bar[B_VFULL + b1], ((k + 1) >> 1) & 1, err, 115)) return;
                cvt_region(smem + F_V + b1 * 32768, K_BYTES, m);
                fence_async_smem();
                mbar_arrive(&bar[B_V16 + b1]);
            }
            // P^T = P0^T (.) Mincl as fp16 [m rows][64 t]
            if (k >= 1 && !mbar_wait_clk(&bar[B_PTFREE], (k - 1) & 1, err, 116)) return;
            if (!mbar_wait_clk(&bar[B_P0DONE], k & 1, err, 117)) return;
            tc_fence_after();
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(RC + lane_base + c0, rr);
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
                        *(uint4*)(sPT + m * 128 + ((((c0 + j8) >> 3) ^ (m & 7)) << 4)) =
                            make_uint4(pack_h2(a[0], a[1]), pack_h2(a[2], a[3]), pack_h2(a[4], a[5]), pack_h2(a[6], a[7]));
                    }
                }
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(&bar[B_PTREADY]);
            // W = diag(beta) (X K), Uh = diag(beta) (X V) as fp16 operands (W over X, Uh over V)
            if (!mbar_wait_clk(&bar[B_D2DONE], k & 1, err, 118)) return;
            tc_fence_after();
            const float bm = (m < N) ? sBeta[b * 128 + m] : 0.f;
            uint8_t* sW = smem + F_X + b * 32768;
            uint8_t* sU = smem + F_V + b * 32768;
#pragma unroll 2
            for (int c0 = 0; c0 < DK + DV; c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(RA + lane_base + c0, rr);
                tmem_ld_wait();
                if (m < N) {
                    uint8_t* dst = (c0 < DK) ? sW : sU;
                    const int col0 = (c0 < DK) ? c0 : c0 - DK;
#pragma unroll
                    for (int j8 = 0; j8 < 32; j8 += 8) *(uint4*)(dst + slab_off(m, col0 + j8, N)) = pack8(rr + j8, bm);
                }
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(&bar[B_WUREADY]);
        }
    } else if (warp < 12) {
        // ------------------------------------------------ out: flow -> ring -----------------------------------
        const int i = tid - 256;
        uint8_t* sQ = smem + F_Q;
        uint8_t* sPT = smem + F_PT;
        for (int k = 0; k < nk; ++k) {
            const int b = k & 1;
            int seq, c;
            item(k, seq, c);
            const int Cv = min(C, g.L - c * C);
            const int slot_i = c % g.R;
            uint8_t* slot = ws.ring + ((size_t)seq * g.R + slot_i) * SLOT_BYTES;
            // the scan must be done with the chunk that used this slot before
            bool ok = true;
            if (c >= g.R && i == 0) ok = flag_wait_ge(&ws.consumed[seq], c - g.R + 1, err, 121);
            ok = ok && mbar_wait_clk(&bar[B_Q16], k & 1, err, 122);
            ok = ok && mbar_wait_clk(&bar[B_D34DONE], k & 1, err, 123);
            tc_fence_after();
            if (!named_bar_and(3, 128, ok)) return;
            uint8_t* sE = smem + F_X + b * 32768;
            uint8_t* sXi = smem + F_V + b * 32768;
            // [Qt^T | OI^T] from RB:  Qt^T[i][t] = Q[t][i] - (W^T P^T)[i][t]  -> staging (over P^T);  OI -> ring
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(RB + lane_base + c0, rr);
                tmem_ld_wait();
#pragma unroll
                for (int j8 = 0; j8 < 32; j8 += 8) {
                    float a[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int t = c0 + j8 + j;
                        a[j] = __uint_as_float(rr[j8 + j]) + __half2float(*(const __half*)(sQ + slab_off(t, i, 64)));
                    }
                    *(uint4*)(sPT + i * 128 + ((((c0 + j8) >> 3) ^ (i & 7)) << 4)) =
                        make_uint4(pack_h2(a[0], a[1]), pack_h2(a[2], a[3]), pack_h2(a[4], a[5]), pack_h2(a[6], a[7]));
                }
            }
            float* oi = (float*)(slot + SLOT_OI) + i;
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(RB + lane_base + 64 + c0, rr);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (c0 + j < Cv) oi[(c0 + j) * DV] = __uint_as_float(rr[j]);
            }
            tc_fence_before();
            mbar_arrive(&bar[B_D4FREE]);
            // [E | Xi] from RA -> staging (E over W, Xi over Uh)
#pragma unroll 2
            for (int c0 = 0; c0 < DK + DV; c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(RA + lane_base + c0, rr);
                tmem_ld_wait();
                uint8_t* dst = (c0 < DK) ? sE : sXi;
                const int col0 = (c0 < DK) ? c0 : c0 - DK;
#pragma unroll
                for (int j8 = 0; j8 < 32; j8 += 8) *(uint4*)(dst + slab_off(i, col0 + j8, 128)) = pack8(rr + j8, 1.f);
            }
            tc_fence_before();
            mbar_arrive(&bar[B_RAFREE]);
            fence_async_smem();
            named_bar(3, 128);
            if (i == 0) {
                bulk_store(slot + SLOT_E, sE, DK * DK * 2);
                bulk_store(slot + SLOT_XI, sXi, DK * DV * 2);
                bulk_store(slot + SLOT_QT, sPT, DK * 128);
                bulk_commit();
                bulk_wait_read_all();
                mbar_arrive(&bar[B_XFREE + b]);
                mbar_arrive(&bar[B_VFREE + b]);
                mbar_arrive(&bar[B_PTFREE]);
                bulk_wait_all();
                fence_async_global();
                __threadfence();
                st_release_gpu(&ws.ready[seq * g.R + slot_i], c + 1);
            }
        }
    } else if (warp == 12) {
        // ------------------------------------------------ TMA loads -------------------------------------------
        if (lane == 0) {
            for (int j = 0; j <= nk; ++j) {
                const int b = j & 1;
                int seq = 0, c = 0;
                if (j < nk) {
                    item(j, seq, c);
                    if (j >= 2 && !mbar_wait_clk(&bar[B_D34DONE], (j - 2) & 1, err, 131)) return;
                    mbar_expect_tx(&bar[B_KFULL + b], K_BYTES);
                    for (int h = 0; h < 2; ++h)
                        tma_load_3d(smem + F_K + b * 32768 + h * KV_SLAB, &maps.k, 64 * h, c * C * r, seq, &bar[B_KFULL + b]);
                }
                if (j >= 1) {
                    int sq, cq;
                    item(j - 1, sq, cq);
                    if (j >= 2 && !mbar_wait_clk(&bar[B_D4FREE], (j - 2) & 1, err, 132)) return;
                    mbar_expect_tx(&bar[B_QFULL], (uint32_t)C * 256);
                    for (int h = 0; h < 2; ++h)
                        tma_load_3d(smem + F_Q + h * 8192, &maps.q, 64 * h, cq * C, sq, &bar[B_QFULL]);
                }
                if (j < nk) {
                    if (j >= 2 && !mbar_wait_clk(&bar[B_VFREE + b], ((j >> 1) - 1) & 1, err, 133)) return;
                    mbar_expect_tx(&bar[B_VFULL + b], K_BYTES);
                    for (int h = 0; h < 2; ++h)
                        tma_load_3d(smem + F_V + b * 32768 + h * KV_SLAB, &maps.v, 64 * h, c * C * r, seq, &bar[B_VFULL + b]);
                }
            }
        }
    } else {
        // ------------------------------------------------ MMA issue -------------------------------------------
        if (lane == 0 && nk > 0) {
            const uint32_t q_b = smem_u32(smem + F_Q), pt_b = smem_u32(smem + F_PT);
            if (!mbar_wait_clk(&bar[B_K16 + 0], 0, err, 141)) return;
            tc_fence_after();
            {
                const uint32_t k_b = smem_u32(smem + F_K);
                gemm_issue<false, false>(RB, k_b, N, k_b, N, N, DK, false, false);     // G(0) = K K^T
                mma_commit(&bar[B_GDONE]);
            }
            for (int k = 0; k < nk; ++k) {
                const int b = k & 1, b1 = b ^ 1;
                const uint32_t k_b = smem_u32(smem + F_K + b * 32768), v_b = smem_u32(smem + F_V + b * 32768),
                               x_b = smem_u32(smem + F_X + b * 32768);
                // [W | Uh] = X [K | V]
                if (!mbar_wait_clk(&bar[B_XREADY + b], (k >> 1) & 1, err, 142)) return;
                if (!mbar_wait_clk(&bar[B_V16 + b], (k >> 1) & 1, err, 143)) return;
                if (k >= 1 && !mbar_wait_clk(&bar[B_RAFREE], (k - 1) & 1, err, 144)) return;
                tc_fence_after();
                gemm_issue<false, true>(RA, x_b, N, k_b, N, DK, N, false, false);
                gemm_issue<false, true>(RA + DK, x_b, N, v_b, N, DV, N, false, false);
                mma_commit(&bar[B_D2DONE]);
                // G of the next chunk
                if (k + 1 < nk) {
                    if (!mbar_wait_clk(&bar[B_K16 + b1], ((k + 1) >> 1) & 1, err, 145)) return;
                    if (!mbar_wait_clk(&bar[B_GFREE], k & 1, err, 146)) return;
                    if (k >= 1 && !mbar_wait_clk(&bar[B_D4FREE], (k - 1) & 1, err, 147)) return;
                    tc_fence_after();
                    const uint32_t k1_b = smem_u32(smem + F_K + b1 * 32768);
                    gemm_issue<false, false>(RB, k1_b, N, k1_b, N, N, DK, false, false);
                    mma_commit(&bar[B_GDONE]);
                }
                // P0^T = K Q^T
                if (!mbar_wait_clk(&bar[B_Q16], k & 1, err, 148)) return;
                tc_fence_after();
                gemm_issue<false, false>(RC, k_b, N, q_b, 64, 64, DK, false, false);
                mma_commit(&bar[B_P0DONE]);
                // [E | Xi] = K^T [-W | Uh]
                if (!mbar_wait_clk(&bar[B_WUREADY], k & 1, err, 149)) return;
                tc_fence_after();
                gemm_issue<true, true>(RA, k_b, N, x_b, N, DK, N, true, false);
                gemm_issue<true, true>(RA + DK, k_b, N, v_b, N, DV, N, false, false);
                // [Qt^T - Q^T | OI^T] = [-W | Uh]^T P^T
                if (!mbar_wait_clk(&bar[B_PTREADY], k & 1, err, 150)) return;
                if (k + 1 < nk && !mbar_wait_clk(&bar[B_GFREE], (k + 1) & 1, err, 151)) return;
                tc_fence_after();
                gemm_issue<true, true>(RB, x_b, N, pt_b, N, 64, N, true, false);
                gemm_issue<true, true>(RB + 64, v_b, N, pt_b, N, 64, N, false, false);
                mma_commit(&bar[B_D34DONE]);
            }
        }
    }
}

// =============================================================================================================
// scan role
// =============================================================================================================
__device__ void scan_role(const FusedGeo& g, const FusedWs& ws, const float* __restrict__ S0, float* __restrict__ O,
                          float* __restrict__ S_final, uint8_t* smem, uint64_t* bar, uint32_t tb, int seq) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int NC = g.NC;
    int* err = ws.status;
    const uint32_t t_delta = tb, t_o = tb + 128;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint8_t* ring = ws.ring + (size_t)seq * g.R * SLOT_BYTES;

    if (warp < 8) {
        // ------------------------------------------------ chain: the state lives here -------------------------
        const int w = warp >> 2, i = tid & 127;
        float S[64];
        const long long srow = ((long long)seq * DK + i) * DV + 64 * w;
#pragma unroll
        for (int j = 0; j < 64; j += 4) {
            float4 v4 = S0 ? *(const float4*)(S0 + srow + j) : make_float4(0.f, 0.f, 0.f, 0.f);
            S[j] = v4.x; S[j + 1] = v4.y; S[j + 2] = v4.z; S[j + 3] = v4.w;
        }
        for (int c = 0; c < NC; ++c) {
            const int st = c % SCAN_STAGES, buf = c & 1;
            if (!mbar_wait_clk(&bar[B_FULL + st], (c / SCAN_STAGES) & 1, err, 201)) return;
            // Xi row i, columns 64w..64w+63 (swizzled 16-byte chunks)
            const uint8_t* xrow = ring + (size_t)(c % g.R) * SLOT_BYTES + SLOT_XI + w * 16384 + i * 128;
            uint4 xi[8];
#pragma unroll
            for (int p = 0; p < 8; ++p) xi[p] = ld_cg_u4(xrow + ((p ^ (i & 7)) << 4));
            // fp16 copy of the state: B operand of Delta, A operand of O^T
            uint8_t* sb = smem + S_S16 + buf * 32768 + w * 16384 + i * 128;
#pragma unroll
            for (int p = 0; p < 8; ++p)
                *(uint4*)(sb + ((p ^ (i & 7)) << 4)) =
                    make_uint4(pack_h2(S[8 * p], S[8 * p + 1]), pack_h2(S[8 * p + 2], S[8 * p + 3]),
                               pack_h2(S[8 * p + 4], S[8 * p + 5]), pack_h2(S[8 * p + 6], S[8 * p + 7]));
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(&bar[B_SREADY + buf * 2 + w]);
            if (!mbar_wait_clk(&bar[B_DDONE + w], c & 1, err, 202)) return;
            tc_fence_after();
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(t_delta + lane_base + 64 * w + c0, rr);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const uint32_t wd = ((const uint32_t*)&xi[(c0 + j) >> 3])[((c0 + j) & 7) >> 1];
                    const float2 xv = __half22float2(*reinterpret_cast<const __half2*>(&wd));
                    S[c0 + j] += __uint_as_float(rr[j]) + xv.x;
                    S[c0 + j + 1] += __uint_as_float(rr[j + 1]) + xv.y;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar[B_EMPTY + st]);
        }
        if (S_final)
#pragma unroll
            for (int j = 0; j < 64; j += 4) *(float4*)(S_final + srow + j) = make_float4(S[j], S[j + 1], S[j + 2], S[j + 3]);
    } else if (warp < 12) {
        // ------------------------------------------------ output: O^T = OI^T + S Qt^T --------------------------
        const int j = tid - 256;
        for (int c = 0; c < NC; ++c) {
            const int st = c % SCAN_STAGES, ob = c & 1;
            const int Cv = min(g.C, g.L - c * g.C);
            if (!mbar_wait_clk(&bar[B_FULL + st], (c / SCAN_STAGES) & 1, err, 211)) return;
            const float* oi = (const float*)(ring + (size_t)(c % g.R) * SLOT_BYTES + SLOT_OI) + j;
            float* orow = O + ((long long)seq * g.L + (long long)c * g.C) * DV + j;
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                float a[32];
#pragma unroll
                for (int t = 0; t < 32; ++t) a[t] = (c0 + t < Cv) ? ld_cg_f32(oi + (c0 + t) * DV) : 0.f;
                if (c0 == 0) {
                    if (!mbar_wait_clk(&bar[B_ODONE + ob], (c >> 1) & 1, err, 212)) return;
                    tc_fence_after();
                }
                uint32_t rr[32];
                tmem_ld32(t_o + ob * 64 + lane_base + c0, rr);
                tmem_ld_wait();
#pragma unroll
                for (int t = 0; t < 32; ++t)
                    if (c0 + t < Cv) orow[(long long)(c0 + t) * DV] = a[t] + __uint_as_float(rr[t]);
            }
            tc_fence_before();
            mbar_arrive(&bar[B_OFREE + ob]);
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar[B_EMPTY + st]);
        }
    } else if (warp == 12) {
        // ------------------------------------------------ producer: ring -> shared memory ----------------------
        if (lane == 0) {
            for (int c = 0; c < NC; ++c) {
                const int st = c % SCAN_STAGES;
                if (c >= SCAN_STAGES) {
                    if (!mbar_wait_clk(&bar[B_EMPTY + st], ((c / SCAN_STAGES) - 1) & 1, err, 221)) return;
                    st_release_gpu(&ws.consumed[seq], c - SCAN_STAGES + 1);
                }
                const int slot_i = c % g.R;
                if (!flag_wait_ge(&ws.ready[seq * g.R + slot_i], c + 1, err, 222)) return;
                fence_async_global();
                const uint8_t* slot = ring + (size_t)slot_i * SLOT_BYTES;
                uint8_t* dst = smem + S_STAGE + st * S_STAGE_BYTES;
                mbar_expect_tx(&bar[B_FULL + st], DK * DK * 2 + DK * 128);
                bulk_load(dst, slot + SLOT_E, DK * DK * 2, &bar[B_FULL + st]);
                bulk_load(dst + 32768, slot + SLOT_QT, DK * 128, &bar[B_FULL + st]);
            }
        }
    } else {
        // ------------------------------------------------ MMA issue -------------------------------------------
        if (lane == 0) {
            for (int c = 0; c < NC; ++c) {
                const int st = c % SCAN_STAGES, buf = c & 1, ob = c & 1;
                const uint32_t e_b = smem_u32(smem + S_STAGE + st * S_STAGE_BYTES), qt_b = e_b + 32768;
                const uint32_t s_b = smem_u32(smem + S_S16 + buf * 32768);
                if (!mbar_wait_clk(&bar[B_FULL + st], (c / SCAN_STAGES) & 1, err, 231)) return;
                for (int w = 0; w < 2; ++w) {
                    if (!mbar_wait_clk(&bar[B_SREADY + buf * 2 + w], (c >> 1) & 1, err, 232)) return;
                    tc_fence_after();
                    // Delta^T[i][j] = sum_i' E[i][i'] S^T[i'][j],  j in the half w
                    gemm_issue<false, true>(t_delta + 64 * w, e_b, 128, s_b + w * 16384, 128, 64, DK, false, false);
                    mma_commit(&bar[B_DDONE + w]);
                }
                if (c >= 2 && !mbar_wait_clk(&bar[B_OFREE + ob], ((c >> 1) - 1) & 1, err, 233)) return;
                tc_fence_after();
                // O^T[j][t] = sum_i S^T[i][j] Qt^T[i][t]
                gemm_issue<true, true>(t_o + ob * 64, s_b, 128, qt_b, 128, 64, DK, false, false);
                mma_commit(&bar[B_ODONE + ob]);
                mma_commit(&bar[B_EMPTY + st]);
            }
        }
    }
}

template <int N>
__global__ void __launch_bounds__(FT, 1)
fused_kernel(const __grid_constant__ FusedMaps maps, FusedGeo g, FusedWs ws, const __nv_bfloat16* __restrict__ beta,
             const float* __restrict__ S0, float* __restrict__ O, float* __restrict__ S_final) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* bar = (uint64_t*)(smem + F_BAR);
    uint32_t& tmem_base_s = *(uint32_t*)(smem + F_BAR + B_COUNT * 8);
    const int tid = threadIdx.x, warp = tid >> 5;
    const bool is_scan = (int)blockIdx.x < g.n_scan;

    if ((smem_u32(smem) & 1023u) != 0) {       // the swizzled layouts need a 1024-byte aligned base
        if (tid == 0) atomicCAS(ws.status, 0, 99);
        return;     // uniform: every thread of the CTA leaves
    }
    if (tid == 0) {
        if (is_scan) {
            for (int s = 0; s < SCAN_STAGES; ++s) { mbar_init(&bar[B_FULL + s], 1); mbar_init(&bar[B_EMPTY + s], 13); }
            for (int x = 0; x < 4; ++x) mbar_init(&bar[B_SREADY + x], 128);
            for (int x = 0; x < 2; ++x) { mbar_init(&bar[B_DDONE + x], 1); mbar_init(&bar[B_ODONE + x], 1); mbar_init(&bar[B_OFREE + x], 128); }
        } else {
            for (int x = 0; x < 2; ++x) {
                mbar_init(&bar[B_KFULL + x], 1); mbar_init(&bar[B_VFULL + x], 1);
                mbar_init(&bar[B_K16 + x], 128); mbar_init(&bar[B_V16 + x], 128);
                mbar_init(&bar[B_XREADY + x], 128);
                mbar_init(&bar[B_XFREE + x], 1); mbar_init(&bar[B_VFREE + x], 1);
            }
            mbar_init(&bar[B_QFULL], 1); mbar_init(&bar[B_Q16], 128);
            mbar_init(&bar[B_GDONE], 1); mbar_init(&bar[B_GFREE], 128);
            mbar_init(&bar[B_D2DONE], 1); mbar_init(&bar[B_WUREADY], 128);
            mbar_init(&bar[B_P0DONE], 1); mbar_init(&bar[B_PTREADY], 128);
            mbar_init(&bar[B_D34DONE], 1); mbar_init(&bar[B_D4FREE], 128); mbar_init(&bar[B_RAFREE], 128);
            mbar_init(&bar[B_PTFREE], 1);
            prefetch_tmap(&maps.q);
            prefetch_tmap(&maps.k);
            prefetch_tmap(&maps.v);
        }
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(&tmem_base_s, 512);
    if (!is_scan) {
        // operands with fewer than 128 rows are read past their tile: keep those bytes finite
        for (int e = tid; e < F_BETA / 16; e += FT) ((uint4*)smem)[e] = make_uint4(0, 0, 0, 0);
        fence_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = tmem_base_s;

    if (is_scan) scan_role(g, ws, S0, O, S_final, smem, bar, tb, (int)blockIdx.x);
    else flow_role<N>(maps, g, ws, beta, smem, bar, tb, (int)blockIdx.x - g.n_scan);

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tb, 512);
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

int sm_count() {
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            sms = 0;
    }
    return sms;
}

int ring_depth(const Problem& p) {
    const int NC = p.chunks_per_seq();
    return NC < 8 ? (NC < 1 ? 1 : NC) : 8;
}

struct Carve {
    size_t status, ready, consumed, ring, total, flag_bytes;
};
Carve carve(const Problem& p) {
    const size_t nseq = (size_t)p.B * p.H;
    const int R = ring_depth(p);
    Carve c{};
    c.status = 0;
    c.ready = 1024;
    c.consumed = c.ready + align_up(nseq * R * 4, 256);
    c.flag_bytes = align_up(c.consumed + nseq * 4, 1024);
    c.ring = c.flag_bytes;
    c.total = c.ring + nseq * R * SLOT_BYTES;
    return c;
}

}  // namespace

bool fused_supported(const Problem& p) {
    if (p.in_dtype != PF_DTYPE_BF16 || p.d_k != DK || p.d_v != DV) return false;
    const int n = p.n();
    if (!(n == 64 || n == 128) || p.chunk > 64 || p.L < 1) return false;
    const long long nseq = (long long)p.B * p.H;
    const int sms = sm_count();
    if (sms < 16) return false;
    if (nseq > sms - 8) return false;                    // one scan CTA per sequence, the rest build flows
    if (nseq * p.chunks_per_seq() > 0x3fffffffLL) return false;
    return true;
}

size_t fused_workspace_bytes(const Problem& p) { return carve(p).total + 1024; }

int fused_forward(const Problem& p, void* workspace) {
    const int NC = p.chunks_per_seq();
    const int nseq = p.B * p.H;
    const Carve cv = carve(p);
    uint8_t* base = (uint8_t*)workspace;
    FusedWs ws;
    ws.status = (int*)(base + cv.status);
    ws.ready = (int*)(base + cv.ready);
    ws.consumed = (int*)(base + cv.consumed);
    ws.ring = base + cv.ring;
    PF_CUDA_TRY(cudaMemsetAsync(base, 0, cv.flag_bytes, p.stream));
    FusedGeo g{};
    g.L = p.L; g.r = p.r; g.C = p.chunk; g.NC = NC; g.nseq = nseq; g.R = ring_depth(p);
    g.items = nseq * NC;
    const int sms = sm_count();
    g.n_scan = nseq;
    g.n_flow = sms - nseq;
    if (g.items < g.n_flow) g.n_flow = g.items > 0 ? g.items : 1;
    FusedMaps maps;
    if (NC > 0) {
        const uint64_t seqs = (uint64_t)nseq;
        if (!make_map(&maps.k, p.k, seqs, (uint64_t)p.L * p.r, p.d_k, p.n()) ||
            !make_map(&maps.q, p.q, seqs, (uint64_t)p.L, p.d_k, p.chunk) ||
            !make_map(&maps.v, p.v, seqs, (uint64_t)p.L * p.r, p.d_v, p.n()))
            return record_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    } else {
        memset(&maps, 0, sizeof(maps));
    }
    const __nv_bfloat16* beta = (const __nv_bfloat16*)p.beta;
    const float* S0 = p.S0;
    float* O = p.O;
    float* Sf = p.S_final;
    void* args[] = {(void*)&maps, (void*)&g, (void*)&ws, (void*)&beta, (void*)&S0, (void*)&O, (void*)&Sf};
    const void* fn = p.n() == 128 ? (const void*)fused_kernel<128> : (const void*)fused_kernel<64>;
    PF_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
    prof_begin("fused", p.stream);
    PF_CUDA_TRY(cudaLaunchCooperativeKernel(fn, dim3((unsigned)(g.n_scan + g.n_flow)), dim3(FT), args, SMEM_BYTES, p.stream));
    prof_end(p.stream);
    count_launch(1);
    return PF_OK;
}

}  // namespace pf
