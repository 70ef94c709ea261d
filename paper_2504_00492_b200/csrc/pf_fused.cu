// fused: the whole tensor-core path in ONE cooperative launch (d_k = d_v = 128, chunks of n = C*r rows in tiles of 64 or 128).
//
// The paper's pipeline (Section 3) is Chunk -> Parallel Compute -> Scan.  Here both stages run at the same
// time on disjoint sets of SMs and hand each chunk's flow over through a small ring that stays in L2:
//
//   flow CTAs (one per SM that is not a scan SM) walk over the chunks in time-major order
//       (chunk 0 of every sequence, then chunk 1, ...) and build for each chunk, from Theorem 3.2,
//           X  = (I + Mstrict (.) (K K^T diag(beta)))^{-1}          (so that T' = diag(beta) X)
//           W  = diag(beta) X K,   Uh = diag(beta) X V
//           E  = -K^T W,  Xi^T = Uh^T K                              (the chunk flow of Proposition 2.1)
//           Qt = Q - P W (stored transposed),  OI = P Uh,            P = (Q K^T) (.) Mincl
//       and store (E, Qt, Xi^T) into slot (chunk mod R) of the sequence's ring, OI into the chunk's rows of O;
//   scan CTAs (one per sequence) carry the state over the chunks,
//           O += S Qt^T,      S <- S + S E^T + Xi^T,
//       reading each slot as soon as its flag is set and freeing it for the flow CTAs afterwards.
//
// The ring (R slots of 80 KB per sequence) is rewritten in place, so the hand-off never has to reach HBM; the
// rows of O that hold OI are updated by the scan a few chunk steps after the flow CTA wrote them, while they
// are still in L2.  The only compulsory HBM traffic is one read of q, k, v, beta and one write of O.
//
// A flow CTA is software-pipelined over two chunks (16 warps):
//   warps 0-3  "solve"  the chain that decides the period: epilogue of G = K K^T (mask, column scaling, fp16), the
//                       16 x 16 diagonal blocks of the inverse (Neumann products (I-A)(I+A^2)(I+A^4)(I+A^8) on
//                       mma.sync, two blocks per warp) and the recursive-doubling merges
//   warps 4-11 "bulk"   one program for everything else, each step spread over all eight warps (two per lane
//                       quarter of tensor memory): [Uh | W] into shared memory, P^T, bf16 -> fp16 of the next
//                       chunk's V, K and Q in place, then the drains of E, Xi^T, Qt^T (into the ring) and OI (into
//                       O); its first thread also issues the TMA loads (K and V double-buffered, Q single) at the
//                       points of the program where their buffers fall free
//   warps 12, 13, 15    tcgen05.mma issue, split by product so that no issuing warp waits behind another's operands:
//                       13 polls (mbarrier.test_wait: try_wait may suspend the warp) for G of the next chunk and
//                       [Uh | W] = X [V | K]; 12 issues E and Xi^T; 15 issues P0^T, Qt^T and OI^T
//   warp 14             ring back-pressure and ready flags
// Tensor memory: RA = columns [0,256) holds [Uh | W] and then [E | Xi^T]; RG = [256,384) holds G of the NEXT
// chunk; RC = [384,448) holds P0^T and then Qt^T; RD = [448,512) holds OI^T.
// G is formed from the bf16 tiles as they land (both operands raw); every other product has a derived fp16
// operand, so K, V and Q are converted to fp16 in place, off the critical path.  Qt^T = Q^T - W^T P^T is formed
// entirely on the tensor pipe: Q^T enters the accumulator as four products of the Q tile with a 16 x 16 identity,
// then the correction accumulates onto it.
// Every mbarrier is waited on by parity, so a waiter must never fall two phases behind its producer: the bulk team
// therefore waits for "G of chunk k complete" on a barrier of chunk k's K buffer, whose next phase cannot come before
// the team itself has requested the tile of chunk k+2 into that buffer.
//
// The images that cross the ring are laid out in unswizzled column groups (ns_off): a warp whose lanes hold
// consecutive rows then writes 512 contiguous bytes per store, and the scan's bulk copies bring them into
// shared memory in a form the MMA descriptors read directly.
//
// A scan CTA: warps 0-7 own the state in registers (row j of S per thread, d_k split in two halves of 64 columns).
// Each chunk they write an fp16 copy of it into TENSOR memory, where it is the A operand of both of the chunk's
// products (Delta = S E^T issued by warp 0, O^T = S Qt^T issued by warp 13), so the serial step never goes
// through shared memory.  Warps 8-11 add OI and write O, warp 12 streams the E / Xi / Qt images in with bulk
// copies and is the only poller of the ready flags, warp 14 reports consumed chunks.
//
// Every wait is bounded (about a second of cycles) and reports a code in the status word.  Outer loops are
// deliberately kept rolled: the instruction footprint of sixteen differently-specialised warps matters.
#include <atomic>
#include <string.h>

#include "pf_common.cuh"
#include "pf_tc.cuh"
#include "pf_tc_prims.cuh"

namespace pf {

using namespace tc;

namespace {

constexpr int FT = 512;                 // threads per CTA
constexpr int DK = 128, DV = 128;

// ---- ring slot layout (bytes) ---------------------------------------------------------------------------
constexpr uint32_t SLOT_E = 0;                          // E image : fp16 [16 groups i'/8][128 rows i][16 B]  (K-major A)
constexpr uint32_t SLOT_QT = SLOT_E + DK * DK * 2;      // Qt image: fp16 [ 8 groups t/8 ][128 rows i][16 B]  (MN-major B)
constexpr uint32_t SLOT_XI = SLOT_QT + DK * 128;        // Xi^T    : fp16 [16 groups i/8 ][128 rows j][16 B]
constexpr uint32_t SLOT_BYTES = SLOT_XI + DK * DV * 2;  // 81920

struct FusedGeo {
    int L, r, C, NC, nseq, R;
    int rm;             // strict-mask group size (Problem::mask_group)
    const float* b32;   // null, or fp32 step sizes used in place of beta (Problem::beta32)
    int n_scan, n_flow;
    int items;          // nseq * NC
};

struct FusedWs {
    int* status;        // word 0: first expired wait (0 = none)
    int* ready;         // [nseq][64] (R <= 64 used): chunk index + 1 once the slot holds that chunk; 256 B per sequence
    int* consumed;      // [nseq][32]: word 0 = number of leading chunks the scan no longer needs; 128 B per sequence
    uint8_t* ring;      // [nseq][R][SLOT_BYTES]
};

struct FusedMaps {
    CUtensorMap q, k, v;
};

// ---- shared memory ----------------------------------------------------------------------------------------
// flow role: two 96 KB regions (chunk parity), each holding  X/W | V/Uh | K  back to back (n*256 bytes each),
// so that [V | K] and [W | Uh] are single 256-column B operands.
constexpr int F_REGION = 98304;
constexpr int F_Q = 2 * F_REGION;               // 16 KB      Q
constexpr int F_PT = F_Q + 16384;               // 16 KB      P^T
constexpr int F_BETA = F_PT + 16384;            // 2 x 128 fp32
constexpr int F_BAR = F_BETA + 1024;
constexpr int F_I16 = F_BAR + 512;              // 16 x 16 fp16 identity, unswizzled K-major (512 B)
constexpr int SMEM_BYTES = F_I16 + 512;         // 231424
// scan role
constexpr int S_E = 0;                          // 2 x 32 KB  E images
constexpr int S_XI = S_E + 2 * 32768;           // 2 x 32 KB  Xi images
constexpr int S_QT = S_XI + 2 * 32768;          // 2 x 16 KB  Qt images
constexpr int S_OUT = S_QT + 2 * 16384;         // 2 x 32 KB  fp32 images of S Qt^T, [t][j], on their way into O
static_assert(S_OUT + 2 * 32768 <= F_BAR, "scan role fits below the barrier block");
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");

// barriers (indices into the uint64_t block at F_BAR)
enum {
    // flow role
    B_KFULL = 0,      // [2] TMA: K landed (bf16)
    B_VFULL = 2,      // [2]
    B_QFULL = 4,
    B_K16 = 5,        // [2] bulk: K converted to fp16
    B_V16 = 7,        // [2]
    B_Q16 = 9,
    B_GDONE = 10,     // mma: G complete
    B_GFREE = 11,     // solve: G drained from tensor memory
    B_XREADY = 12,    // [2] solve: X complete
    B_D2DONE = 14,    // mma: [Uh | W] complete
    B_WUREADY = 15,   // bulk: W, Uh in shared memory (RA drained)
    B_P0DONE = 16,    // mma: P0^T complete
    B_PTREADY = 17,   // bulk: P^T in shared memory (RC drained)
    B_D4DONE = 18,    // mma: [Qt^T | OI^T] complete (and everything issued before it)
    B_D4FREE = 19,    // bulk: RC (Qt^T) and RD (OI^T) drained
    B_RAFREE = 20,    // bulk: RA ([E | Xi^T]) drained
    B_GK = 21,        // [2] mma: G complete, per K buffer (the bulk warps convert that K tile only then)
    B_OUTDONE = 27,   // bulk: the chunk's images are stored
    B_SLOTOK = 28,    // flag warp: the chunk's ring slot may be written
    B_RADONE = 29,    // mma: [E | Xi^T] complete
    // scan role
    B_EFULL = 32,     // [2] producer: E image landed
    B_EEMPTY = 34,    // [2] chain: Delta of that chunk complete
    B_XIFULL = 36,    // [2] producer: Xi image landed
    B_XIEMPTY = 38,   // [2] chain: Xi added to the state (one arrival per chain warp)
    B_QTFULL = 40,    // [2] producer: Qt image landed
    B_QTEMPTY = 42,   // [2] mma: O^T of that chunk complete
    B_APUB = 44,      // [2 buffers] mma: Delta of the chunk complete (the O^T product may be issued)
    B_S16FREE = 46,   // [2 buffers] mma: the MMAs that read that fp16 copy of the state are complete
    B_DDONE = 48,     // Delta complete
    B_ODONE = 50,     // [2] mma: O^T complete
    B_OFREE = 52,     // [2] output warps: O^T drained
    B_COUNT = 54
};

#define PF_WAIT(idx, parity, code) mbar_wait_clk(&bar[idx], (uint32_t)(parity), err, code)

__device__ __forceinline__ uint4 pack8n(const uint32_t* r) {
    return make_uint4(pack_h2(__uint_as_float(r[0]), __uint_as_float(r[1])), pack_h2(__uint_as_float(r[2]), __uint_as_float(r[3])),
                      pack_h2(__uint_as_float(r[4]), __uint_as_float(r[5])), pack_h2(__uint_as_float(r[6]), __uint_as_float(r[7])));
}
__device__ __forceinline__ uint4 pack8(const uint32_t* r, float scale) {
    return make_uint4(pack_h2(__uint_as_float(r[0]) * scale, __uint_as_float(r[1]) * scale),
                      pack_h2(__uint_as_float(r[2]) * scale, __uint_as_float(r[3]) * scale),
                      pack_h2(__uint_as_float(r[4]) * scale, __uint_as_float(r[5]) * scale),
                      pack_h2(__uint_as_float(r[6]) * scale, __uint_as_float(r[7]) * scale));
}

// bf16 -> fp16 in place, elementwise (so the swizzled layout is untouched); `nthr` threads, this one is `t`
static __device__ __noinline__ void cvt_region(uint8_t* base, int bytes, int t, int nthr) {
    uint4* p = (uint4*)base;
    const int chunks = bytes >> 4;
#pragma unroll 4
    for (int e = t; e < chunks; e += nthr) {
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

// =============================================================================================================
// flow role
// =============================================================================================================
template <int N>
__device__ void flow_role(const FusedMaps& maps, const FusedGeo& g, const FusedWs& ws,
                          const __nv_bfloat16* __restrict__ beta, float* __restrict__ O, uint8_t* smem, uint64_t* bar,
                          uint32_t tb, int fid) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int r = g.r, C = g.C, nseq = g.nseq;
    int* err = ws.status;
    const int nk = fid < g.items ? (g.items - fid + g.n_flow - 1) / g.n_flow : 0;
    const uint32_t RA = tb, RG = tb + 256, RC = tb + 384, RD = tb + 448;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    constexpr int X_OFF = 0, V_OFF = N * 256, K_OFF = 2 * N * 256;   // inside a parity region

    auto item = [&](int k, int& seq, int& c) {
        const int q = fid + k * g.n_flow;
        c = q / nseq;
        seq = q - c * nseq;
    };

    if (warp < 4) {
        // ------------------------------------------------ solve: G epilogue + triangular inverse -------------
        const int m = tid;
        const int row_lim = (m / g.rm) * g.rm; // rows m' < row_lim: earlier tokens (sum form) / earlier rows (product form)
        const bool deep = g.rm == 1;           // (with groups of two or more rows the 16 x 16 blocks have A^8 = 0)
        float* sBeta = (float*)(smem + F_BETA);
        float beta_next = 0.f;
        if (nk > 0) {
            int seq, c;
            item(0, seq, c);
            const int nv = min(C, g.L - c * C) * r;
            if (m < nv) {
                const long long bi = ((long long)seq * g.L + (long long)c * C) * r + m;
                beta_next = g.b32 ? g.b32[bi] : __bfloat162float(beta[bi]);
            }
        }
#pragma unroll 1
        for (int k = 0; k < nk; ++k) {
            const int b = k & 1;
            uint8_t* sX = smem + b * F_REGION + X_OFF;
            const uint32_t x_b = smem_u32(sX);
            float* sB = sBeta + b * 128;
            const float bm = beta_next;
            beta_next = 0.f;
            if (k + 1 < nk) {
                int seq, c;
                item(k + 1, seq, c);
                const int nv = min(C, g.L - c * C) * r;
                if (m < nv) {
                    const long long bi = ((long long)seq * g.L + (long long)c * C) * r + m;
                    beta_next = g.b32 ? g.b32[bi] : __bfloat162float(beta[bi]);
                }
            }
            // A failed wait must not strand the other threads at a named barrier: the first barrier after the
            // waits carries the outcome, and the whole warpgroup leaves together.
            bool ok = true;
            // (G of chunk k is issued only once W of chunk k-2, in this X region, has been read by all of that chunk's
            //  products; by then the beta half of chunk k-2 has been read by that chunk's [Uh | W] epilogue as well, so it is
            //  rewritten only after this wait: the solve warps may run far ahead of a bulk team that waits for a ring slot)
            ok = PF_WAIT(B_GDONE, k & 1, 102);
            sB[m] = bm;
            tc_fence_after();
            if (!named_bar_and(1, 128, ok)) return;
            // A = Mstrict (.) (G diag(beta)) as fp16 into X.  Warp w holds rows 32w .. 32w+31: the 32-column groups
            // left of 32w lie entirely below the mask's edge (but for the last columns of the nearest one when the
            // token groups of r = 3 rows straddle 32w), the group at 32w holds the edge, the groups to the right are zero.
            if (32 * warp < N) {
#pragma unroll 1
                for (int c0 = 0; c0 < N; c0 += 32) {
                    if (c0 > 32 * warp) {
#pragma unroll
                        for (int j8 = 0; j8 < 4; ++j8) *(uint4*)(sX + chunk_off(m, (c0 >> 3) + j8, N)) = make_uint4(0, 0, 0, 0);
                        continue;
                    }
                    uint32_t rr[32];
                    tmem_ld32(RG + lane_base + c0, rr);
                    float bb[32];
#pragma unroll
                    for (int j4 = 0; j4 < 8; ++j4) {
                        const float4 bv = *(const float4*)(sB + c0 + 4 * j4);
                        bb[4 * j4] = bv.x; bb[4 * j4 + 1] = bv.y; bb[4 * j4 + 2] = bv.z; bb[4 * j4 + 3] = bv.w;
                    }
                    tmem_ld_wait();
                    if (c0 + 32 <= ((32 * warp) / g.rm) * g.rm) {      // (below the edge for every row of the warp)
#pragma unroll
                        for (int j8 = 0; j8 < 32; j8 += 8) {
                            float a[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) a[j] = bb[j8 + j] * __uint_as_float(rr[j8 + j]);
                            *(uint4*)(sX + chunk_off(m, (c0 + j8) >> 3, N)) =
                                make_uint4(pack_h2(a[0], a[1]), pack_h2(a[2], a[3]), pack_h2(a[4], a[5]), pack_h2(a[6], a[7]));
                        }
                    } else {
#pragma unroll
                        for (int j8 = 0; j8 < 32; j8 += 8) {
                            float a[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) a[j] = (c0 + j8 + j < row_lim) ? bb[j8 + j] * __uint_as_float(rr[j8 + j]) : 0.f;
                            *(uint4*)(sX + chunk_off(m, (c0 + j8) >> 3, N)) =
                                make_uint4(pack_h2(a[0], a[1]), pack_h2(a[2], a[3]), pack_h2(a[4], a[5]), pack_h2(a[6], a[7]));
                        }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(&bar[B_GFREE]);
            // 16 x 16 diagonal blocks 2w and 2w+1: their rows were written by this warp
            __syncwarp();
            if (32 * warp < N) {
                diag_inverse16(x_b, sX, 2 * warp, lane, N, deep);
                diag_inverse16(x_b, sX, 2 * warp + 1, lane, N, deep);
            }
            named_bar(1, 128);
            merge_level<N, 16, 1>(x_b, sX, warp, lane);
            merge_level<N, 32, 1>(x_b, sX, warp, lane);
            if (N == 128) merge_level<N, 64, 1>(x_b, sX, warp, lane);
            fence_async_smem();
            mbar_arrive(&bar[B_XREADY + b]);
        }
    } else if (warp < 12) {
        // ------------------------------------------------ bulk: everything else, eight warps per step ----------
        // thread (h, m): lane quarter of row m = 32 (warp & 3) + lane; h = 0 takes the Uh / Xi^T / OI side of
        // every step, h = 1 the W / E / Qt side.
        //
        // Thread 0 of the team also issues the TMA loads, each right after the wait that shows its buffer free.
        const int bt = tid - 128;
        const int h = bt >> 7, m = bt & 127;
        const int tokm = m / r;
        const float* sBeta = (const float*)(smem + F_BETA);
        const uint32_t sw16 = (uint32_t)(m & 7) << 4;
        constexpr uint32_t KV_SLAB = N * 128;                 // bytes of one 64-column slab of K / V / W / Uh
        constexpr uint32_t K_BYTES = N * 256;
        const int dq_c = g.n_flow / nseq, dq_s = g.n_flow - dq_c * nseq;            // how (chunk, sequence) advance per item
        auto advance = [&](int& sq, int& ch) {
            sq += dq_s;
            ch += dq_c;
            if (sq >= nseq) { sq -= nseq; ++ch; }
        };
        auto load_k = [&](int bb, int sq, int ch) {
            mbar_expect_tx(&bar[B_KFULL + bb], K_BYTES);
            for (int hh = 0; hh < 2; ++hh)
                tma_load_3d(smem + bb * F_REGION + K_OFF + hh * KV_SLAB, &maps.k, 64 * hh, ch * C * r, sq, &bar[B_KFULL + bb]);
        };
        auto load_v = [&](int bb, int sq, int ch) {
            mbar_expect_tx(&bar[B_VFULL + bb], K_BYTES);
            for (int hh = 0; hh < 2; ++hh)
                tma_load_3d(smem + bb * F_REGION + V_OFF + hh * KV_SLAB, &maps.v, 64 * hh, ch * C * r, sq, &bar[B_VFULL + bb]);
        };
        auto load_q = [&](int sq, int ch) {
            mbar_expect_tx(&bar[B_QFULL], (uint32_t)C * 256);
            for (int hh = 0; hh < 2; ++hh) tma_load_3d(smem + F_Q + hh * 8192, &maps.q, 64 * hh, ch * C, sq, &bar[B_QFULL]);
        };
        // conversions of chunk kk's V and K tiles (buffers kk & 1); K only once its Gram product has read the bf16 tile
        auto convert_vk = [&](int kk) -> bool {
            const int bb = kk & 1, ph = (kk >> 1) & 1;
            if (!PF_WAIT(B_VFULL + bb, ph, 112)) return false;
            cvt_region(smem + bb * F_REGION + V_OFF, K_BYTES, bt, 256);
            fence_async_smem();
            mbar_arrive(&bar[B_V16 + bb]);
            if (!PF_WAIT(B_KFULL + bb, ph, 111) || !PF_WAIT(B_GK + bb, ph, 110)) return false;
            cvt_region(smem + bb * F_REGION + K_OFF, K_BYTES, bt, 256);
            fence_async_smem();
            mbar_arrive(&bar[B_K16 + bb]);
            return true;
        };
        auto convert_q = [&](int kk) -> bool {
            if (!PF_WAIT(B_QFULL, kk & 1, 114)) return false;
            cvt_region(smem + F_Q, 16384, bt, 256);
            fence_async_smem();
            mbar_arrive(&bar[B_Q16]);
            return true;
        };
        int seq, c;
        item(0, seq, c);
        if (nk > 0) {
            if (bt == 0) {
                int s1 = seq, c1 = c;
                load_k(0, seq, c);
                load_q(seq, c);
                load_v(0, seq, c);
                if (nk > 1) {
                    advance(s1, c1);
                    load_k(1, s1, c1);
                    load_v(1, s1, c1);
                }
            }
            if (!convert_vk(0) || !convert_q(0)) return;
        }
#pragma unroll 1
        for (int k = 0; k < nk; ++k) {
            const int b = k & 1;
            const int Cv = min(C, g.L - c * C), nv = Cv * r;
            uint8_t* slot = ws.ring + ((size_t)seq * g.R + (c % g.R)) * SLOT_BYTES;
            // ---- RA = X [V | K]:  h = 0: Uh = diag(beta) (X V) over V;  h = 1: -W = -diag(beta) (X K) over X   (fp16)
            if (!PF_WAIT(B_D2DONE, k & 1, 118)) return;
            tc_fence_after();
            {
                const float bs = (m < N) ? sBeta[b * 128 + m] : 0.f;
                const float bm = h ? -bs : bs;
                uint8_t* mrow = smem + b * F_REGION + (h ? X_OFF : V_OFF) + m * 128;
                const uint32_t src = RA + lane_base + h * 128;
                // (a tensor-memory load and its wait cost the same ~170 cycles whatever the width: two 32-column loads per wait)
#pragma unroll 1
                for (int sl = 0; sl < 2; ++sl) {                 // 64-column slab
                    uint32_t ra[32], rb[32];
                    tmem_ld32(src + 64 * sl, ra);
                    tmem_ld32(src + 64 * sl + 32, rb);
                    tmem_ld_wait();
                    if (m < N) {
                        uint8_t* base = mrow + sl * (N * 128);
#pragma unroll
                        for (int j8 = 0; j8 < 4; ++j8) {
                            *(uint4*)(base + (((uint32_t)j8 << 4) ^ sw16)) = pack8(ra + 8 * j8, bm);
                            *(uint4*)(base + (((uint32_t)(j8 + 4) << 4) ^ sw16)) = pack8(rb + 8 * j8, bm);
                        }
                    }
                }
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(&bar[B_WUREADY]);
            // ---- P^T = P0^T (.) Mincl as fp16 [m rows][64 t]: 32 columns per half  (P^T of chunk k-1 was last read by
            //      that chunk's Qt / OI products, complete before the drains of chunk k-1 started)
            if (!PF_WAIT(B_P0DONE, k & 1, 117)) return;
            tc_fence_after();
            {
                const int lo = m < nv ? tokm : 64;               // tokens t in [lo, Cv) see row m
                uint8_t* prow_ = smem + F_PT + m * 128;          // (one slab: 64 columns)
                const int c0 = 32 * h;
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
                            a[j] = (t >= lo && t < Cv) ? __uint_as_float(rr[j8 + j]) : 0.f;
                        }
                        *(uint4*)(prow_ + (((uint32_t)((c0 + j8) >> 3) << 4) ^ sw16)) =
                            make_uint4(pack_h2(a[0], a[1]), pack_h2(a[2], a[3]), pack_h2(a[4], a[5]), pack_h2(a[6], a[7]));
                    }
                }
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(&bar[B_PTREADY]);
            // ---- RA = [E | Xi^T]: h = 1: row m of E, h = 0: row m of Xi^T, one 16-byte piece per column group, into the ring
            if (!PF_WAIT(B_SLOTOK, k & 1, 120) || !PF_WAIT(B_RADONE, k & 1, 124)) return;
            tc_fence_after();
            // ---- K of chunk k+2 into the buffer that the products of [E | Xi^T] of this chunk, the last to read it, are
            //      done with (issued before the drain: the next Gram product but one waits for this tile)
            if (bt == 0 && k + 2 < nk) {
                int s2 = seq, c2 = c;
                advance(s2, c2);
                advance(s2, c2);
                load_k(b, s2, c2);
            }
            {
                uint8_t* row = slot + (h ? SLOT_E : SLOT_XI) + m * 16;
                const uint32_t src = RA + lane_base + (h ? 0 : DK);
#pragma unroll 1
                for (int sl = 0; sl < 2; ++sl) {
                    uint32_t ra[32], rb[32];
                    tmem_ld32(src + 64 * sl, ra);
                    tmem_ld32(src + 64 * sl + 32, rb);
                    tmem_ld_wait();
#pragma unroll
                    for (int j8 = 0; j8 < 4; ++j8) {
                        *(uint4*)(row + sl * 16384 + j8 * 2048) = pack8n(ra + 8 * j8);
                        *(uint4*)(row + sl * 16384 + (j8 + 4) * 2048) = pack8n(rb + 8 * j8);
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(&bar[B_RAFREE]);
            // ---- conversions for chunk k+1: only now, so that they do not take shared-memory bandwidth from the products
            //      of [E | Xi^T] (which hold the tensor-memory columns the next [Uh | W] waits for)
            if (k + 1 < nk && !convert_vk(k + 1)) return;
            // ---- h = 1: RC: Qt^T (row i = m of the Qt image);  h = 0: RD: OI^T[j][t] -> OI[t][j = m] (fp32) into the rows of O
            if (!PF_WAIT(B_D4DONE, k & 1, 126)) return;
            tc_fence_after();
            if (bt == 0 && k + 1 < nk) {       // (the Q tile and Uh of this chunk have been read by its last product)
                int s2 = seq, c2 = c;
                advance(s2, c2);
                load_q(s2, c2);
                if (k + 2 < nk) {
                    advance(s2, c2);
                    load_v(b, s2, c2);
                }
            }
            {
                uint32_t ra[32], rb[32];
                const uint32_t src = (h ? RC : RD) + lane_base;
                tmem_ld32(src, ra);
                tmem_ld32(src + 32, rb);
                tmem_ld_wait();
                if (h == 1) {
                    uint8_t* qrow = slot + SLOT_QT + m * 16;
#pragma unroll
                    for (int j8 = 0; j8 < 4; ++j8) {
                        *(uint4*)(qrow + j8 * 2048) = pack8n(ra + 8 * j8);
                        *(uint4*)(qrow + (j8 + 4) * 2048) = pack8n(rb + 8 * j8);
                    }
                } else {
                    float* oi = O + ((long long)seq * g.L + (long long)c * C) * DV + m;
                    if (Cv == 64) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            oi[j * DV] = __uint_as_float(ra[j]);
                            oi[(32 + j) * DV] = __uint_as_float(rb[j]);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (j < Cv) oi[j * DV] = __uint_as_float(ra[j]);
                            if (32 + j < Cv) oi[(32 + j) * DV] = __uint_as_float(rb[j]);
                        }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(&bar[B_D4FREE]);
            mbar_arrive(&bar[B_OUTDONE]);
            // ---- Q of chunk k+1
            if (k + 1 < nk && !convert_q(k + 1)) return;
            advance(seq, c);
        }
    } else if (warp == 13) {
        // ------------------------------------------------ MMA issue, first of three warps: G and [Uh | W] --------
        // Five products per chunk -- G, P0^T, [Uh | W], [E | Xi^T], [Qt^T | OI^T] -- are issued by three warps on three
        // different schedulers (an issuing warp shares its scheduler with busy worker warps, and one warp alone cannot
        // issue fast enough to keep the tensor pipe fed).  Each product is issued as soon as its inputs are there and
        // its accumulator is free, in chunk order per product; this warp polls for whichever of its two is ready, so
        // that G of the next chunk (which the solve warps wait for) is never held back by X of this one, or vice versa.
        int ig = 0, ip3 = 0;
        const uint32_t reg0 = smem_u32(smem);
        auto ph2 = [](int kk) { return (uint32_t)((kk >> 1) & 1); };
        long long t_last = clock64();
#pragma unroll 1
        while (ip3 < nk) {
            bool progress = false;
            // (G of chunk ig: its K tile has landed; the solve warps have drained G of chunk ig-1; and the last product of
            //  chunk ig-2 is done with W in the X region G's epilogue goes to.  The bulk warps, which convert K of chunk ig
            //  only after this product, wait for it on a barrier of that K buffer: its next phase is the Gram product of
            //  chunk ig+2, whose tile they request themselves after that conversion, so they cannot miss a phase, and the
            //  Gram product of the next chunk need not wait for them.)
            if (ig < nk && mbar_test(&bar[B_KFULL + (ig & 1)], ph2(ig)) && (ig == 0 || mbar_test(&bar[B_GFREE], (ig - 1) & 1)) &&
                (ig < 2 || mbar_test(&bar[B_D4DONE], (ig - 2) & 1))) {
                tc_fence_after();
                const uint32_t k_b = reg0 + (ig & 1) * F_REGION + K_OFF;
                gemm_uni<false, false, N, DK, N, N, true>(RG, k_b, k_b);            // G = K K^T from the bf16 tile as it landed
                commit_uni(&bar[B_GDONE]);
                commit_uni(&bar[B_GK + (ig & 1)]);
                ++ig;
                progress = true;
            }
            if (mbar_test(&bar[B_XREADY + (ip3 & 1)], ph2(ip3)) && mbar_test(&bar[B_V16 + (ip3 & 1)], ph2(ip3)) &&
                mbar_test(&bar[B_K16 + (ip3 & 1)], ph2(ip3)) && (ip3 == 0 || mbar_test(&bar[B_RAFREE], (ip3 - 1) & 1))) {
                tc_fence_after();
                const uint32_t x_b = reg0 + (ip3 & 1) * F_REGION + X_OFF;
                gemm_uni<false, true, DV + DK, N, N, N>(RA, x_b, x_b + V_OFF);      // [Uh | W] (before the row scaling) = X [V | K]
                commit_uni(&bar[B_D2DONE]);
                ++ip3;
                progress = true;
            }
            if (progress) {
                t_last = clock64();
            } else if (clock64() - t_last > WAIT_CYCLES) {
                atomicCAS(err, 0, 142);
                return;
            } else if (*(volatile int*)err != 0) {
                return;
            }
        }
    } else if (warp == 12) {
        // ------------------------------------------------ MMA issue, second warp: [E | Xi^T] -------------------------
#pragma unroll 1
        for (int k = 0; k < nk; ++k) {
            const uint32_t x_b = smem_u32(smem + (k & 1) * F_REGION + X_OFF), v_b = x_b + V_OFF, k_b = x_b + K_OFF;
            if (!PF_WAIT(B_WUREADY, k & 1, 149)) return;
            tc_fence_after();
            gemm_uni<true, true, DK, N, N, N>(RA, k_b, x_b);                        // E = K^T (-W)     (lanes i, columns i')
            gemm_uni<true, true, DK, N, N, N>(RA + DK, v_b, k_b);                   // Xi^T = Uh^T K    (lanes j, columns i)
            commit_uni(&bar[B_RADONE]);
        }
    } else if (warp == 15) {
        // ------------------------------------------------ MMA issue, third warp: P0^T and [Qt^T | OI^T] --------------
        const uint32_t q_b = smem_u32(smem + F_Q), pt_b = smem_u32(smem + F_PT), i16_b = smem_u32(smem + F_I16);
#pragma unroll 1
        for (int k = 0; k < nk; ++k) {
            const uint32_t x_b = smem_u32(smem + (k & 1) * F_REGION + X_OFF), v_b = x_b + V_OFF, k_b = x_b + K_OFF;
            // P0^T = K Q^T  (RC: Qt^T of the chunk before has been drained)
            if (!PF_WAIT(B_K16 + (k & 1), (k >> 1) & 1, 152) || !PF_WAIT(B_Q16, k & 1, 153)) return;
            if (k >= 1 && !PF_WAIT(B_D4FREE, (k - 1) & 1, 147)) return;
            tc_fence_after();
            gemm_uni<false, false, 64, DK, N, 64>(RC, k_b, q_b);
            commit_uni(&bar[B_P0DONE]);
            // Qt^T = Q^T + (-W)^T P^T (over P0^T, which the bulk warps have turned into P^T): Q^T first, 16 columns t at a
            // time, as Q^T times a 16 x 16 identity (A = the Q tile read MN-major, one K-step of 16 tokens per block of
            // columns);  OI^T = Uh^T P^T.   (All of the bulk warps have passed W / Uh on before they pass P^T on.)
            if (!PF_WAIT(B_PTREADY, k & 1, 150)) return;
            tc_fence_after();
#pragma unroll
            for (int cb = 0; cb < 4; ++cb)
                gemm_lay<L_SWMN, L_NSK, 16, 16, 64, 16>(RC + 16 * cb, q_b + 2048 * cb, i16_b);
            gemm_uni<true, true, 64, N, N, N, false, true>(RC, x_b, pt_b);
            gemm_uni<true, true, 64, N, N, N>(RD, v_b, pt_b);
            commit_uni(&bar[B_D4DONE]);
        }
    } else if (warp == 14) {
        // ------------------------------------------------ flag warp: ring back-pressure, ready flags ---------
        if (lane == 0) {
#pragma unroll 1
            for (int k = 0; k < nk; ++k) {
                int seq, c;
                item(k, seq, c);
                const int slot_i = c % g.R;
                // the scan must be done with the chunk that used this slot before
                if (c >= g.R && !flag_wait_ge(&ws.consumed[seq * 32], c - g.R + 1, err, 161)) return;
                mbar_arrive(&bar[B_SLOTOK]);
                if (!PF_WAIT(B_OUTDONE, k & 1, 163)) return;
                __threadfence();
                st_release_gpu(&ws.ready[seq * 64 + slot_i], c + 1);
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
    const uint32_t t_delta = tb, t_o = tb + 128, t_a = tb + 256;     // Delta | 2 x O^T | 2 x fp16 state
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint8_t* ring = ws.ring + (size_t)seq * g.R * SLOT_BYTES;
    const int* ready = ws.ready + seq * 64;
    volatile int* vis = (volatile int*)(smem + F_BAR + B_COUNT * 8 + 8);   // chunks whose ready flag the producer has acquired
    volatile int* odone = (volatile int*)(smem + F_BAR + B_COUNT * 8 + 12); // output-warp completions (4 per chunk)

    if (warp < 8) {
        // ------------------------------------------------ chain: the state lives here -------------------------
        // thread (w, j): row j of S, columns i = 64w .. 64w+63
        const int w = warp >> 2, j = tid & 127;
        float S[64];
        const long long sbase = ((long long)seq * DK + 64 * w) * DV + j;
#pragma unroll
        for (int ii = 0; ii < 64; ++ii) S[ii] = S0 ? S0[sbase + (long long)ii * DV] : 0.f;
#pragma unroll 1
        for (int c = 0; c < NC; ++c) {
            const int buf = c & 1;
            // fp16 copy of the state into tensor memory (A operand of Delta and of O^T): 32 packed columns per thread
            bool ok = true;
            if (c >= 2) ok = PF_WAIT(B_S16FREE + buf, ((c >> 1) - 1) & 1, 201);
            tc_fence_after();
            {
                uint32_t pk[32];
#pragma unroll
                for (int q = 0; q < 32; ++q) pk[q] = pack_h2(S[2 * q], S[2 * q + 1]);
                tmem_st32(t_a + buf * 64 + 32 * w + lane_base, pk);
                tmem_st_wait();
            }
            tc_fence_before();
            if (!named_bar_and(1, 256, ok)) return;
            // warp 0 issues Delta[j][i] = sum_i' S[j][i'] E[i][i']; its completion also releases warp 13, which
            // issues the O^T product of the same copy (so that O^T never sits in front of Delta in the tensor pipe)
            if (warp == 0) {
                if (!PF_WAIT(B_EFULL + buf, (c >> 1) & 1, 231)) return;
                tc_fence_after();
                gemm_ta<L_NSK, DK, DK, 128>(t_delta, t_a + buf * 64, smem_u32(smem + S_E + buf * 32768));
                commit_uni(&bar[B_DDONE]);
                commit_uni(&bar[B_EEMPTY + buf]);
                commit_uni(&bar[B_APUB + buf]);
            }
            if (!PF_WAIT(B_XIFULL + buf, (c >> 1) & 1, 203)) return;
            if (!PF_WAIT(B_DDONE, c & 1, 202)) return;
            tc_fence_after();
            // S += Delta + Xi^T   (row j, columns 64w..64w+63; Xi^T from its column-group image)
            const uint8_t* xrow = smem + S_XI + buf * 32768 + w * 16384 + j * 16;
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(t_delta + lane_base + 64 * w + c0, rr);
                uint4 xi[4];
#pragma unroll
                for (int p = 0; p < 4; ++p) xi[p] = *(const uint4*)(xrow + ((c0 >> 3) + p) * 2048);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    const uint32_t wd = ((const uint32_t*)&xi[e >> 3])[(e & 7) >> 1];
                    const float2 xv = __half22float2(*reinterpret_cast<const __half2*>(&wd));
                    S[c0 + e] += __uint_as_float(rr[e]) + xv.x;
                    S[c0 + e + 1] += __uint_as_float(rr[e + 1]) + xv.y;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar[B_XIEMPTY + buf]);
        }
        if (S_final)
#pragma unroll
            for (int ii = 0; ii < 64; ++ii) S_final[sbase + (long long)ii * DV] = S[ii];
    } else if (warp < 12) {
        // ------------------------------------------------ output: O = OI + (S Qt^T)^T ---------------------------
        // OI is already in the rows of O (left there by the flow CTA, visible once the chunk's ready flag has been
        // acquired).  The chunk's S Qt^T goes from tensor memory into a [t][j] fp32 image in shared memory, which
        // is exactly the layout of the chunk's rows of O, and one bulk reduction adds the image to them at the L2:
        // OI is never read back, and the only per-thread work is the transposing copy.
        const int j = tid - 256;
#pragma unroll 1
        for (int c = 0; c < NC; ++c) {
            const int ob = c & 1;
            const int Cv = min(g.C, g.L - c * g.C);
            float* img = (float*)(smem + S_OUT + ob * 32768);
            bool ok = PF_WAIT(B_ODONE + ob, (c >> 1) & 1, 212);
            tc_fence_after();
            // the reduction of chunk c-2 has read this image (its issuing thread waits, the rest learn of it here)
            if (tid == 256) {
                bulk_wait_read_1();
                ok = ok && smem_wait_ge(vis, c + 1, err, 211);     // (long since true: Qt was loaded after it)
            }
            if (!named_bar_and(2, 128, ok)) break;      // (every thread of the four warps leaves together)
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t rr[32];
                tmem_ld32(t_o + ob * 64 + lane_base + c0, rr);
                tmem_ld_wait();
#pragma unroll
                for (int t = 0; t < 32; ++t) img[(c0 + t) * DV + j] = __uint_as_float(rr[t]);
            }
            tc_fence_before();
            mbar_arrive(&bar[B_OFREE + ob]);
            fence_async_smem();
            named_bar(2, 128);
            if (tid == 256) {
                fence_async_global();
                bulk_reduce_add_f32(O + ((long long)seq * g.L + (long long)c * g.C) * DV, img, (uint32_t)Cv * DV * 4u);
                bulk_commit();
                atomicAdd((int*)odone, 4);       // (a counter, not a barrier: the reporter may lag by any amount)
            }
        }
        if (tid == 256) bulk_wait_all();
    } else if (warp == 12) {
        // ------------------------------------------------ producer: ring -> shared memory ----------------------
        if (lane == 0) {
            auto load_e = [&](int c) -> bool {
                const int st = c & 1;
                if (!smem_wait_ge(vis, c + 1, err, 222)) return false;      // (warp 14 polls the ready flags, ahead of the loads)
                fence_async_global();
                if (c >= 2 && !PF_WAIT(B_EEMPTY + st, ((c >> 1) - 1) & 1, 221)) return false;
                mbar_expect_tx(&bar[B_EFULL + st], DK * DK * 2);
                bulk_load(smem + S_E + st * 32768, ring + (size_t)(c % g.R) * SLOT_BYTES + SLOT_E, DK * DK * 2, &bar[B_EFULL + st]);
                return true;
            };
#pragma unroll 1
            for (int c = 0; c < NC; ++c) {
                if (c == 0 && !load_e(0)) return;
                // (the flag of chunk c was acquired by load_e(c))
                const uint8_t* slot = ring + (size_t)(c % g.R) * SLOT_BYTES;
                const int b = c & 1;
                if (c >= 2 && !PF_WAIT(B_XIEMPTY + b, ((c >> 1) - 1) & 1, 224)) return;
                mbar_expect_tx(&bar[B_XIFULL + b], DK * DV * 2);
                bulk_load(smem + S_XI + b * 32768, slot + SLOT_XI, DK * DV * 2, &bar[B_XIFULL + b]);
                if (c >= 2 && !PF_WAIT(B_QTEMPTY + b, ((c >> 1) - 1) & 1, 223)) return;
                mbar_expect_tx(&bar[B_QTFULL + b], DK * 128);
                bulk_load(smem + S_QT + b * 16384, slot + SLOT_QT, DK * 128, &bar[B_QTFULL + b]);
                if (c + 1 < NC && !load_e(c + 1)) return;
            }
        }
    } else if (warp == 13) {
        // ------------------------------------------------ O^T[j][t] = sum_i S[j][i] Qt^T[i][t] (whole warp) -----
#pragma unroll 1
        for (int c = 0; c < NC; ++c) {
            const int buf = c & 1;
            if (!PF_WAIT(B_APUB + buf, (c >> 1) & 1, 235)) return;
            if (!PF_WAIT(B_QTFULL + buf, (c >> 1) & 1, 234)) return;
            if (c >= 2 && !PF_WAIT(B_OFREE + buf, ((c >> 1) - 1) & 1, 233)) return;
            tc_fence_after();
            gemm_ta<L_NSMN, 64, DK, 128>(t_o + buf * 64, t_a + buf * 64, smem_u32(smem + S_QT + buf * 16384));
            commit_uni(&bar[B_ODONE + buf]);
            commit_uni(&bar[B_QTEMPTY + buf]);
            commit_uni(&bar[B_S16FREE + buf]);
        }
    } else if (warp == 14) {
        // ------------------------------------------------ ready flags in, consumed reports out -----------------
        // One lane polls the ring's ready flags in chunk order, as far ahead of the loads as the flow CTAs are, and
        // publishes the count in shared memory (so that no load waits a trip to the L2 for a flag that was set long
        // ago).  The same loop reports consumption: once the four output warps are done with chunk c, chunks < c
        // are consumed (the chain finished chunk c-1 before it published the state for chunk c) and their ring
        // slots may be rewritten.  It polls a shared counter and always reports the latest value, however far it
        // has fallen behind.
        if (lane == 0) {
            int reported = 0, seen = 0;
            const long long t0 = clock64();
            long long t_last = t0;
            while (reported < NC - 1 || seen < NC) {
                bool progress = false;
                if (seen < NC && ld_acquire_gpu(&ready[seen % g.R]) >= seen + 1) {
                    ++seen;
                    __threadfence_block();
                    *vis = seen;
                    progress = true;
                }
                const int chunks_done = *odone >> 2;
                if (chunks_done - 1 > reported) {
                    reported = chunks_done - 1;
                    __threadfence_block();
                    st_release_gpu(&ws.consumed[seq * 32], reported);
                    progress = true;
                }
                if (progress) {
                    t_last = clock64();
                } else if (clock64() - t_last > WAIT_CYCLES) {
                    atomicCAS(err, 0, 232);
                    break;
                } else if (*(volatile int*)err != 0) {
                    break;
                } else if (seen == NC) {
                    __nanosleep(200);
                }
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
            for (int x = 0; x < 2; ++x) {
                mbar_init(&bar[B_EFULL + x], 1); mbar_init(&bar[B_EEMPTY + x], 1);
                mbar_init(&bar[B_XIFULL + x], 1); mbar_init(&bar[B_XIEMPTY + x], 8);
                mbar_init(&bar[B_QTFULL + x], 1); mbar_init(&bar[B_QTEMPTY + x], 1);
                mbar_init(&bar[B_APUB + x], 1); mbar_init(&bar[B_S16FREE + x], 1);
                mbar_init(&bar[B_DDONE + x], 1); mbar_init(&bar[B_ODONE + x], 1); mbar_init(&bar[B_OFREE + x], 128);
            }
        } else {
            for (int x = 0; x < 2; ++x) {
                                mbar_init(&bar[B_KFULL + x], 1); mbar_init(&bar[B_VFULL + x], 1);
                mbar_init(&bar[B_K16 + x], 256); mbar_init(&bar[B_V16 + x], 256);
                mbar_init(&bar[B_XREADY + x], 128);
            }
            mbar_init(&bar[B_QFULL], 1); mbar_init(&bar[B_Q16], 256);
            prefetch_tmap(&maps.q);
            prefetch_tmap(&maps.k);
            prefetch_tmap(&maps.v);
            mbar_init(&bar[B_GDONE], 1); mbar_init(&bar[B_GFREE], 128); mbar_init(&bar[B_GK], 1); mbar_init(&bar[B_GK + 1], 1);
            mbar_init(&bar[B_D2DONE], 1); mbar_init(&bar[B_WUREADY], 256);
            mbar_init(&bar[B_P0DONE], 1); mbar_init(&bar[B_PTREADY], 256);
            mbar_init(&bar[B_D4DONE], 1); mbar_init(&bar[B_RADONE], 1); mbar_init(&bar[B_D4FREE], 256); mbar_init(&bar[B_RAFREE], 256);
            mbar_init(&bar[B_OUTDONE], 256);
            mbar_init(&bar[B_SLOTOK], 1);
        }
        *(volatile int*)(smem + F_BAR + B_COUNT * 8 + 8) = 0;
        *(volatile int*)(smem + F_BAR + B_COUNT * 8 + 12) = 0;
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(&tmem_base_s, 512);
    if (!is_scan) {
        // operands with fewer than 128 rows are read past their tile: keep those bytes finite
        for (int e = tid; e < F_BETA / 16; e += FT) ((uint4*)smem)[e] = make_uint4(0, 0, 0, 0);
    }
    // a 16 x 16 fp16 identity, element (n, k) at ns_off(n, k, 16): the second operand of the products that add an fp16
    // image to an accumulator (Q^T into Qt^T in the flow role, Xi^T into the state's increment in the scan role)
    if (tid < 256) *(__half*)(smem + F_I16 + ns_off(tid >> 4, tid & 15, 16)) = __float2half_rn((tid >> 4) == (tid & 15) ? 1.f : 0.f);
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = tmem_base_s;

    if (is_scan) scan_role(g, ws, S0, O, S_final, smem, bar, tb, (int)blockIdx.x);
    else flow_role<N>(maps, g, ws, beta, O, smem, bar, tb, (int)blockIdx.x - g.n_scan);


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

// SM count of the current device (cached per device ordinal: a process may use several devices)
int sm_count() {
    constexpr int MAX_DEV = 64;
    static std::atomic<int> cache[MAX_DEV];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (dev >= 0 && dev < MAX_DEV) {
        const int have = cache[dev].load(std::memory_order_relaxed);
        if (have) return have;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (dev >= 0 && dev < MAX_DEV) cache[dev].store(sms, std::memory_order_relaxed);
    return sms;
}

// Slots per sequence (pf_params.ring_depth, 3..64).  Default 8; 16 for long sequences while all rings together stay
// well inside the L2: over a thousand chunks the flow CTAs drift apart and a deeper ring absorbs it (measured at
// 32 sequences of 1024 chunks: 2.29 ms against 2.50 ms; no difference at 128 chunks).
int ring_depth(const Problem& p) {
    const int NC = p.chunks_per_seq();
    int want = p.ring_depth;
    if (want <= 0) want = (NC > 256 && (size_t)p.B * p.H * 16 * SLOT_BYTES <= ((size_t)48 << 20)) ? 16 : 8;
    return NC < want ? (NC < 1 ? 1 : NC) : want;
}

struct Carve {
    size_t status, ready, consumed, ring, total, flag_bytes;
};
Carve carve(const Problem& p) {
    const size_t nseq = (size_t)p.B * p.H;
    const int R = ring_depth(p);
    Carve c{};
    c.status = 0;
    c.ready = 4096;
    c.consumed = c.ready + nseq * 256;          // every sequence's flags in cache lines of their own
    c.flag_bytes = align_up(c.consumed + nseq * 128, 1024);
    c.ring = c.flag_bytes;
    c.total = c.ring + nseq * R * SLOT_BYTES;
    return c;
}

}  // namespace

// One CTA per sequence scans, the rest build flows.  Measured at d = 128, r = 2: up to about 100 sequences the single
// launch beats the two-launch form (96: 400 against 477 us at L = 2048), beyond that too few SMs are left for the
// flows (120: 865 against 600 us; 136: 2194 against 669 us).
bool fused_preferred(const Problem& p) {
    return (long long)p.B * p.H * 10 <= (long long)sm_count() * 7;
}

bool fused_supported(const Problem& p) {
    if (p.in_dtype != PF_DTYPE_BF16 || p.d_k != DK || p.d_v != DV) return false;
    if (p.tile_rows() == 0 || p.chunk > 64 || p.L < 1) return false;
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
    ws.status = p.status;
    ws.ready = (int*)(base + cv.ready);
    ws.consumed = (int*)(base + cv.consumed);
    ws.ring = base + cv.ring;
    PF_CUDA_TRY(cudaMemsetAsync(base, 0, cv.flag_bytes, p.stream));
    FusedGeo g{};
    g.L = p.L; g.r = p.r; g.C = p.chunk; g.NC = NC; g.nseq = nseq; g.R = ring_depth(p); g.rm = p.mask_group(); g.b32 = p.beta32;
    g.items = nseq * NC;
    const int sms = sm_count();
    g.n_scan = nseq;
    g.n_flow = sms - nseq;
    if (g.items < g.n_flow) g.n_flow = g.items > 0 ? g.items : 1;
    FusedMaps maps;
    if (NC > 0) {
        const uint64_t seqs = (uint64_t)nseq;
        if (!make_map(&maps.k, p.k, seqs, (uint64_t)p.L * p.r, p.d_k, p.tile_rows()) ||
            !make_map(&maps.q, p.q, seqs, (uint64_t)p.L, p.d_k, p.chunk) ||
            !make_map(&maps.v, p.v, seqs, (uint64_t)p.L * p.r, p.d_v, p.tile_rows()))
            return record_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    } else {
        memset(&maps, 0, sizeof(maps));
    }
    const __nv_bfloat16* beta = (const __nv_bfloat16*)p.beta;
    const float* S0 = p.S0;
    float* O = p.O;
    float* Sf = p.S_final;
    void* args[] = {(void*)&maps, (void*)&g, (void*)&ws, (void*)&beta, (void*)&S0, (void*)&O, (void*)&Sf};
    const void* fn = p.tile_rows() == 128 ? (const void*)fused_kernel<128> : (const void*)fused_kernel<64>;
    PF_CUDA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
    prof_begin("fused", p.stream);
    PF_CUDA_TRY(cudaLaunchCooperativeKernel(fn, dim3((unsigned)(g.n_scan + g.n_flow)), dim3(FT), args, SMEM_BYTES, p.stream));
    prof_end(p.stream);
    count_launch(1);
    return PF_OK;
}

}  // namespace pf
