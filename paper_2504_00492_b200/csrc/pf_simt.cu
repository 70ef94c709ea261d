// fp32 SIMT (FFMA) evaluation of the chunk form of Theorem 3.2.  This is the path of the fp32
// entry point (tolerance 1e-5 rules out reduced-precision tensor-core operands) and the on-device
// reference the tensor-core kernels are debugged against.  Four kernels:
//
//   simt_gram   per chunk:  A = Mstrict (.) diag(beta) K K^T   and   P = (Q K^T) (.) Mincl
//   simt_solve  per chunk:  T' = (I + A)^{-1} diag(beta)        (column-parallel forward substitution)
//   simt_wu     per chunk:  W = T' K,  Uh = T' V
//   simt_scan   per (b, h, d_v slice), serial over chunks:
//               U' = Uh - W S^T,  O = Q S^T + P U',  S <- S + U'^T K
//
// With option "wu_builder" = 1, simt_solve and simt_wu are replaced by simt_sigdelta, which obtains the same W and Uh
// from the two-index system of Theorem 3.3 (the "signature kernel inspired algorithm"), swept along its
// antidiagonals.
//
// Rows of a chunk are m = t*r + j (token t, factor j), n = chunk*r.  Rows past the end of the
// sequence behave as beta = 0, k = 0, which leaves the state untouched; their outputs are not stored.
#include "pf_common.cuh"
#include "pf_tc.cuh"

namespace pf {
namespace {

template <class T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) {
    return __bfloat162float(*p);
}

struct Geo {
    int L, d_k, d_v, r, C, n, NC;   // NC = chunks per sequence
    int rm;                         // strict-mask group size (Problem::mask_group)
    const float* b32;               // null, or fp32 step sizes used in place of beta (Problem::beta32)
};

// Workspace (fp32), G = total chunks:  T [G][n][n]  W [G][n][d_k]  U [G][n][d_v]  P [G][C][n]
struct Ws {
    float* T;
    float* W;
    float* U;
    float* P;
    double* D;      // wu_builder 1 only: [G][3][cells_max][r][d_k + d_v], three antidiagonals of the two-index system
};

// ------------------------------------------------------------------------------------------
// 64 x BN tile GEMM for one CTA of 256 threads; thread (ty, tx) owns rows ty*4..+3 and
// BN/16 columns.  fa(mm, kk) = A[m0+mm][kk], fb(kk, nn) = B[kk][n0+nn]; both must return 0
// outside their valid range.  A_KFAST picks the loader order that makes fa's global reads coalesced.
// ------------------------------------------------------------------------------------------
constexpr int TK = 16;
constexpr int TM = 64;

template <int BN, bool A_KFAST, class FA, class FB>
__device__ __forceinline__ void tile_gemm(float (&acc)[4][BN / 16], int kbeg, int kend, FA fa, FB fb,
                                          float* As /*[TK][TM+4]*/, float* Bs /*[TK][BN+4]*/) {
    constexpr int TN = BN / 16;
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    for (int k0 = kbeg; k0 < kend; k0 += TK) {
        __syncthreads();
#pragma unroll
        for (int e = tid; e < TK * TM; e += 256) {
            int mm, kk;
            if (A_KFAST) { mm = e / TK; kk = e % TK; } else { kk = e / TM; mm = e % TM; }
            As[kk * (TM + 4) + mm] = (k0 + kk < kend) ? fa(mm, k0 + kk) : 0.f;
        }
#pragma unroll
        for (int e = tid; e < TK * BN; e += 256) {
            int kk = e / BN, nn = e % BN;
            Bs[kk * (BN + 4) + nn] = (k0 + kk < kend) ? fb(k0 + kk, nn) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            float a[4], b[TN];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk * (TM + 4) + ty * 4 + i];
#pragma unroll
            for (int j = 0; j < TN; ++j) b[j] = Bs[kk * (BN + 4) + tx * TN + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
    }
}

template <int TN> __device__ __forceinline__ void zero_acc(float (&acc)[4][TN]) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;
}

// ------------------------------------------------------------------------------------------
// simt_gram: one CTA per chunk.
// ------------------------------------------------------------------------------------------
template <class Tin>
__global__ void __launch_bounds__(256) simt_gram(const Tin* __restrict__ q, const Tin* __restrict__ k,
                                                 const Tin* __restrict__ beta, Geo g, Ws ws) {
    __shared__ float As[TK * (TM + 4)];
    __shared__ float Bs[TK * (64 + 4)];
    const long long gc = blockIdx.x;
    const long long seq = gc / g.NC;
    const int c = (int)(gc % g.NC);
    const int t0 = c * g.C;
    const int Cv = min(g.C, g.L - t0);
    const int nv = Cv * g.r;
    const int n = g.n, r = g.r, d_k = g.d_k;
    const Tin* Kc = k + ((seq * g.L + t0) * r) * (long long)d_k;
    const Tin* Qc = q + (seq * g.L + t0) * (long long)d_k;
    const Tin* bc = beta + (seq * g.L + t0) * (long long)r;
    float* Tg = ws.T + gc * (long long)n * n;
    float* Pg = ws.P + gc * (long long)g.C * n;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;

    // A[m][m'] = beta_m (k_m . k_m') for tok(m') < tok(m) (product form: m' < m), else 0
    for (int m0 = 0; m0 < n; m0 += TM)
        for (int n0 = 0; n0 < n; n0 += 64) {
            float acc[4][4];
            zero_acc(acc);
            if (n0 < m0 + TM) {   // tiles entirely above the diagonal stay zero
                auto fa = [&](int mm, int kk) { return (m0 + mm < nv) ? ldf(Kc + (long long)(m0 + mm) * d_k + kk) : 0.f; };
                auto fb = [&](int kk, int nn) { return (n0 + nn < nv) ? ldf(Kc + (long long)(n0 + nn) * d_k + kk) : 0.f; };
                tile_gemm<64, true>(acc, 0, d_k, fa, fb, As, Bs);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int m = m0 + ty * 4 + i;
                if (m >= n) continue;
                const float bm = (m < nv) ? (g.b32 ? g.b32[(seq * g.L + t0) * (long long)r + m] : ldf(bc + m)) : 0.f;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int mp = n0 + tx * 4 + j;
                    if (mp >= n) continue;
                    Tg[(long long)m * n + mp] = (mp / g.rm < m / g.rm) ? bm * acc[i][j] : 0.f;
                }
            }
        }

    // P[t][m] = q_t . k_m for tok(m) <= t, else 0
    for (int m0 = 0; m0 < g.C; m0 += TM)
        for (int n0 = 0; n0 < n; n0 += 64) {
            float acc[4][4];
            zero_acc(acc);
            auto fa = [&](int mm, int kk) { return (m0 + mm < Cv) ? ldf(Qc + (long long)(m0 + mm) * d_k + kk) : 0.f; };
            auto fb = [&](int kk, int nn) { return (n0 + nn < nv) ? ldf(Kc + (long long)(n0 + nn) * d_k + kk) : 0.f; };
            tile_gemm<64, true>(acc, 0, d_k, fa, fb, As, Bs);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int t = m0 + ty * 4 + i;
                if (t >= g.C) continue;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int m = n0 + tx * 4 + j;
                    if (m >= n) continue;
                    Pg[(long long)t * n + m] = (m / r <= t) ? acc[i][j] : 0.f;
                }
            }
        }
}

// ------------------------------------------------------------------------------------------
// simt_solve: one CTA per chunk, thread c owns column c of X = (I + A)^{-1} diag(beta):
//   X[c][c] = beta_c,   X[m][c] = - sum_{m' = c}^{first row of tok(m) - 1} A[m][m'] X[m'][c]   (m > c)
// A thread only ever reads its own column, so no synchronisation is needed between rows; rows of
// A are staged through shared memory RB at a time.  X is kept as a packed lower triangle.
// ------------------------------------------------------------------------------------------
constexpr int RB = 16;

template <class Tin>
__global__ void simt_solve(const Tin* __restrict__ beta, Geo g, Ws ws) {
    extern __shared__ float sm[];
    const int n = g.n, r = g.r;
    float* Xt = sm;                                  // packed: row m at m(m+1)/2
    float* Ar = sm + (size_t)n * (n + 1) / 2;        // [RB][n]
    const long long gc = blockIdx.x;
    const long long seq = gc / g.NC;
    const int ci = (int)(gc % g.NC);
    const int t0 = ci * g.C;
    const int nv = min(g.C, g.L - t0) * r;
    const Tin* bc = beta + (seq * g.L + t0) * (long long)r;
    float* Tg = ws.T + gc * (long long)n * n;
    const int c = threadIdx.x;
    const float bcol = (c < nv) ? (g.b32 ? g.b32[(seq * g.L + t0) * (long long)r + c] : ldf(bc + c)) : 0.f;
    const int wstart = (c / 32) * 32;                // first column of this warp: warp-uniform loop start

    for (int m0 = 0; m0 < n; m0 += RB) {
        __syncthreads();
        for (int e = threadIdx.x; e < RB * n; e += blockDim.x) {
            const int mm = e / n, mp = e % n;
            Ar[e] = (m0 + mm < n) ? Tg[(long long)(m0 + mm) * n + mp] : 0.f;
        }
        __syncthreads();
        for (int mm = 0; mm < RB; ++mm) {
            const int m = m0 + mm;
            if (m >= n || m < wstart) continue;      // whole warp above the diagonal
            const int lim = (m / g.rm) * g.rm;       // rows of the same token do not interact (sum form)
            float acc = 0.f;
            for (int mp = wstart; mp < lim; ++mp) {
                const float a = Ar[mm * n + mp];                              // broadcast
                const float x = (mp >= c && c <= m) ? Xt[(size_t)mp * (mp + 1) / 2 + c] : 0.f;
                acc = fmaf(a, x, acc);
            }
            if (c <= m) Xt[(size_t)m * (m + 1) / 2 + c] = (c == m) ? bcol : -acc;
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < n * n; e += blockDim.x) {
        const int m = e / n, cc = e % n;
        Tg[e] = (cc <= m) ? Xt[(size_t)m * (m + 1) / 2 + cc] : 0.f;
    }
}

// ------------------------------------------------------------------------------------------
// simt_wu: one CTA per chunk:  [W | Uh] = T' [K | V]   (T' lower triangular: k-range stops at the tile)
// ------------------------------------------------------------------------------------------
template <class Tin>
__global__ void __launch_bounds__(256) simt_wu(const Tin* __restrict__ k, const Tin* __restrict__ v, Geo g, Ws ws) {
    __shared__ float As[TK * (TM + 4)];
    __shared__ float Bs[TK * (64 + 4)];
    const long long gc = blockIdx.x;
    const long long seq = gc / g.NC;
    const int c = (int)(gc % g.NC);
    const int t0 = c * g.C;
    const int nv = min(g.C, g.L - t0) * g.r;
    const int n = g.n, d_k = g.d_k, d_v = g.d_v;
    const Tin* Kc = k + ((seq * g.L + t0) * g.r) * (long long)d_k;
    const Tin* Vc = v + ((seq * g.L + t0) * g.r) * (long long)d_v;
    const float* Tg = ws.T + gc * (long long)n * n;
    float* Wg = ws.W + gc * (long long)n * d_k;
    float* Ug = ws.U + gc * (long long)n * d_v;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;

    for (int m0 = 0; m0 < n; m0 += TM) {
        const int kend = min(n, m0 + TM);
        auto fa = [&](int mm, int kk) { return (m0 + mm < n) ? Tg[(long long)(m0 + mm) * n + kk] : 0.f; };
        for (int n0 = 0; n0 < d_k + d_v; n0 += 64) {
            float acc[4][4];
            zero_acc(acc);
            const bool isK = n0 < d_k;
            const Tin* src = isK ? Kc : Vc;
            const int ld = isK ? d_k : d_v;
            const int col0 = isK ? n0 : n0 - d_k;
            auto fb = [&](int kk, int nn) { return (kk < nv) ? ldf(src + (long long)kk * ld + col0 + nn) : 0.f; };
            tile_gemm<64, true>(acc, 0, kend, fa, fb, As, Bs);
            float* dst = isK ? Wg : Ug;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int m = m0 + ty * 4 + i;
                if (m >= n) continue;
#pragma unroll
                for (int j = 0; j < 4; ++j) dst[(long long)m * ld + col0 + tx * 4 + j] = acc[i][j];
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// simt_scan: one CTA per (sequence, 32-wide slice of d_v); the state slice St[i][j] = S[j0+j][i]
// lives in shared memory for the whole sequence.
// ------------------------------------------------------------------------------------------
constexpr int DVS = 32;

template <class Tin>
__global__ void __launch_bounds__(256) simt_scan(const Tin* __restrict__ q, const Tin* __restrict__ k,
                                                 const float* __restrict__ S0, float* __restrict__ O,
                                                 float* __restrict__ S_final, Geo g, Ws ws) {
    extern __shared__ float sm[];
    const int n = g.n, d_k = g.d_k, d_v = g.d_v, r = g.r;
    float* St = sm;                           // [d_k][DVS]
    float* Up = St + d_k * DVS;               // [n][DVS]
    float* As = Up + n * DVS;                 // [TK][TM+4]
    float* Bs = As + TK * (TM + 4);           // [TK][DVS+4]
    const int slices = d_v / DVS;
    const long long seq = blockIdx.x / slices;
    const int j0 = (int)(blockIdx.x % slices) * DVS;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    constexpr int TN = DVS / 16;

    for (int e = threadIdx.x; e < d_k * DVS; e += 256) {
        const int i = e / DVS, j = e % DVS;
        St[e] = S0 ? S0[(seq * d_k + i) * (long long)d_v + j0 + j] : 0.f;
    }
    __syncthreads();

    for (int c = 0; c < g.NC; ++c) {
        const long long gc = seq * g.NC + c;
        const int t0 = c * g.C;
        const int Cv = min(g.C, g.L - t0);
        const int nv = Cv * r;
        const Tin* Kc = k + ((seq * g.L + t0) * r) * (long long)d_k;
        const Tin* Qc = q + (seq * g.L + t0) * (long long)d_k;
        const float* Wg = ws.W + gc * (long long)n * d_k;
        const float* Ug = ws.U + gc * (long long)n * d_v;
        const float* Pg = ws.P + gc * (long long)g.C * n;
        auto fS = [&](int kk, int nn) { return St[kk * DVS + nn]; };
        auto fUp = [&](int kk, int nn) { return Up[kk * DVS + nn]; };

        // U' = Uh - W S^T     (rows past nv: W = Uh = 0, so U' = 0)
        for (int m0 = 0; m0 < n; m0 += TM) {
            float acc[4][TN];
            zero_acc(acc);
            auto fa = [&](int mm, int kk) { return (m0 + mm < n) ? Wg[(long long)(m0 + mm) * d_k + kk] : 0.f; };
            tile_gemm<DVS, true>(acc, 0, d_k, fa, fS, As, Bs);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int m = m0 + ty * 4 + i;
                if (m >= n) continue;
#pragma unroll
                for (int j = 0; j < TN; ++j) {
                    const int jj = tx * TN + j;
                    Up[m * DVS + jj] = Ug[(long long)m * d_v + j0 + jj] - acc[i][j];
                }
            }
        }
        __syncthreads();

        // O = Q S^T + P U'
        for (int m0 = 0; m0 < g.C; m0 += TM) {
            float acc[4][TN];
            zero_acc(acc);
            auto fq = [&](int mm, int kk) { return (m0 + mm < Cv) ? ldf(Qc + (long long)(m0 + mm) * d_k + kk) : 0.f; };
            tile_gemm<DVS, true>(acc, 0, d_k, fq, fS, As, Bs);
            auto fp = [&](int mm, int kk) { return (m0 + mm < g.C) ? Pg[(long long)(m0 + mm) * n + kk] : 0.f; };
            tile_gemm<DVS, true>(acc, 0, n, fp, fUp, As, Bs);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int t = m0 + ty * 4 + i;
                if (t >= Cv) continue;
#pragma unroll
                for (int j = 0; j < TN; ++j)
                    O[(seq * g.L + t0 + t) * (long long)d_v + j0 + tx * TN + j] = acc[i][j];
            }
        }
        __syncthreads();   // every read of the old state is done

        // S^T += K^T U'
        for (int m0 = 0; m0 < d_k; m0 += TM) {
            float acc[4][TN];
            zero_acc(acc);
            auto fk = [&](int mm, int kk) { return (kk < nv) ? ldf(Kc + (long long)kk * d_k + m0 + mm) : 0.f; };
            tile_gemm<DVS, false>(acc, 0, n, fk, fUp, As, Bs);
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) St[(m0 + ty * 4 + i) * DVS + tx * TN + j] += acc[i][j];
        }
        __syncthreads();
    }

    if (S_final)
        for (int e = threadIdx.x; e < d_k * DVS; e += 256) {
            const int i = e / DVS, j = e % DVS;
            S_final[(seq * d_k + i) * (long long)d_v + j0 + j] = St[e];
        }
}

// ------------------------------------------------------------------------------------------
// simt_sigdelta: one CTA per chunk.  Theorem 3.3: the solution W_{t_k} of
//     W_{t_k} = A_{t_k} + sum_{m<k} W_{t_m} B_{t_m}^T A_{t_k}
// is the diagonal W(t_k, t_k) of the system
//     W(t_0, t_k) = A_{t_k},
//     W(t_{k+1}, t_{k+1}) = W(t_k, t_{k+1}) + W(t_k, t_k) B_{t_k}^T A_{t_{k+1}},
//     W(t_{m+1}, t_{k+1}) = W(t_m, t_{k+1}) + W(t_{m+1}, t_k) - W(t_m, t_k) + W(t_m, t_m) B_{t_m}^T (A_{t_{k+1}} - A_{t_k})   (m < k).
// A cell (m, k), m <= k, holds the R rows of token k (d_k values of W, then d_v values of the same system driven by
// V, which gives Uh).  Cells with the same m + k do not depend on each other: the grid is swept antidiagonal by
// antidiagonal (2C - 1 steps), all cells of one antidiagonal at once, with the two previous antidiagonals kept in
// global memory (L2).  In the row notation used here  A_{t_k} -> rows beta_m k_m,  and the R x R coefficients
// B_{t_m}^T A_{t_k} are, up to sign, the entries A[(k,j)][(m,i)] = beta_(k,j) k_(k,j).k_(m,i) that simt_gram left in T.
// Product form: the same system with every row a token of its own (C*r tokens, R = 1).
// The cells are kept in fp64: each update adds two neighbours and subtracts a third, all of the size of the result,
// 2C - 1 times in a row, and in fp32 that alone costs 2e-5 of max|O| at 256 rows, more than the fp32 entry point is
// allowed in total.  Inputs, coefficients and the finished rows of W and Uh stay fp32.
// ------------------------------------------------------------------------------------------
template <class Tin>
__global__ void __launch_bounds__(256) simt_sigdelta(const Tin* __restrict__ k, const Tin* __restrict__ v,
                                                     const Tin* __restrict__ beta, Geo g, Ws ws, int cells_max) {
    const long long gc = blockIdx.x;
    const long long seq = gc / g.NC;
    const int ci = (int)(gc % g.NC);
    const int t0 = ci * g.C;
    const int n = g.n, d_k = g.d_k, d_v = g.d_v, DT = g.d_k + g.d_v;
    const int nv = min(g.C, g.L - t0) * g.r;
    const int R = g.rm;                 // rows per token of the system: r (sum form) or 1 (product form)
    const int CT = n / R;               // tokens of the system
    const Tin* Kc = k + ((seq * g.L + t0) * g.r) * (long long)d_k;
    const Tin* Vc = v + ((seq * g.L + t0) * g.r) * (long long)d_v;
    const Tin* bc = beta + (seq * g.L + t0) * (long long)g.r;
    const float* Tg = ws.T + gc * (long long)n * n;
    float* Wg = ws.W + gc * (long long)n * d_k;
    float* Ug = ws.U + gc * (long long)n * d_v;
    double* Dg = ws.D + gc * 3ll * cells_max * R * DT;
    const long long dstride = (long long)cells_max * R * DT;
    auto m_lo = [&](int s) { return max(0, s - (CT - 1)); };

    for (int s = 0; s <= 2 * (CT - 1); ++s) {
        const int lo = m_lo(s), hi = s >> 1;
        const int total = (hi - lo + 1) * R * DT;
        double* Ds = Dg + (s % 3) * dstride;
        const double* D1 = Dg + ((s + 2) % 3) * dstride;    // antidiagonal s - 1
        const double* D2 = Dg + ((s + 1) % 3) * dstride;    // antidiagonal s - 2
        const int lo1 = m_lo(s - 1), lo2 = m_lo(s - 2);
        for (int e = threadIdx.x; e < total; e += 256) {
            const int x = e % DT;
            const int j = (e / DT) % R;
            const int m = lo + e / (DT * R);
            const int kk = s - m;
            const int row = kk * R + j;
            double val;
            if (m == 0) {
                float b = 0.f, a = 0.f;
                if (row < nv) {
                    b = g.b32 ? g.b32[(seq * g.L + t0) * (long long)g.r + row] : ldf(bc + row);
                    a = (x < d_k) ? ldf(Kc + (long long)row * d_k + x) : ldf(Vc + (long long)row * d_v + (x - d_k));
                }
                val = (double)(b * a);                                          // W(t_0, t_k) = A_{t_k}
            } else {
                const float* fin = (x < d_k) ? (Wg + (long long)(m - 1) * R * d_k + x) : (Ug + (long long)(m - 1) * R * d_v + (x - d_k));
                const int fstride = (x < d_k) ? d_k : d_v;
                const long long c1 = ((long long)(m - 1 - lo1) * R + j) * DT + x;            // (m-1, k)   on s - 1
                double acc = 0.0;
                if (m == kk) {
                    val = D1[c1];
                    for (int i = 0; i < R; ++i)
                        acc += (double)(fin[(long long)i * fstride] * Tg[(long long)row * n + (m - 1) * R + i]);
                } else {
                    const long long c2 = ((long long)(m - lo1) * R + j) * DT + x;            // (m, k-1)   on s - 1
                    const long long c3 = ((long long)(m - 1 - lo2) * R + j) * DT + x;        // (m-1, k-1) on s - 2
                    val = D1[c1] + D1[c2] - D2[c3];
                    for (int i = 0; i < R; ++i)
                        acc += (double)fin[(long long)i * fstride] *
                               ((double)Tg[(long long)row * n + (m - 1) * R + i] - (double)Tg[(long long)(row - R) * n + (m - 1) * R + i]);
                }
                val -= acc;
            }
            Ds[((long long)(m - lo) * R + j) * DT + x] = val;
            if (m == kk) {                                                      // diagonal cell: W_{t_k} itself
                if (x < d_k) Wg[(long long)row * d_k + x] = (float)val;
                else Ug[(long long)row * d_v + (x - d_k)] = (float)val;
            }
        }
        __syncthreads();
    }
}

// cells on the longest antidiagonal of the two-index system
int sigdelta_cells_max(const Problem& p) { return (p.n() / p.mask_group()) / 2 + 1; }
size_t sigdelta_bytes(const Problem& p) {
    if (!p.wu_builder) return 0;
    return align_up((size_t)p.total_chunks() * 3 * sigdelta_cells_max(p) * p.mask_group() * (p.d_k + p.d_v) * sizeof(double), 256);
}

Ws carve(const Problem& p, void* workspace) {
    const size_t G = (size_t)p.total_chunks();
    const size_t n = p.n();
    char* base = (char*)workspace;
    Ws ws;
    ws.T = (float*)base;
    base += align_up(G * n * n * sizeof(float), 256);
    ws.W = (float*)base;
    base += align_up(G * n * p.d_k * sizeof(float), 256);
    ws.U = (float*)base;
    base += align_up(G * n * p.d_v * sizeof(float), 256);
    ws.P = (float*)base;
    base += align_up(G * (size_t)p.chunk * n * sizeof(float), 256);
    ws.D = p.wu_builder ? (double*)base : nullptr;
    return ws;
}

template <class Tin>
int run(const Problem& p, void* workspace, bool prepare_only) {
    Geo g{p.L, p.d_k, p.d_v, p.r, p.chunk, p.n(), p.chunks_per_seq(), p.mask_group(), p.beta32};
    const long long G = p.total_chunks();
    const long long nseq = (long long)p.B * p.H;
    const Tin* q = (const Tin*)p.q;
    const Tin* k = (const Tin*)p.k;
    const Tin* v = (const Tin*)p.v;
    const Tin* beta = (const Tin*)p.beta;
    Ws ws = carve(p, workspace);
    const size_t scan_smem = sizeof(float) * ((size_t)p.d_k * DVS + (size_t)g.n * DVS + TK * (TM + 4) + TK * (DVS + 4));
    const size_t solve_smem = sizeof(float) * ((size_t)g.n * (g.n + 1) / 2 + (size_t)RB * g.n);
    PF_CUDA_TRY(cudaFuncSetAttribute(simt_solve<Tin>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)solve_smem));
    PF_CUDA_TRY(cudaFuncSetAttribute(simt_scan<Tin>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)scan_smem));
    int launches = 0;
    if (G > 0) {
        if (G > 0x7fffffffLL) return PF_ERR_UNSUPPORTED;
        prof_begin("simt_gram", p.stream);
        simt_gram<Tin><<<(unsigned)G, 256, 0, p.stream>>>(q, k, beta, g, ws);
        prof_end(p.stream);
        if (p.wu_builder) {
            prof_begin("simt_sigdelta", p.stream);
            simt_sigdelta<Tin><<<(unsigned)G, 256, 0, p.stream>>>(k, v, beta, g, ws, sigdelta_cells_max(p));
            prof_end(p.stream);
            launches += 2;
        } else {
            prof_begin("simt_solve", p.stream);
            simt_solve<Tin><<<(unsigned)G, g.n, solve_smem, p.stream>>>(beta, g, ws);
            prof_end(p.stream);
            prof_begin("simt_wu", p.stream);
            simt_wu<Tin><<<(unsigned)G, 256, 0, p.stream>>>(k, v, g, ws);
            prof_end(p.stream);
            launches += 3;
        }
    }
    if (prepare_only) {
        PF_CUDA_TRY(cudaGetLastError());
        count_launch(launches);
        return PF_OK;
    }
    // With L = 0 the scan still runs: it copies S0 to S_final.
    prof_begin("simt_scan", p.stream);
    simt_scan<Tin><<<(unsigned)(nseq * (p.d_v / DVS)), 256, scan_smem, p.stream>>>(q, k, p.S0, p.O, p.S_final, g, ws);
    prof_end(p.stream);
    launches += 1;
    PF_CUDA_TRY(cudaGetLastError());
    count_launch(launches);
    return PF_OK;
}

}  // namespace

size_t simt_workspace_bytes(const Problem& p) {
    const size_t G = (size_t)p.total_chunks();
    const size_t n = p.n();
    return align_up(G * n * n * sizeof(float), 256) + align_up(G * n * p.d_k * sizeof(float), 256) +
           align_up(G * n * p.d_v * sizeof(float), 256) + align_up(G * (size_t)p.chunk * n * sizeof(float), 256) +
           sigdelta_bytes(p) + 256;
}

int simt_forward(const Problem& p, void* workspace) {
    if (p.in_dtype == PF_DTYPE_F32) return run<float>(p, workspace, false);
    return run<__nv_bfloat16>(p, workspace, false);
}

int simt_prepare(const Problem& p, void* workspace, float** W, float** U, float** P) {
    Ws ws = carve(p, workspace);
    *W = ws.W;
    *U = ws.U;
    *P = ws.P;
    if (p.in_dtype == PF_DTYPE_F32) return run<float>(p, workspace, true);
    return run<__nv_bfloat16>(p, workspace, true);
}

}  // namespace pf
