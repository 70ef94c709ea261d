/*
 * pf_oracle.c -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, fp64 CPU evaluation of the generalized rank-r delta-rule recurrence, token by
 * token, exactly as the paper defines it.  Nothing here is chunked, blocked, fused or reordered;
 * there is no W/U compact form and no triangular solve.  Only tests, the smoke check and the
 * bench's cpu_baseline leg may call it.  It shares no code with the CUDA path.
 *
 * What it computes, per (batch b, head h), with S in R^{d_v x d_k}:
 *
 *     S_t = S_{t-1} (I - sum_j beta_{t,j} k_{t,j} k_{t,j}^T) + sum_j beta_{t,j} v_{t,j} k_{t,j}^T
 *     o_t = S_t q_t
 *
 * Sources: the (recurrence) / (memory readout) pair of Section 1.1 gives S_t = S_{t-1} <> A_t +
 * v_t k_t^T and o_t = S_t q_t (readout uses the state AFTER token t's update); the (DeltaNet)
 * equation of Section 1.3 gives the rank-1 delta rule; Eq. (discretization) of Section 3.1 with
 * the R=1 Remark generalised to R columns (A_t = K_t diag(beta_t), A~_t = -V_t diag(beta_t),
 * B_t = -K_t) turns the discrete step  S_{k+1} = S_k + S_k A_k B_k^T + A~_k B_k^T  into the line
 * above.  All r factors of a token read the SAME old state (diagonal R x R blocks of
 * Id - M (.) A B^T are the identity, proof of Theorem 3.2), i.e. the "sum" form.
 *
 * A second entry point evaluates the PRODUCT form, in which the r factors of a token act one after
 * another, each on the state the previous one left:
 *
 *     S_t = S_{t-1} prod_j (I - beta_{t,j} k_{t,j} k_{t,j}^T)  + (the matching v terms),
 *
 * i.e. the rank-1 delta rule of Section 1.3 applied r times per token (the same thing as rank-1
 * DeltaNet on the length L*r sequence of factors, read out after every r-th step).  In the chunk form
 * of Theorem 3.2 this is the general block-triangular case, with the mask strict in the flattened
 * row index instead of the time index.
 *
 * Both forms can also take the EXACT step of a rank-1 factor instead of the Euler step.  The subsection
 * "An alternative representation of the flow as product of exponentials" replaces Id + dw by exp(dw)
 * and gives, for rank 1,  exp(a b^T) = Id + ((e^{<b,a>} - 1) / <b,a>) a b^T  (the printed fraction has the
 * "- 1" inside the exponent; the power series two lines above it fixes the reading).  With a = beta k,
 * b = -k this is  exp(-beta k k^T) = Id - beta' k k^T,  beta' = (1 - e^{-beta |k|^2}) / |k|^2.  The paper
 * treats only the homogeneous part; solving the same linear equation over the step with the constant
 * input beta v k^T gives the same factor on the input term, so the exact step is the delta rule with beta'
 * in place of beta.  It needs rank-1 factors: r = 1, or the product form with any r.
 *
 * Every pin that ties this file to something other than itself is in tests/test_oracle_pins.py.
 *
 * Layouts (all row-major, host memory):
 *     q    [B,H,L,d_k]     float   (the exact input values the GPU receives, bf16 or fp32, widened)
 *     k    [B,H,L,r,d_k]   float
 *     v    [B,H,L,r,d_v]   float
 *     beta [B,H,L,r]       float
 *     S0   [B,H,d_k,d_v]   double or NULL (zeros);  S0[b,h,i,j] = S[j][i]
 *     O    [B,H,L,d_v]     double
 *     S_final [B,H,d_k,d_v] double or NULL
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* One sequence.  S is kept as S[j*d_k + i], j in [0,d_v), i in [0,d_k). */
static void pf_oracle_one_sequence(const float* q, const float* k, const float* v, const float* beta,
                                   const double* beta_eff, /* NULL, or step sizes that replace beta */
                                   const double* S0, int L, int d_k, int d_v, int r,
                                   double* O, double* S_final, double* S, double* p)
{
    for (int j = 0; j < d_v; ++j)
        for (int i = 0; i < d_k; ++i)
            S[(size_t)j * d_k + i] = S0 ? S0[(size_t)i * d_v + j] : 0.0;

    for (int t = 0; t < L; ++t) {
        const float* kt = k + (size_t)t * r * d_k;
        const float* vt = v + (size_t)t * r * d_v;
        const float* bt = beta + (size_t)t * r;

        /* predictions p_f = S_{t-1} k_{t,f} for every factor f, all from the old state */
        for (int f = 0; f < r; ++f)
            for (int j = 0; j < d_v; ++j) {
                double acc = 0.0;
                for (int i = 0; i < d_k; ++i)
                    acc += S[(size_t)j * d_k + i] * (double)kt[(size_t)f * d_k + i];
                p[(size_t)f * d_v + j] = acc;
            }

        /* S_t = S_{t-1} + sum_f beta_f (v_f - p_f) k_f^T */
        for (int f = 0; f < r; ++f) {
            double b = beta_eff ? beta_eff[(size_t)t * r + f] : (double)bt[f];
            for (int j = 0; j < d_v; ++j) {
                double e = b * ((double)vt[(size_t)f * d_v + j] - p[(size_t)f * d_v + j]);
                for (int i = 0; i < d_k; ++i)
                    S[(size_t)j * d_k + i] += e * (double)kt[(size_t)f * d_k + i];
            }
        }

        /* o_t = S_t q_t */
        const float* qt = q + (size_t)t * d_k;
        for (int j = 0; j < d_v; ++j) {
            double acc = 0.0;
            for (int i = 0; i < d_k; ++i)
                acc += S[(size_t)j * d_k + i] * (double)qt[i];
            O[(size_t)t * d_v + j] = acc;
        }
    }

    if (S_final)
        for (int j = 0; j < d_v; ++j)
            for (int i = 0; i < d_k; ++i)
                S_final[(size_t)i * d_v + j] = S[(size_t)j * d_k + i];
}

/* One sequence, product form: factor f reads the state factor f-1 left (rank-1 delta rule, r times). */
static void pf_oracle_one_sequence_product(const float* q, const float* k, const float* v, const float* beta,
                                           const double* beta_eff,
                                           const double* S0, int L, int d_k, int d_v, int r,
                                           double* O, double* S_final, double* S, double* p)
{
    for (int j = 0; j < d_v; ++j)
        for (int i = 0; i < d_k; ++i)
            S[(size_t)j * d_k + i] = S0 ? S0[(size_t)i * d_v + j] : 0.0;

    for (int t = 0; t < L; ++t) {
        for (int f = 0; f < r; ++f) {
            const float* kf = k + ((size_t)t * r + f) * d_k;
            const float* vf = v + ((size_t)t * r + f) * d_v;
            const double b = beta_eff ? beta_eff[(size_t)t * r + f] : (double)beta[(size_t)t * r + f];
            /* prediction from the CURRENT state, then S <- S + beta (v - S k) k^T */
            for (int j = 0; j < d_v; ++j) {
                double acc = 0.0;
                for (int i = 0; i < d_k; ++i)
                    acc += S[(size_t)j * d_k + i] * (double)kf[i];
                p[j] = acc;
            }
            for (int j = 0; j < d_v; ++j) {
                double e = b * ((double)vf[j] - p[j]);
                for (int i = 0; i < d_k; ++i)
                    S[(size_t)j * d_k + i] += e * (double)kf[i];
            }
        }
        /* o_t = S_t q_t, after the token's last factor */
        const float* qt = q + (size_t)t * d_k;
        for (int j = 0; j < d_v; ++j) {
            double acc = 0.0;
            for (int i = 0; i < d_k; ++i)
                acc += S[(size_t)j * d_k + i] * (double)qt[i];
            O[(size_t)t * d_v + j] = acc;
        }
    }

    if (S_final)
        for (int j = 0; j < d_v; ++j)
            for (int i = 0; i < d_k; ++i)
                S_final[(size_t)i * d_v + j] = S[(size_t)j * d_k + i];
}

/* Returns 0 on success, -1 on a bad argument, -2 on allocation failure.
 * num_threads <= 0 means "whatever OpenMP picks"; sequences (b,h) are independent, and that is the
 * only parallelism used.  *threads_used (may be NULL) receives the thread count actually used. */
/* beta' = (1 - e^{-beta |k|^2}) / |k|^2 for every factor (rows of k); beta itself where k = 0 (the limit). */
static void pf_oracle_exact_steps(const float* k, const float* beta, size_t rows, int d_k, double* out)
{
    for (size_t m = 0; m < rows; ++m) {
        double s = 0.0;
        for (int i = 0; i < d_k; ++i)
            s += (double)k[m * d_k + i] * (double)k[m * d_k + i];
        const double b = (double)beta[m];
        out[m] = s > 0.0 ? -expm1(-b * s) / s : b;
    }
}

static int pf_oracle_run(int product, int exact, const float* q, const float* k, const float* v, const float* beta,
                         const double* S0, int B, int H, int L, int d_k, int d_v, int r,
                         double* O, double* S_final, int num_threads, int* threads_used)
{
    if (!q || !k || !v || !beta || !O) return -1;
    if (B < 1 || H < 1 || L < 0 || d_k < 1 || d_v < 1 || r < 1) return -1;
    if (exact && !product && r != 1) return -1;      /* the exact step is defined for rank-1 factors */
    const int nseq = B * H;
    double* beta_eff = NULL;
    if (exact) {
        const size_t rows = (size_t)nseq * L * r;
        beta_eff = (double*)malloc(sizeof(double) * (rows ? rows : 1));
        if (!beta_eff) return -2;
        pf_oracle_exact_steps(k, beta, rows, d_k, beta_eff);
    }
    int nt = 1;
#ifdef _OPENMP
    nt = num_threads > 0 ? num_threads : omp_get_max_threads();
    if (nt > nseq) nt = nseq;
    if (nt < 1) nt = 1;
#else
    (void)num_threads;
#endif
    if (threads_used) *threads_used = nt;
    int failed = 0;

#ifdef _OPENMP
#pragma omp parallel num_threads(nt)
#endif
    {
        double* S = (double*)malloc(sizeof(double) * (size_t)d_v * d_k);
        double* p = (double*)malloc(sizeof(double) * (size_t)r * d_v);
        if (!S || !p) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            failed = 1;
        } else {
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
            for (int s = 0; s < nseq; ++s) {
                (product ? pf_oracle_one_sequence_product : pf_oracle_one_sequence)(
                                       q + (size_t)s * L * d_k,
                                       k + (size_t)s * L * r * d_k,
                                       v + (size_t)s * L * r * d_v,
                                       beta + (size_t)s * L * r,
                                       beta_eff ? beta_eff + (size_t)s * L * r : NULL,
                                       S0 ? S0 + (size_t)s * d_k * d_v : NULL,
                                       L, d_k, d_v, r,
                                       O + (size_t)s * L * d_v,
                                       S_final ? S_final + (size_t)s * d_k * d_v : NULL,
                                       S, p);
            }
        }
        free(S);
        free(p);
    }
    free(beta_eff);
    return failed ? -2 : 0;
}

int pf_oracle_deltanet_fwd_f64(const float* q, const float* k, const float* v, const float* beta,
                               const double* S0, int B, int H, int L, int d_k, int d_v, int r,
                               double* O, double* S_final, int num_threads, int* threads_used)
{
    return pf_oracle_run(0, 0, q, k, v, beta, S0, B, H, L, d_k, d_v, r, O, S_final, num_threads, threads_used);
}

/* Product form (see the header): same arguments, same layouts, same return codes. */
int pf_oracle_deltanet_product_fwd_f64(const float* q, const float* k, const float* v, const float* beta,
                                       const double* S0, int B, int H, int L, int d_k, int d_v, int r,
                                       double* O, double* S_final, int num_threads, int* threads_used)
{
    return pf_oracle_run(1, 0, q, k, v, beta, S0, B, H, L, d_k, d_v, r, O, S_final, num_threads, threads_used);
}

/* Either form with the exact rank-1 step (see the header).  product: 0 = sum form (needs r = 1), 1 = product
 * form.  Same arguments, layouts and return codes otherwise. */
int pf_oracle_deltanet_exact_fwd_f64(int product, const float* q, const float* k, const float* v, const float* beta,
                                     const double* S0, int B, int H, int L, int d_k, int d_v, int r,
                                     double* O, double* S_final, int num_threads, int* threads_used)
{
    return pf_oracle_run(product ? 1 : 0, 1, q, k, v, beta, S0, B, H, L, d_k, d_v, r, O, S_final, num_threads,
                         threads_used);
}
