/*
 * pf.h -- C ABI of the chunkwise-parallel forward pass of the rank-r generalized delta rule.
 *
 * The operation (per batch b and head h, state S in R^{d_v x d_k}):
 *
 *     S_t = S_{t-1} (I - sum_j beta_{t,j} k_{t,j} k_{t,j}^T) + sum_j beta_{t,j} v_{t,j} k_{t,j}^T
 *     o_t = S_t q_t                                   (readout after token t's update)
 *
 * This is the associative linear RNN of Section 1.1 (recurrence + memory readout) with the
 * DeltaNet transition of Section 1.3, generalised to rank-R updates by the drivers of Section 3.1,
 * Eq. (discretization):  A_t = K_t diag(beta_t),  A~_t = -V_t diag(beta_t),  B_t = -K_t  (the R=1
 * Remark applied column by column).  All r factors of a token act on the same previous state.
 *
 * It is evaluated chunk by chunk in the "Parallel Flows" order of Section 3 (Chunk -> Parallel
 * Compute -> Scan).  For a chunk of C tokens, rows m = t*r + j, n = C*r, Theorem 3.2 becomes
 *
 *     Lm = I + Mstrict (.) (diag(beta) K K^T),      Mstrict[m,m'] = 1(tok(m') < tok(m))
 *     T' = Lm^{-1} diag(beta),   W = T' K,   Uh = T' V          (compact W/U form of the chunk flow)
 *     U' = Uh - W S^T,           P = (Q K^T) (.) 1(tok(m) <= t)
 *     O  = Q S^T + P U',         S <- S + U'^T K                (= S (I - W^T K) + Uh^T K)
 *
 * Everything behind these entry points runs in CUDA kernels for sm_100a; there is no CPU path.
 *
 * Conventions for every call
 *   - Tensor pointers are DEVICE pointers owned by the caller, dense row-major in the shapes given;
 *     the library neither frees nor keeps them.  q/k/v/beta/O must be 16-byte aligned.
 *   - `stream` is a cudaStream_t (NULL = the default stream).  Work is enqueued; the calls do not
 *     synchronise (pf_read_status and pf_profile_read do).  Unless a workspace is passed through pf_deltanet_fwd_ex, scratch memory is
 *     taken and returned with stream-ordered allocation on `stream`.
 *   - O must not alias an input.  S_final may alias S0.
 *   - Return value: PF_OK (0) or a negative pf_status.  Nothing is launched when an argument check
 *     fails.  No exceptions, no exit().
 *   - Supported shapes: d_k, d_v in {64, 128}; r in {1,2,3,4}; chunk in {16, 32, 64}; any L >= 0
 *     (a ragged last chunk is handled); B, H >= 1.  Anything else returns PF_ERR_UNSUPPORTED --
 *     there is no slow fallback.
 */
#ifndef PF_H_
#define PF_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum pf_status {
    PF_OK = 0,
    PF_ERR_INVALID = -1,      /* null pointer, non-positive size, aliasing */
    PF_ERR_UNSUPPORTED = -2,  /* shape / dtype / impl outside the supported set */
    PF_ERR_ALIGNMENT = -3,    /* a tensor pointer is not 16-byte aligned */
    PF_ERR_ARCH = -4,         /* current device is not compute capability 10.x */
    PF_ERR_CUDA = -5,         /* a CUDA runtime call failed; see pf_last_error_string() */
    PF_ERR_WORKSPACE = -6,    /* caller workspace too small or misaligned */
    PF_ERR_TIMEOUT = -7       /* a bounded device-side wait expired; returned by pf_read_status (see there) */
} pf_status;

enum { PF_DTYPE_BF16 = 0, PF_DTYPE_F32 = 1 };

/* How the r factors of one token combine (pf_params.mode).
 *   PF_MODE_SUM     : all r factors read the same previous state,
 *                         S_t = S_{t-1} (I - sum_j beta_j k_j k_j^T) + sum_j beta_j v_j k_j^T.
 *                     This is the paper's rank-R form (Section 3.1; in the proof of Theorem 3.2 the
 *                     diagonal R x R blocks of Id - M (.) A B^T are the identity) and what every entry
 *                     point without a mode argument computes.
 *   PF_MODE_PRODUCT : the factors act one after another, each on the state the previous one left,
 *                         S_t = S_{t-1} prod_j (I - beta_j k_j k_j^T) + (the matching v terms),
 *                     i.e. the rank-1 delta rule of Section 1.3 applied r times per token, read out after
 *                     the token's last factor.  In the chunk form it is the general block-triangular
 *                     case of Theorem 3.2: Mstrict[m,m'] = 1(m' < m) in the flattened row index; every
 *                     other formula is unchanged.  Every factor is a contraction for beta in [0, 2]. */
enum { PF_MODE_SUM = 0, PF_MODE_PRODUCT = 1 };

/* How one rank-1 factor advances the state (pf_params.step).
 *   PF_STEP_EULER : S <- S (I - beta k k^T) + beta v k^T, the discretisation the paper's chunk algorithms use
 *                   (Eq. (discretization), Section 3.1).  Default.
 *   PF_STEP_EXACT : the exact solution of the same linear equation over the step, from the subsection "An
 *                   alternative representation of the flow as product of exponentials":
 *                       exp(-beta k k^T) = I - beta' k k^T,   beta' = (1 - e^{-beta |k|^2}) / |k|^2,
 *                   and the input term takes the same beta'.  It is the delta rule with beta' in place of beta,
 *                   computed by one extra kernel before the others (fp32, one warp per factor; beta' = beta
 *                   where k = 0).  Defined for rank-1 factors: r = 1, or PF_MODE_PRODUCT with any r; the sum
 *                   form with r > 1 returns PF_ERR_UNSUPPORTED.  beta' < 1/|k|^2, so every factor contracts. */
enum { PF_STEP_EULER = 0, PF_STEP_EXACT = 1 };

/* Which kernels evaluate the chunk form.
 *   PF_IMPL_AUTO : tensor-core path where it supports the shape/dtype, else the fp32 SIMT path.  The result does
 *                  not depend on the chunk length beyond rounding, so AUTO may evaluate with another chunk length
 *                  than the one passed when that puts the problem on the tensor-core kernels, which take up to 128
 *                  rows (chunk * r) per chunk: a chunk with more rows is evaluated as consecutive blocks of whole
 *                  tokens (r = 4 with chunk 64 as blocks of 32 tokens, r = 3 with chunk 64 as blocks of 42), the
 *                  block forward substitution of the chunk's triangular system with the coupling between blocks
 *                  carried by the state; a chunk with fewer than 64 rows is lengthened.  pf_select_chunk tells which
 *                  length is used.  PF_IMPL_TC and PF_IMPL_TC_SPLIT split long chunks into blocks the same way but
 *                  never lengthen a chunk; PF_IMPL_SIMT and PF_IMPL_TC_REFFLOW use `chunk` as given.
 *   PF_IMPL_SIMT : fp32 FFMA kernels (any supported shape; the only path for PF_DTYPE_F32).
 *   PF_IMPL_TC   : tcgen05 tensor-core kernels (bf16 inputs); PF_ERR_UNSUPPORTED otherwise.  For
 *                  d_k = d_v = 128 with at most (SM count - 8) sequences this is ONE cooperative launch in
 *                  which flow-building CTAs and state-scanning CTAs run side by side; other shapes take
 *                  the two-launch form below.  (PF_IMPL_AUTO takes the single launch only up to 0.7 x SM count
 *                  sequences: beyond that too few SMs are left for building flows and two launches are faster.)   */
enum { PF_IMPL_AUTO = 0, PF_IMPL_SIMT = 1, PF_IMPL_TC = 2,
       /* diagnostic: per-chunk flows built by the fp32 SIMT kernels, state scan on tensor cores */
       PF_IMPL_TC_REFFLOW = 3,
       /* tensor-core path as two launches (all flows, then the scan), whatever the shape */
       PF_IMPL_TC_SPLIT = 4 };

/*
 * pf_deltanet_fwd -- the central call: bf16 inputs, fp32 accumulation, fp32 outputs.
 *   q    [B,H,L,d_k]     bf16
 *   k    [B,H,L,r,d_k]   bf16     row (t,j) contiguous
 *   v    [B,H,L,r,d_v]   bf16
 *   beta [B,H,L,r]       bf16
 *   S0   [B,H,d_k,d_v]   fp32 or NULL (zero state);  S0[b,h,i,j] = S[j][i]
 *   O    [B,H,L,d_v]     fp32     (written)
 *   S_final [B,H,d_k,d_v] fp32 or NULL (not wanted)   (written)
 * Defined by: recurrence/readout of Section 1.1, delta rule of Section 1.3, rank-R drivers of
 * Section 3.1, evaluated per chunk through Theorem 3.2 and carried across chunks (Section 3).
 * Value range: the tensor-core kernels round q, k, v, the per-chunk operands derived from them and, once per chunk,
 * the state S to fp16 before each product (fp32 accumulation).  fp16 has the 8 significant bits of bf16 and more, but
 * only the exponent range 6.1e-5 .. 65504: an element of v, S0 or of the running state beyond 65504 in magnitude becomes
 * infinite without an error code, and elements below 6.1e-5 lose precision gradually.  The stated tolerance (2e-3 of
 * max|O|) is tested for |v|, |S| up to the order of 1e3.  The operation is linear in (v, S0): scale them by a power
 * of two and O, S_final back for data outside that range, or ask for PF_IMPL_SIMT (fp32 throughout, no such limit).
 */
int pf_deltanet_fwd(const void* q, const void* k, const void* v, const void* beta, const float* S0,
                    int B, int H, int L, int d_k, int d_v, int r, int chunk,
                    float* O, float* S_final, void* stream);

/* Same operation with fp32 q, k, v, beta (all arithmetic fp32 FFMA).  Same passages. */
int pf_deltanet_fwd_f32(const float* q, const float* k, const float* v, const float* beta,
                        const float* S0, int B, int H, int L, int d_k, int d_v, int r, int chunk,
                        float* O, float* S_final, void* stream);

/*
 * pf_deltanet_fwd_f32_static -- pf_deltanet_fwd_f32 for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a packaging variant of the fp32 path, same arithmetic.)
 *
 * Who needs it: code that runs where cudaMalloc / cudaMallocAsync is off limits -- inside a region that
 * must not touch the allocator (a real-time loop, a host that gave this library a fixed memory budget,
 * a process whose device allocator belongs to another runtime).  The other entry points take their
 * per-chunk scratch from the stream-ordered allocator or from the caller; this one uses a fixed array
 * of PF_STATIC_SCRATCH_BYTES that is part of the library image, so it calls no allocating routine.
 *
 *   - Arguments, layouts, results, checks and error codes are those of pf_deltanet_fwd_f32 (the fp32 SIMT kernels,
 *     default options); pf_last_launch_count() and the profile list describe it like any other call.
 *   - A problem whose scratch (pf_static_scratch_need(...) bytes: T', W, Uh and P of every chunk in fp32) exceeds
 *     PF_STATIC_SCRATCH_BYTES is refused with PF_ERR_WORKSPACE and nothing is launched.
 *   - The array occupies PF_STATIC_SCRATCH_BYTES on every GPU that loads the library, until exit.
 *   - The first call on each device looks up the array's device address (one cudaGetSymbolAddress,
 *     with that device current); make that first call before starting any stream capture.
 *   - All calls on a device share the array and it keeps the previous call's contents.  Nothing in it
 *     needs clearing (each call writes what it later reads), but two calls that overlap on the GPU
 *     (different streams, no ordering between them) race on it: serialise them.
 */
#define PF_STATIC_SCRATCH_BYTES (8u << 20)
int pf_deltanet_fwd_f32_static(const float* q, const float* k, const float* v, const float* beta,
                               const float* S0, int B, int H, int L, int d_k, int d_v, int r, int chunk,
                               float* O, float* S_final, void* stream);
/* The compiled-in value of PF_STATIC_SCRATCH_BYTES. */
size_t pf_static_scratch_bytes(void);
/* Bytes of the fixed array that pf_deltanet_fwd_f32_static would use for this problem (host arithmetic). */
size_t pf_static_scratch_need(int B, int H, int L, int d_k, int d_v, int r, int chunk);

typedef struct pf_params {
    const void* q;            /* as in pf_deltanet_fwd, element type given by in_dtype */
    const void* k;
    const void* v;
    const void* beta;
    const float* S0;
    int B, H, L, d_k, d_v, r, chunk;
    float* O;
    float* S_final;
    int in_dtype;             /* PF_DTYPE_BF16 or PF_DTYPE_F32 */
    int impl;                 /* PF_IMPL_* */
    void* workspace;          /* device scratch of >= pf_workspace_bytes(...) bytes, 256-byte aligned,
                                 or NULL: stream-ordered allocation inside the call */
    size_t workspace_bytes;
    void* stream;
    int mode;                 /* PF_MODE_SUM (0) or PF_MODE_PRODUCT; anything else: PF_ERR_INVALID */
    int step;                 /* PF_STEP_EULER (0) or PF_STEP_EXACT; anything else: PF_ERR_INVALID */
    /* Options.  0 always means the default; results agree within rounding whatever their values. */
    int segments;             /* S > 1 (up to 64): cut every sequence into S segments of L/S tokens and evaluate them
                                 side by side (Section 3, "Scan": the flow of an interval is the pair (P, Xi) with
                                 S_end = S_start P + Xi, Proposition 2.1, and flows of consecutive intervals compose).
                                 The pass is linear in (start state, v), so two passes over the segments suffice: from
                                 the zero state with the caller's v (gives each segment's own part of O, and Xi) and from
                                 the identity with v = 0 (gives P and, as its output, every token's response to its
                                 segment's start state).  A small kernel composes the S flows of every sequence into the
                                 segments' start states and one GEMM per segment adds start state x response to O.
                                 About twice the work, but S times the parallelism and no pass waits for another's
                                 states: meant for problems with far fewer sequences (B*H) than the GPU has SMs.  Needs
                                 d_k = d_v and L a multiple of S, otherwise PF_ERR_UNSUPPORTED; the workspace grows by
                                 four arrays of B*H*S*d_k*d_v floats, an O-sized array and a v-sized array of zeros. */
    int wu_builder;           /* how the fp32 SIMT kernels obtain W and Uh of a chunk.  0: the triangular inverse T' of
                                 Theorem 3.2, then W = T'K, Uh = T'V.  1: the two-index system of Theorem 3.3 (the
                                 "signature kernel inspired algorithm", no inverse), swept along its antidiagonals by one
                                 kernel; needs more workspace.  The tensor-core kernels do not use it, except
                                 PF_IMPL_TC_REFFLOW, whose flows come from the SIMT kernels. */
    int ring_depth;           /* 3..64: slots per sequence of the L2-resident ring through which the single-launch
                                 tensor-core path hands each chunk's flow to the state scan.  Default 8, and 16 for
                                 sequences of more than 256 chunks while all rings together stay within 48 MB. */
    int* status;              /* NULL, or a 4-byte aligned DEVICE word (owned by the caller) that receives the code of the
                                 first bounded device-side wait that expired during this call (0 = none): see
                                 pf_read_status. */
} pf_params;

/* Same operation with explicit options.  The workspace holds per-chunk intermediates (T', W, Uh, P
 * of Theorem 3.2 in the forms the selected kernels exchange) and, at its end, the fp32 step sizes of
 * PF_STEP_EXACT; its content after the call is unspecified.  Same passages as pf_deltanet_fwd, plus those
 * named at PF_MODE_* and PF_STEP_*. */
int pf_deltanet_fwd_ex(const pf_params* p);

/* Bytes of scratch pf_deltanet_fwd_ex needs for this problem with this in_dtype/impl and every option at its
 * default (0 on an unsupported combination).  Host arithmetic; for the tensor-core implementations it asks the
 * current device for its SM count (no allocation, no launch, no synchronisation). */
size_t pf_workspace_bytes(int B, int H, int L, int d_k, int d_v, int r, int chunk, int in_dtype, int impl);
/* The same for a filled-in pf_params (shape, in_dtype, impl, mode and the options are read; pointers are not). */
size_t pf_workspace_bytes_ex(const pf_params* p);

/* Which PF_IMPL_* pf_deltanet_fwd_ex would run for this problem (negative pf_status if none). */
int pf_select_impl(int B, int H, int L, int d_k, int d_v, int r, int chunk, int in_dtype, int impl);
/* The chunk length the kernels would be run with: `chunk` itself for an explicit implementation; under PF_IMPL_AUTO
 * possibly another supported length (see PF_IMPL_AUTO).  Negative pf_status if the problem is not supported. */
int pf_select_chunk(int B, int H, int L, int d_k, int d_v, int r, int chunk, int in_dtype, int impl);

/*
 * Device-side waits and the status word.
 *
 * The tensor-core kernels synchronise their warps, and the single-launch path its CTAs, with waits on barriers and
 * flags.  Every such wait is bounded (about a second of SM cycles).  A wait that runs out writes its code into a
 * 4-byte STATUS WORD and the kernels give up: they return, every other wait that sees the word set returns too, and
 * O / S_final of that call are undefined.  Nothing traps, hangs or faults, and the context stays usable.
 *
 * Where the word lives, in this order: pf_params.status if given; else word 0 of pf_params.workspace if the caller
 * passed one; else a word owned by the library (one per device).  Every forward call first sets the word it uses
 * to 0, in stream order, so a word describes the LAST call that used it.
 *
 * pf_read_status(word, stream): synchronises `stream`, reads the word and returns PF_OK (0 in it) or PF_ERR_TIMEOUT.
 * `word` is the pointer described above -- the status pointer, the workspace pointer, or NULL for the library's own
 * word on the current device.  pf_last_wait_code() then gives the code that was read (host thread local):
 *     1xx  flow-building role of the single-launch path (101-103 solve warps, 11x-12x bulk warps, 14x-15x MMA-issuing
 *          warps, 16x flag warp),   2xx  its scanning role (20x chain, 21x output, 22x loads, 23x MMA issue),
 *     1-99 the two-launch path (tc_flow, tc_scan),   99  shared memory not 1024-byte aligned,   900  pf_wait_selftest.
 * The fp32 SIMT kernels have no such waits.
 */
int pf_read_status(const void* word, void* stream);
int pf_last_wait_code(void);
/* Diagnostic (no counterpart in the paper): launches one warp that waits, with the library's bounded-wait routine and a
 * limit of `limit_us` microseconds (1..1000000), for a flag that nothing ever sets, so that the wait runs out, the
 * status word (as for a forward call: `status`, or NULL for the library's own word) receives code 900 and the kernel
 * returns.  For testing the reporting path above; it does not synchronise. */
int pf_wait_selftest(int* status, int limit_us, void* stream);

/* Number of kernels the last successful call on this host thread enqueued. */
int pf_last_launch_count(void);

/* Optional per-kernel timing for benchmarks.  While enabled, each kernel of a forward call is
 * bracketed by CUDA events on the call's stream.  After the call, pf_profile_count() gives the number
 * of kernels and pf_profile_read(i, ...) waits for kernel i to finish and returns its name and device
 * time in milliseconds.  Process-wide, not thread-safe; leave it off in production. */
void pf_profile_enable(int on);
int pf_profile_count(void);
int pf_profile_read(int idx, char* name, int name_cap, float* ms);

/* Diagnostic for the tensor-core building blocks (no counterpart in the paper): one tcgen05 GEMM
 *   D[128][N] (fp32) = (+-A) * B^T  over a contraction of 128, fp16 operands staged in shared memory.
 * variant bit 0: A is given as [k][m] (MN-major) instead of [m][k]; bit 1: B is given as [k][n]
 * instead of [n][k]; bit 2: negate A; bits 3 / 4: A / B staged unswizzled (column groups of 8) instead of
 * 128-byte swizzled; bit 5: A (given as [m][k]) is placed in tensor memory instead of shared memory.
 * A is 128x128 fp16, B is N x 128 (or 128 x N) fp16, N a multiple
 * of 16 in [16, 256].  Device pointers.  Synchronises the stream and allocates; for tests only. */
int pf_tc_selftest(int variant, const void* A, const void* B, float* D, int N, void* stream);

const char* pf_status_string(int status);
/* Text of the last CUDA error seen by this host thread inside the library ("" if none). */
const char* pf_last_error_string(void);
int pf_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PF_H_ */
