// sm_100a building blocks for the tensor-core path: mbarrier, TMA (tensor and bulk copies),
// tcgen05 (TMEM allocation, MMA, commit, load), shared-memory matrix descriptors for the
// 128-byte-swizzled canonical layouts, and warp-level mma.sync/ldmatrix for the small solve.
//
// Shared-memory operand convention used everywhere in this path ("slab"): a matrix X[R rows][Cc cols]
// of 16-bit elements is stored as Cc/64 slabs; slab s holds columns 64s..64s+63 as R rows of 128 bytes;
// inside a slab the 16-byte chunk c of row r sits at chunk position c ^ (r & 7) (the 128B swizzle that
// TMA's SWIZZLE_128B writes and tcgen05's SWIZZLE_128B descriptors read).  Slab bases are 1024-byte
// aligned.  The same bytes serve as
//   * a K-major operand  (MN index = row, contraction index = column), or
//   * an MN-major operand (contraction index = row, MN index = column),
// only the descriptor differs.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace pf {
namespace tc {

constexpr uint32_t SPIN_LIMIT = 1u << 26;   // bounded waits: ~ a second, then the kernel gives up

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// byte offset of element (row, col) in a slab-stored matrix with R rows
__device__ __host__ __forceinline__ uint32_t slab_off(int row, int col, int R) {
    return (uint32_t)(col >> 6) * (uint32_t)R * 128u + (uint32_t)row * 128u +
           ((((uint32_t)(col & 63) >> 3) ^ ((uint32_t)row & 7u)) << 4) + ((uint32_t)col & 7u) * 2u;
}

// ---- mbarrier ------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Non-blocking test of a phase (try_wait may suspend the thread for a while; a poller of several barriers must not).
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and raises *err_flag) if the phase never completes.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* err_flag, int code) {
    for (uint32_t it = 0; it < SPIN_LIMIT; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 64) __nanosleep(32);
    }
    if (err_flag) atomicExch(err_flag, code);
    return false;
}

// Bounded wait by elapsed cycles (about a second) instead of an iteration count, without sleeping:
// the waits of the fused kernel sit on latency-critical paths.  Also gives up early once another
// thread has reported a failure in *err_flag, so that one expired wait drains the whole grid quickly.
constexpr long long WAIT_CYCLES = 2000000000ll;
// The polling loop is kept out of line: dozens of call sites would otherwise bloat the instruction footprint.
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar_addr, uint32_t parity, int* err_flag, int code) {
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar_addr), "r"(parity)
            : "memory");
        if (ok) return true;
        if ((it & 255u) == 0) {
            if (clock64() - t0 > WAIT_CYCLES) break;
            if ((it & 4095u) == 0 && *(volatile int*)err_flag != 0) return false;
        }
    }
    atomicCAS(err_flag, 0, code);
    return false;
}
__device__ __forceinline__ bool mbar_wait_clk(uint64_t* bar, uint32_t parity, int* err_flag, int code) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(smem_u32(bar), parity, err_flag, code);
}

// ---- named barriers, global-memory flags, cache-bypassing loads ----------------------------------------
__device__ __forceinline__ void named_bar(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
// Barrier + AND-reduction of a per-thread predicate over the participating threads.
__device__ __forceinline__ bool named_bar_and(int id, int nthreads, bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %3, 0;\n\tbar.red.and.pred p, %1, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"(id), "r"(nthreads), "r"((uint32_t)pred)
        : "memory");
    return out != 0;
}
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_gpu(int* p, int v) {
    asm volatile("st.release.gpu.global.b32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Loads of data another CTA wrote during this kernel: L2 only (a recycled ring slot must never hit a
// stale L1 line).
__device__ __forceinline__ uint4 ld_cg_u4(const void* p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float ld_cg_f32(const float* p) {
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory");
    return v;
}
// Waits until *p >= want (acquire), bounded by elapsed cycles.
static __device__ __noinline__ bool flag_wait_ge_limit(const int* p, int want, int* err_flag, int code, long long limit) {
    if (ld_acquire_gpu(p) >= want) return true;
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (ld_acquire_gpu(p) >= want) return true;
        if ((it & 15u) == 0) {
            if (clock64() - t0 > limit) break;
            if ((it & 255u) == 0 && *(volatile int*)err_flag != 0) return false;
        }
    }
    atomicCAS(err_flag, 0, code);
    return false;
}
__device__ __forceinline__ bool flag_wait_ge(const int* p, int want, int* err_flag, int code) {
    return flag_wait_ge_limit(p, want, err_flag, code, WAIT_CYCLES);
}

// Waits until a shared-memory counter reaches `want` (written by another warp of the CTA after
// __threadfence_block()), bounded by elapsed cycles.
static __device__ __noinline__ bool smem_wait_ge(volatile int* p, int want, int* err_flag, int code) {
    if (*p >= want) { __threadfence_block(); return true; }
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (*p >= want) { __threadfence_block(); return true; }
        if ((it & 255u) == 0) {
            if (clock64() - t0 > WAIT_CYCLES) break;
            if ((it & 4095u) == 0 && *(volatile int*)err_flag != 0) return false;
        }
    }
    atomicCAS(err_flag, 0, code);
    return false;
}

// ---- proxies / fences ----------------------------------------------------------------------------
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ---- TMA -----------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
        : "memory");
}
// 1-D bulk copy global -> shared; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// 1-D bulk copy shared -> global (bulk async-group completion); same alignment rules.
__device__ __forceinline__ void bulk_store(void* gdst, const void* ssrc, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_u32(ssrc)), "r"(bytes)
                 : "memory");
}
// 1-D bulk fp32 add of a shared-memory image into global memory, performed at the L2 (bulk async-group completion)
__device__ __forceinline__ void bulk_reduce_add_f32(void* gdst, const void* ssrc, uint32_t bytes) {
    asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;" ::"l"(gdst),
                 "r"(smem_u32(ssrc)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// ---- TMEM ----------------------------------------------------------------------------------------
// One full warp calls these.  ncols: power of two in [32, 512].
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp gets lane (taddr.lane + t), columns c..c+31.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- descriptors ---------------------------------------------------------------------------------
// Shared-memory matrix descriptor, SWIZZLE_128B, 16-bit elements, slab layout above.
//   K-major : rows 128 B apart, 8-row groups SBO = 1024 B apart; LBO unused (1).
//   MN-major: contraction rows 128 B apart, 8-row groups SBO = 1024 B apart; the next 64 MN elements
//             (next slab) LBO bytes further.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);            // start address, bits [0,14)
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;   // leading byte offset, bits [16,30)
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;   // stride byte offset, bits [32,46)
    d |= (uint64_t)1 << 46;                              // descriptor version (Blackwell)
    d |= (uint64_t)2 << 61;                              // SWIZZLE_128B
    return d;
}
// ---- unswizzled ("interleaved") operands ---------------------------------------------------------------
// A matrix X[R rows][Cc cols] of 16-bit elements stored as Cc/8 column groups; group g holds columns 8g..8g+7
// as R rows of 16 bytes:  offset(row, col) = (col/8)*R*16 + row*16 + (col%8)*2.  Eight consecutive rows of a
// group are one 128-byte core matrix.  A warp whose lane l writes the 16-byte piece of row (r0 + l) writes
// 512 contiguous bytes, which is why images that cross global memory use this form.
//   K-major  (contraction index = column): core matrices 128 B apart along MN (SBO), R*16 apart along K (LBO)
//   MN-major (contraction index = row)   : core matrices 128 B apart along K (LBO), R*16 apart along MN (SBO)
__device__ __host__ __forceinline__ uint32_t ns_off(int row, int col, int R) {
    return (uint32_t)(col >> 3) * (uint32_t)R * 16u + (uint32_t)row * 16u + ((uint32_t)col & 7u) * 2u;
}
__device__ __forceinline__ uint64_t make_desc_ns(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;                              // descriptor version (Blackwell); swizzle field 0 = none
    return d;
}
__device__ __forceinline__ uint64_t desc_ns_kmajor(uint32_t saddr, int R) { return make_desc_ns(saddr, (uint32_t)R * 16u, 128u); }
__device__ __forceinline__ uint64_t desc_ns_mnmajor(uint32_t saddr, int R) { return make_desc_ns(saddr, 128u, (uint32_t)R * 16u); }
// byte advance of the start address per K-step of 16
__device__ __host__ __forceinline__ uint32_t ns_kstep_kmajor(int R) { return 2u * (uint32_t)R * 16u; }
__device__ __host__ constexpr uint32_t ns_kstep_mnmajor() { return 256u; }

__device__ __forceinline__ uint64_t desc_kmajor(uint32_t saddr) { return make_desc(saddr, 16, 1024); }
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t saddr, uint32_t slab_bytes) {
    return make_desc(saddr, slab_bytes, 1024);
}

// Instruction descriptor for kind::f16 with fp16 A and B, fp32 accumulator, M = 128.
//   bits [4,6) D format (1 = f32), [7,10) A format (0 = f16), [10,13) B format, 13 negate A, 14 negate B,
//   15 A major (1 = MN), 16 B major (1 = MN), [17,23) N >> 3, [24,29) M >> 4.
__device__ __host__ constexpr uint32_t make_idesc(int N, bool a_mn, bool b_mn, bool neg_a) {
    return (1u << 4) | ((neg_a ? 1u : 0u) << 13) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// D[tmem] (+)= A * B^T, one K = 16 step.  Issued by ONE thread.
__device__ __forceinline__ void mma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
    const uint32_t acc = accumulate ? 1u : 0u;
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
// Same with the A operand in tensor memory: lane m holds row m, 32-bit column c holds elements k = 2c (low
// half) and 2c+1 (high half); one K = 16 step reads 8 columns.  The instruction descriptor must say K-major A.
__device__ __forceinline__ void mma_f16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, bool accumulate) {
    const uint32_t acc = accumulate ? 1u : 0u;
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns, registers -> tensor memory (one full warp)
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// Arrives on `bar` when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// A full GEMM  D[128 x N] (+)= A[128 x Kdim] * B[N x Kdim]^T  from slab-stored operands.
//   a_base/b_base: shared addresses of slab 0; a_rows/b_rows: rows per slab of each operand.
//   K-major operand : contraction index = column -> step kk uses slab kk/4, byte offset (kk%4)*32.
//   MN-major operand: contraction index = row    -> step kk starts at row 16*kk (2048 B further).
template <bool A_MN, bool B_MN>
__device__ __forceinline__ void gemm_issue(uint32_t d_tmem, uint32_t a_base, int a_rows, uint32_t b_base, int b_rows,
                                           int N, int Kdim, bool neg_a, bool accumulate_first) {
    const uint32_t idesc = make_idesc(N, A_MN, B_MN, neg_a);
    for (int kk = 0; kk < Kdim / 16; ++kk) {
        uint64_t ad, bd;
        if (A_MN) ad = desc_mnmajor(a_base + (uint32_t)kk * 2048u, (uint32_t)a_rows * 128u);
        else ad = desc_kmajor(a_base + (uint32_t)(kk >> 2) * (uint32_t)a_rows * 128u + (uint32_t)(kk & 3) * 32u);
        if (B_MN) bd = desc_mnmajor(b_base + (uint32_t)kk * 2048u, (uint32_t)b_rows * 128u);
        else bd = desc_kmajor(b_base + (uint32_t)(kk >> 2) * (uint32_t)b_rows * 128u + (uint32_t)(kk & 3) * 32u);
        mma_f16(d_tmem, ad, bd, idesc, accumulate_first || kk > 0);
    }
}

// Warp-uniform issue with every shape known at compile time: the WHOLE warp runs this (converged) and one
// elected lane issues each instruction.  The two base descriptors are built once and each K-step only adds a
// constant to the start-address field; with uniform control flow that arithmetic stays in the uniform
// datapath, which makes the issue several times cheaper than a single diverged lane rebuilding descriptors.
// BF16: both operands are bf16 instead of fp16 (same 16-bit layouts).
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}
// Operand layouts: 128-byte swizzled slabs (SW) or unswizzled column groups (NS), K-major or MN-major.
enum { L_SWK = 0, L_SWMN = 1, L_NSK = 2, L_NSMN = 3 };
template <int LAY, int ROWS>
__device__ __forceinline__ uint64_t desc_of(uint32_t base) {
    return LAY == L_SWK ? desc_kmajor(base) : LAY == L_SWMN ? desc_mnmajor(base, (uint32_t)ROWS * 128u)
         : LAY == L_NSK ? desc_ns_kmajor(base, ROWS) : desc_ns_mnmajor(base, ROWS);
}
template <int LAY, int ROWS>
__device__ __forceinline__ constexpr uint32_t kstep_off(int kk) {
    return LAY == L_SWK ? (uint32_t)(kk >> 2) * (uint32_t)ROWS * 128u + (uint32_t)(kk & 3) * 32u
         : LAY == L_SWMN ? (uint32_t)kk * 2048u
         : LAY == L_NSK ? (uint32_t)kk * 2u * (uint32_t)ROWS * 16u : (uint32_t)kk * 256u;
}
// ACC: accumulate onto what the accumulator holds (from the first K-step on) instead of overwriting it.
template <int AL, int BL, int NCOLS, int KDIM, int A_ROWS, int B_ROWS, bool BF16 = false, bool ACC = false>
__device__ __forceinline__ void gemm_lay(uint32_t d_tmem, uint32_t a_base, uint32_t b_base) {
    constexpr bool A_MN = (AL == L_SWMN || AL == L_NSMN), B_MN = (BL == L_SWMN || BL == L_NSMN);
    constexpr uint32_t idesc = make_idesc(NCOLS, A_MN, B_MN, false) | (BF16 ? ((1u << 7) | (1u << 10)) : 0u);
    const uint64_t a0 = desc_of<AL, A_ROWS>(a_base), b0 = desc_of<BL, B_ROWS>(b_base);
#pragma unroll
    for (int kk = 0; kk < KDIM / 16; ++kk) {
        const uint64_t ad = a0 + (uint64_t)(kstep_off<AL, A_ROWS>(kk) >> 4), bd = b0 + (uint64_t)(kstep_off<BL, B_ROWS>(kk) >> 4);
        if (elect_one()) mma_f16(d_tmem, ad, bd, idesc, ACC || kk > 0);
    }
}
// D[128 x NCOLS] = A * B^T with A (fp16, K-major, KDIM/2 packed columns) in tensor memory; whole warp, converged.
template <int BL, int NCOLS, int KDIM, int B_ROWS, bool ACC = false>
__device__ __forceinline__ void gemm_ta(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_base) {
    constexpr bool B_MN = (BL == L_SWMN || BL == L_NSMN);
    constexpr uint32_t idesc = make_idesc(NCOLS, false, B_MN, false);
    const uint64_t b0 = desc_of<BL, B_ROWS>(b_base);
#pragma unroll
    for (int kk = 0; kk < KDIM / 16; ++kk) {
        const uint64_t bd = b0 + (uint64_t)(kstep_off<BL, B_ROWS>(kk) >> 4);
        if (elect_one()) mma_f16_ta(d_tmem, a_tmem + 8u * (uint32_t)kk, bd, idesc, ACC || kk > 0);
    }
}
template <bool A_MN, bool B_MN, int NCOLS, int KDIM, int A_ROWS, int B_ROWS, bool BF16 = false, bool ACC = false>
__device__ __forceinline__ void gemm_uni(uint32_t d_tmem, uint32_t a_base, uint32_t b_base) {
    gemm_lay<A_MN ? L_SWMN : L_SWK, B_MN ? L_SWMN : L_SWK, NCOLS, KDIM, A_ROWS, B_ROWS, BF16, ACC>(d_tmem, a_base, b_base);
}
__device__ __forceinline__ void commit_uni(uint64_t* bar) {
    if (elect_one()) mma_commit(bar);
}

// ---- warp-level MMA for the small triangular solve -------------------------------------------------
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t saddr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(saddr) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t saddr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(saddr) : "memory");
}
__device__ __forceinline__ uint32_t pack_h2(float lo, float hi) {
    __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

// byte offset of the 16-byte piece `col8` (= column / 8) of row `row` in a slab-stored matrix with R rows
__device__ __forceinline__ uint32_t chunk_off(int row, int col8, int R) {
    return (uint32_t)(col8 >> 3) * (uint32_t)R * 128u + (uint32_t)row * 128u + ((((uint32_t)col8 & 7u) ^ ((uint32_t)row & 7u)) << 4);
}

// ---- the triangular inverse X = (I + A)^{-1}, A strictly (block) lower triangular, fp16, slab-stored, N x N ----------
// (Proposition on block-triangular inversion: diagonal blocks first, then off-diagonal blocks from them.)
//
// A 16 x 16 diagonal block by its Neumann product: A is nilpotent (A^16 = 0), so
//     (I + A)^{-1} = (I - A)(I + A^2)(I + A^4)(I + A^8).
// One warp, all in registers: the accumulator fragment of mma.m16n8k16 is, after packing to fp16, the A-operand
// fragment of the same matrix, and the A-operand fragment of M^T serves as the two B-operand fragments of M, so the
// powers are carried as the pair (M, M^T).  `deep`: include the A^8 factor (not needed when the mask groups rows in
// pairs or more, since then A^8 = 0).  The block is read from and written back to rows/columns [16 blk, 16 blk + 16).
__device__ __forceinline__ void frag_mul(float (&c)[2][4], const uint32_t (&x)[4], const uint32_t (&mt)[4]) {
    mma_16816(c[0], x, mt[0], mt[2]);     // columns 0..7 of  X * M   (mt = A-operand fragment of M^T)
    mma_16816(c[1], x, mt[1], mt[3]);     // columns 8..15
}
__device__ __forceinline__ void frag_pack(uint32_t (&f)[4], const float (&c)[2][4]) {
    f[0] = pack_h2(c[0][0], c[0][1]);
    f[1] = pack_h2(c[0][2], c[0][3]);
    f[2] = pack_h2(c[1][0], c[1][1]);
    f[3] = pack_h2(c[1][2], c[1][3]);
}
__device__ __forceinline__ void frag_zero(float (&c)[2][4]) {
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int e = 0; e < 4; ++e) c[h][e] = 0.f;
}
__device__ __forceinline__ void diag_inverse16(uint32_t xb, uint8_t* xg, int blk, int lane, int N, bool deep) {
    const int R0 = 16 * blk, c8 = 2 * blk;
    uint32_t a[4], at[4];
    ldmatrix_x4(a, xb + chunk_off(R0 + (lane & 15), c8 + (lane >> 4), N));
    ldmatrix_x4_trans(at, xb + chunk_off(R0 + (lane & 7) + ((lane >> 4) << 3), c8 + ((lane >> 3) & 1), N));
    float c[2][4], ct[2][4];
    uint32_t a2[4], a2t[4], a4[4], a4t[4];
    frag_zero(c); frag_zero(ct);
    frag_mul(c, a, at);         // A^2
    frag_mul(ct, at, a);        // (A^2)^T = A^T A^T
    frag_pack(a2, c); frag_pack(a2t, ct);
    frag_zero(c); frag_zero(ct);
    frag_mul(c, a2, a2t);       // A^4
    frag_mul(ct, a2t, a2);
    frag_pack(a4, c); frag_pack(a4t, ct);
    // R = I - A in accumulator layout: thread (g, t) holds rows g, g+8 and columns 8h + 2t, 8h + 2t + 1
    const int gq = lane >> 2, t4 = lane & 3;
    float r[2][4];
    {
        const __half2 h0 = *reinterpret_cast<const __half2*>(&a[0]), h1 = *reinterpret_cast<const __half2*>(&a[1]);
        const __half2 h2 = *reinterpret_cast<const __half2*>(&a[2]), h3 = *reinterpret_cast<const __half2*>(&a[3]);
        const float2 f0 = __half22float2(h0), f1 = __half22float2(h1), f2 = __half22float2(h2), f3 = __half22float2(h3);
        const float d0 = (gq == 2 * t4) ? 1.f : 0.f, d1 = (gq == 2 * t4 + 1) ? 1.f : 0.f;
        r[0][0] = d0 - f0.x; r[0][1] = d1 - f0.y;     // row g,   columns 2t, 2t+1
        r[0][2] = -f1.x;     r[0][3] = -f1.y;         // row g+8, columns 2t, 2t+1
        r[1][0] = -f2.x;     r[1][1] = -f2.y;         // row g,   columns 8+2t, 8+2t+1
        r[1][2] = d0 - f3.x; r[1][3] = d1 - f3.y;     // row g+8, columns 8+2t, 8+2t+1
    }
    uint32_t rf[4];
    frag_pack(rf, r);
    frag_mul(r, rf, a2t);       // R (I + A^2)
    frag_pack(rf, r);
    frag_mul(r, rf, a4t);       // ... (I + A^4)
    if (deep) {
        frag_zero(ct);
        frag_mul(ct, a4t, a4);  // (A^8)^T
        uint32_t a8t[4];
        frag_pack(a8t, ct);
        frag_pack(rf, r);
        frag_mul(r, rf, a8t);   // ... (I + A^8)
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        *(uint32_t*)(xg + chunk_off(R0 + gq, c8 + h, N) + 4 * t4) = pack_h2(r[h][0], r[h][1]);
        *(uint32_t*)(xg + chunk_off(R0 + gq + 8, c8 + h, N) + 4 * t4) = pack_h2(r[h][2], r[h][3]);
    }
}

// One level of the recursive-doubling inverse: diagonal blocks of size S are merged into blocks of size 2S,
//     X_hi,lo = -X_hi,hi A_hi,lo X_lo,lo.
// Task = (merge, 16-row strip): N/32 tasks, one warp each; the four warps synchronise on named barrier BAR
// (128 threads; BAR = 0 is the CTA barrier of a 128-thread CTA).
template <int N, int S, int BAR>
__device__ __forceinline__ void merge_level(uint32_t xb, uint8_t* xg, int warp, int lane) {
    constexpr int TASKS = N / 32;
    constexpr int STRIPS = S / 16;
    constexpr int NT = S / 8;
    float z[NT][4];
    const bool has_task = warp < TASKS;
    const int q = warp / STRIPS, strip = warp % STRIPS;
    const int lo0 = 2 * S * q, hi0 = lo0 + S, R0 = hi0 + 16 * strip;
    const int id = lane >> 3;
    if (has_task) {
        float u[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) u[nt][e] = 0.f;
        // (all column offsets below are multiples of 8, all row offsets multiples of 8 plus a lane term)
        const int a_row = R0 + (lane & 15), a_c8 = (hi0 >> 3) + (lane >> 4);
        const int b_rowl = (lane & 7) + ((id & 1) << 3), b_c8l = (id >> 1);
#pragma unroll
        for (int kk = 0; kk < S / 16; ++kk) {
            if (kk > strip) continue;   // X_hi,hi is lower triangular
            uint32_t a[4];
            ldmatrix_x4(a, xb + chunk_off(a_row, a_c8 + 2 * kk, N));
#pragma unroll
            for (int np = 0; np < S / 16; ++np) {
                uint32_t b[4];
                ldmatrix_x4_trans(b, xb + chunk_off(hi0 + 16 * kk + b_rowl, (lo0 >> 3) + 2 * np + b_c8l, N));
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
                ldmatrix_x4_trans(b, xb + chunk_off(lo0 + 16 * kk + b_rowl, (lo0 >> 3) + 2 * np + b_c8l, N));
                mma_16816(z[2 * np], a, b[0], b[1]);
                mma_16816(z[2 * np + 1], a, b[2], b[3]);
            }
        }
    }
    named_bar(BAR, 128);   // every strip has read A_hi,lo before anyone overwrites it
    if (has_task) {
        const int gq = lane >> 2, t4 = lane & 3;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int c8 = (lo0 >> 3) + nt;
            *(uint32_t*)(xg + chunk_off(R0 + gq, c8, N) + 4 * t4) = pack_h2(-z[nt][0], -z[nt][1]);
            *(uint32_t*)(xg + chunk_off(R0 + gq + 8, c8, N) + 4 * t4) = pack_h2(-z[nt][2], -z[nt][3]);
        }
    }
    named_bar(BAR, 128);
}

}  // namespace tc
}  // namespace pf
