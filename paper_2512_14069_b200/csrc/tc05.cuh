// Thin inline-PTX layer over the Blackwell (sm_100a) primitives the tree-attention kernel uses:
// mbarriers with bounded waits, TMA tile loads, tensor-memory allocation, tcgen05 MMA issue / commit
// and tensor-memory loads and stores.  Nothing here knows about attention.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace radar {
namespace tc05 {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- mbarrier -----------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after `limit` polls (each poll itself blocks for a hardware-defined short
// time) or once *abort_flag has been set by another thread.  Returns false on give-up and sets the
// flag.  A wait that is satisfied at once costs one try_wait and nothing else: the flag is looked at
// only while polling (reading it on every wait cost more than the wait itself).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          uint32_t limit = 4u << 20) {
    if (mbar_try_wait(bar, parity)) return true;
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            __nanosleep(64);
        }
    }
    *abort_flag = 1;
    return false;
}
// The same for a whole (converged) warp: one lane polls, the others learn the outcome from it, so that
// the barrier word is not hit by 32 polls at a time.  `ok` chains earlier outcomes (false: do not wait).
__device__ __forceinline__ bool mbar_wait_warp(bool ok, uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    int r = 0;
    if ((threadIdx.x & 31) == 0) r = ok && mbar_wait(bar, parity, abort_flag);
    return __shfl_sync(0xffffffffu, r, 0) != 0;
}

// ---- proxies and fences -------------------------------------------------------------------------
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ---- TMA (tiled tensor loads into this CTA's shared memory; no multicast) -------------------------
__device__ __forceinline__ void tma_prefetch_desc(const void* tmap) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}
// x (c0) times the element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const void* tmap, uint64_t* bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

__device__ __forceinline__ void tma_load_4d(void* smem_dst, const void* tmap, uint64_t* bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}

// ---- tensor memory ------------------------------------------------------------------------------
// One warp allocates / frees; ncols is a power of two in [32, 512].  The base address lands in *smem_dst.
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// ---- descriptors ----------------------------------------------------------------------------------
// Shared-memory operand descriptor for tiles written by TMA with the 128-byte swizzle: rows of 128
// bytes, 8 rows per 1024-byte swizzle atom.
//   K-major operand  (rows = M or N index, the 128 bytes run along K): SBO = bytes between 8-row groups.
//   MN-major operand (rows = K index, the 128 bytes run along M/N): SBO = bytes between 8-row (8 K) groups,
//                     LBO = bytes between consecutive 64-element blocks along M/N.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3ffff) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fff) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fff) << 32;
    d |= (uint64_t)1 << 46;     // descriptor version of this architecture
    d |= (uint64_t)2 << 61;     // 128-byte swizzle
    return d;
}
// Instruction descriptor of kind::f16 with bf16 operands and fp32 accumulation.
__host__ __device__ constexpr uint32_t idesc_bf16_f32(int M, int N, bool a_mn_major, bool b_mn_major) {
    return (1u << 4)                       // D = f32
           | (1u << 7) | (1u << 10)        // A, B = bf16
           | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16)
           | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ---- MMA issue (one thread) -----------------------------------------------------------------------
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
// Predicated forms for a warp that runs the issue code converged: every lane executes the instruction
// stream (so the descriptor arithmetic stays warp-uniform), the lane with `pred` != 0 issues.
__device__ __forceinline__ uint32_t elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b32 r;\n\telect.sync r|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred;
}
__device__ __forceinline__ void mma_ss_if(uint32_t pred, uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate), "r"(pred)
        : "memory");
}
__device__ __forceinline__ void mma_ts_if(uint32_t pred, uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                          bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate), "r"(pred)
        : "memory");
}
__device__ __forceinline__ void mma_commit_if(uint32_t pred, uint64_t* bar) {
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(smem_u32(bar)), "r"(pred)
        : "memory");
}
// Groups of MMAs over consecutive K steps in ONE instruction sequence: the descriptor low words advance by a
// constant per step, the predicates are set once.  All lanes execute the sequence, the lane with pred != 0
// issues.  `hi` is the high word shared by all shared-memory descriptors of the kernel.
//   SS: four steps of 16 K-elements inside one 64-element swizzle block (32 B = 2 descriptor units per step).
__device__ __forceinline__ void mma_ss_x4(uint32_t pred, uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi,
                                          uint32_t idesc, bool acc_first) {
    asm volatile(
        "{\n\t.reg .pred q, p0, p1;\n\t.reg .b32 a, b;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 q, %0, 0;\n\t"
        "setp.ne.b32 p0, %6, 0;\n\t"
        "setp.eq.b32 p1, 0, 0;\n\t"
        "mov.b64 da, {%2, %4};\n\tmov.b64 db, {%3, %4};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], da, db, %5, p0;\n\t"
        "add.u32 a, %2, 2;\n\tadd.u32 b, %3, 2;\n\tmov.b64 da, {a, %4};\n\tmov.b64 db, {b, %4};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], da, db, %5, p1;\n\t"
        "add.u32 a, %2, 4;\n\tadd.u32 b, %3, 4;\n\tmov.b64 da, {a, %4};\n\tmov.b64 db, {b, %4};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], da, db, %5, p1;\n\t"
        "add.u32 a, %2, 6;\n\tadd.u32 b, %3, 6;\n\tmov.b64 da, {a, %4};\n\tmov.b64 db, {b, %4};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], da, db, %5, p1;\n\t}"
        ::"r"(pred), "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"((uint32_t)acc_first)
        : "memory");
}
//   TS: four steps; A advances by 8 tensor-memory columns (16 bf16) and B by 128 descriptor units (16 rows of
//   an N-major tile) per step.  Steps at or beyond `nsteps` are not issued.
__device__ __forceinline__ void mma_ts_x4(uint32_t pred, uint32_t nsteps, uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo,
                                          uint32_t hi, uint32_t idesc, bool acc_first) {
#define RADAR_TS_STEP(K, P)                                                                            \
        "setp.gt.and.u32 qk, %1, " #K ", q;\n\t"                                                        \
        "add.u32 a, %3, " #K " * 8;\n\tadd.u32 b, %4, " #K " * 128;\n\tmov.b64 db, {b, %5};\n\t"         \
        "@qk tcgen05.mma.cta_group::1.kind::f16 [%2], [a], db, %6, " #P ";\n\t"
    asm volatile(
        "{\n\t.reg .pred q, qk, p0, p1;\n\t.reg .b32 a, b;\n\t.reg .b64 db;\n\t"
        "setp.ne.b32 q, %0, 0;\n\t"
        "setp.ne.b32 p0, %7, 0;\n\t"
        "setp.eq.b32 p1, 0, 0;\n\t"
        RADAR_TS_STEP(0, p0) RADAR_TS_STEP(1, p1) RADAR_TS_STEP(2, p1) RADAR_TS_STEP(3, p1)
        "}"
        ::"r"(pred), "r"(nsteps), "r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"((uint32_t)acc_first)
        : "memory");
#undef RADAR_TS_STEP
}
//   TS, all four steps, no per-step predicate.
__device__ __forceinline__ void mma_ts_x4_full(uint32_t pred, uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi,
                                               uint32_t idesc, bool acc_first) {
#define RADAR_TS_STEP(K, P)                                                                            \
        "add.u32 a, %2, " #K " * 8;\n\tadd.u32 b, %3, " #K " * 128;\n\tmov.b64 db, {b, %4};\n\t"         \
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a], db, %5, " #P ";\n\t"
    asm volatile(
        "{\n\t.reg .pred q, p0, p1;\n\t.reg .b32 a, b;\n\t.reg .b64 db;\n\t"
        "setp.ne.b32 q, %0, 0;\n\t"
        "setp.ne.b32 p0, %6, 0;\n\t"
        "setp.eq.b32 p1, 0, 0;\n\t"
        RADAR_TS_STEP(0, p0) RADAR_TS_STEP(1, p1) RADAR_TS_STEP(2, p1) RADAR_TS_STEP(3, p1)
        "}"
        ::"r"(pred), "r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"((uint32_t)acc_first)
        : "memory");
#undef RADAR_TS_STEP
}
// The barrier receives one arrival once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// ---- tensor-memory loads / stores (warp-collective; lane l of warp w touches TMEM lane 32 (w % 4) + l) ----
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
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
          "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
          "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]), "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

}  // namespace tc05
}  // namespace radar
