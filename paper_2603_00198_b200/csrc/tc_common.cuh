// sm_100a building blocks in inline PTX: mbarriers with bounded waits, TMA tile loads, tcgen05
// (TMEM allocation, UMMA descriptors, MMA issue, commit, TMEM loads).  Internal to libstr.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace tc {

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t globaltimer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// ---- mbarrier -------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
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
// Bounded wait.  Each failed probe parks the warp for a hardware-defined slice of time, so the limit is
// a count of probes (millions: far beyond any legitimate wait inside these kernels, which last
// microseconds).  Gives up at once when another role of the CTA has raised *abort.  Returns false on
// give-up; the caller records STR_ERR_TIMEOUT and leaves its loops.  Kept to a handful of
// instructions and never unrolled: warp-specialised kernels have dozens of wait sites and their
// combined footprint has to stay inside the instruction cache.
constexpr uint32_t WAIT_PROBE_LIMIT = 1u << 22;
// Non-blocking probe: has the phase with this parity completed?
__device__ __forceinline__ bool mbar_test_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort) {
    if (mbar_test_wait(bar, parity)) return true;        // the common case in a pipeline that runs ahead
    uint32_t probes = 0;
#pragma unroll 1
    while (!mbar_try_wait(bar, parity)) {
        if (++probes > WAIT_PROBE_LIMIT || *abort) { *abort = 1; return false; }
    }
    return true;
}

// Has an earlier CTA of this launch (or an earlier launch) recorded an error?  Thread 0 reads the status word and
// the block agrees on the answer, so that a CTA leaves whole or not at all: warps that stayed behind would run
// warp-collective tcgen05 instructions and barriers with roles missing.
__device__ __forceinline__ bool cta_should_leave(const int *status) {
    return __syncthreads_or(threadIdx.x == 0 && *(volatile const int *)status != 0) != 0;
}

// ---- TMA ------------------------------------------------------------------------------------
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap *m) {
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)m) : "memory");
}
__device__ __forceinline__ void prefetch_l1(const void *p) {
    asm volatile("prefetch.global.L1 [%0];" ::"l"(p));
}
// 2-D tile load global -> shared, completion counted in bytes on an mbarrier.  c0 is the innermost
// (contiguous) coordinate and must be a multiple of 16 bytes worth of elements.
__device__ __forceinline__ void tma_load_2d(void *smem_dst, const CUtensorMap *m, uint64_t *bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"((uint64_t)m), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(void *smem_dst, const CUtensorMap *m, uint64_t *bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"((uint64_t)m), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// One lane of a converged warp (the lowest active one).  Used to predicate single-thread instructions
// (tcgen05.mma, tcgen05.commit) while the whole warp runs the surrounding loop, so that addresses and
// descriptors stay warp-uniform values.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}

// ---- tcgen05 --------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t *smem_slot, uint32_t ncols) {   // whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_slot)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {      // whole warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor (64-bit).  Fields: start address >> 4 [0,14), leading-dimension
// byte offset >> 4 [16,30), stride-dimension byte offset >> 4 [32,46), descriptor version 1 for
// sm_100 [46,48), swizzle mode [61,64): 0 none, 2 = 128-byte, 4 = 64-byte, 6 = 32-byte.
constexpr uint64_t SWZ_NONE = 0, SWZ_128B = 2, SWZ_64B = 4, SWZ_32B = 6;
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint64_t swz) {
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (swz << 61);
}
// K-major operand tile written by TMA with 128-byte swizzle: rows of 64 bf16 (128 B), 8-row groups
// 1024 B apart.  The tile base must be 1024-byte aligned; k_elem selects the 16-element K slice.
__device__ __forceinline__ uint64_t desc_kmajor_sw128(uint32_t tile_saddr, int k_elem) {
    return make_smem_desc(tile_saddr + (uint32_t)k_elem * 2u, 16, 1024, SWZ_128B);
}

// Instruction descriptor for kind::f16 with bf16 operands and fp32 accumulation.
// a_mn / b_mn: 0 = K-major operand, 1 = MN-major operand.
__host__ __device__ constexpr uint32_t make_idesc_bf16(int M, int N, int a_mn, int b_mn) {
    return (1u << 4)            /* D format fp32 */
           | (1u << 7)          /* A format bf16 */
           | (1u << 10)         /* B format bf16 */
           | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem]; issued by ONE thread.
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]; issued by ONE thread.
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
// ---- several K-slices of one product in ONE instruction block ---------------------------------
// Measured on B200 (one issuing warp next to arithmetic warps on its scheduler): a product written as a
// loop of single tcgen05.mma statements, or issued from an `if (lane == 0)` region, costs 100-400 clocks
// per instruction once the scheduler has other ready warps, because every instruction in between is a
// chance to lose the issue slot.  The same K-slices written as one straight-line block inside a region
// entered through elect_one() (which the compiler knows to be single-threaded) issue at the tensor pipe's
// own rate (about 50 clocks for N = 64, 64 for N = 128) whatever the other warps do.  So issuer roles
// enter elect_one() ONCE, stay in it for their whole loop, and issue each product with these helpers.
// `Step` gives the descriptor / tensor-memory address advance of K-slice ks as a compile-time constant.
struct StepKMajor2x64 {   // K-major operand stored as two 64-column halves 16 KB apart (128-byte swizzle), 16-byte units
    static __host__ __device__ constexpr uint32_t at(int ks) { return (uint32_t)(ks >> 2) * 1024u + (uint32_t)(ks & 3) * 2u; }
};
struct StepKMajor64 {     // K-major operand, one 64-column tile: 32 bytes per K-slice
    static __host__ __device__ constexpr uint32_t at(int ks) { return (uint32_t)ks * 2u; }
};
struct StepMNMajor {      // MN-major operand: 16 K-rows x 128 bytes = 2 KB per K-slice
    static __host__ __device__ constexpr uint32_t at(int ks) { return (uint32_t)ks * 128u; }
};
struct StepTmem8 {        // bf16 A operand in tensor memory, K-slices in consecutive groups of 8 columns
    static __host__ __device__ constexpr uint32_t at(int ks) { return (uint32_t)ks * 8u; }
};
struct StepTmem16 {       // bf16 A operand in tensor memory, K-slice ks in the first 8 of columns [16 ks, 16 ks + 16)
    static __host__ __device__ constexpr uint32_t at(int ks) { return (uint32_t)ks * 16u; }
};

#define STR_MMA_TAIL_SS(n, ia, ib)                                                        \
    "add.s64 a, %1, %" #ia ";\n\tadd.s64 b, %2, %" #ib ";\n\t"                            \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
#define STR_MMA_TAIL_TS(n, ia, ib)                                                        \
    "add.u32 at, %1, %" #ia ";\n\tadd.s64 b, %2, %" #ib ";\n\t"                           \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], b, %3, pt;\n\t"

// Eight K-slices, both operands in shared memory.  The first slice accumulates iff acc_first.
template <class SA, class SB>
__device__ __forceinline__ void mma8_ss(uint32_t d_tmem, uint64_t a0, uint64_t b0, uint32_t idesc, bool acc_first) {
    asm volatile(
        "{\n\t.reg .pred pf, pt;\n\t.reg .b64 a, b;\n\t"
        "setp.ne.b32 pf, %4, 0;\n\tsetp.eq.u32 pt, 0, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pf;\n\t"
        STR_MMA_TAIL_SS(1, 5, 6) STR_MMA_TAIL_SS(2, 7, 8) STR_MMA_TAIL_SS(3, 9, 10) STR_MMA_TAIL_SS(4, 11, 12)
        STR_MMA_TAIL_SS(5, 13, 14) STR_MMA_TAIL_SS(6, 15, 16) STR_MMA_TAIL_SS(7, 17, 18)
        "}"
        ::"r"(d_tmem), "l"(a0), "l"(b0), "r"(idesc), "r"((uint32_t)acc_first),
          "n"(SA::at(1)), "n"(SB::at(1)), "n"(SA::at(2)), "n"(SB::at(2)), "n"(SA::at(3)), "n"(SB::at(3)), "n"(SA::at(4)), "n"(SB::at(4)),
          "n"(SA::at(5)), "n"(SB::at(5)), "n"(SA::at(6)), "n"(SB::at(6)), "n"(SA::at(7)), "n"(SB::at(7))
        : "memory");
}
// Eight K-slices, A (bf16) in tensor memory, B in shared memory.
template <class SA, class SB>
__device__ __forceinline__ void mma8_ts(uint32_t d_tmem, uint32_t a_tmem0, uint64_t b0, uint32_t idesc, bool acc_first) {
    asm volatile(
        "{\n\t.reg .pred pf, pt;\n\t.reg .b64 b;\n\t.reg .b32 at;\n\t"
        "setp.ne.b32 pf, %4, 0;\n\tsetp.eq.u32 pt, 0, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, pf;\n\t"
        STR_MMA_TAIL_TS(1, 5, 6) STR_MMA_TAIL_TS(2, 7, 8) STR_MMA_TAIL_TS(3, 9, 10) STR_MMA_TAIL_TS(4, 11, 12)
        STR_MMA_TAIL_TS(5, 13, 14) STR_MMA_TAIL_TS(6, 15, 16) STR_MMA_TAIL_TS(7, 17, 18)
        "}"
        ::"r"(d_tmem), "r"(a_tmem0), "l"(b0), "r"(idesc), "r"((uint32_t)acc_first),
          "n"(SA::at(1)), "n"(SB::at(1)), "n"(SA::at(2)), "n"(SB::at(2)), "n"(SA::at(3)), "n"(SB::at(3)), "n"(SA::at(4)), "n"(SB::at(4)),
          "n"(SA::at(5)), "n"(SB::at(5)), "n"(SA::at(6)), "n"(SB::at(6)), "n"(SA::at(7)), "n"(SB::at(7))
        : "memory");
}
// Four K-slices (one 64-column stage), both operands in shared memory.
template <class SA, class SB>
__device__ __forceinline__ void mma4_ss(uint32_t d_tmem, uint64_t a0, uint64_t b0, uint32_t idesc, bool acc_first) {
    asm volatile(
        "{\n\t.reg .pred pf, pt;\n\t.reg .b64 a, b;\n\t"
        "setp.ne.b32 pf, %4, 0;\n\tsetp.eq.u32 pt, 0, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pf;\n\t"
        STR_MMA_TAIL_SS(1, 5, 6) STR_MMA_TAIL_SS(2, 7, 8) STR_MMA_TAIL_SS(3, 9, 10)
        "}"
        ::"r"(d_tmem), "l"(a0), "l"(b0), "r"(idesc), "r"((uint32_t)acc_first),
          "n"(SA::at(1)), "n"(SB::at(1)), "n"(SA::at(2)), "n"(SB::at(2)), "n"(SA::at(3)), "n"(SB::at(3))
        : "memory");
}
#undef STR_MMA_TAIL_SS
#undef STR_MMA_TAIL_TS

// Arrive on an mbarrier when all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void mma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// ---- CTA pairs (cta_group::2) ------------------------------------------------------------------
// Two CTAs of a cluster of two, on neighbouring SMs, run ONE tcgen05.mma of M = 256: CTA r holds rows
// [128 r, 128 r + 128) of A, rows [N/2 r, N/2 r + N/2) of B (both at the same shared-memory offsets in the two CTAs)
// and, in its own tensor memory, rows [128 r, 128 r + 128) of the accumulator.  The instruction is issued by one
// thread of CTA 0 only.  Each SM then reads half the B operand per K-slice that a lone CTA reads for the same
// accumulator width.  Tensor memory is allocated and freed by the same warp of BOTH CTAs.
__device__ __forceinline__ uint32_t cluster_cta_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// All threads of all CTAs of the cluster; orders shared-memory accesses (mbarrier initialisation included) across it.
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The shared::cluster address of `p`'s counterpart (same offset) in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(const void *p, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Tile load into this CTA's shared memory whose bytes are counted on an mbarrier that may live in the pair's
// other CTA (given by its shared::cluster address).
__device__ __forceinline__ void tma_load_2d_pair(void *smem_dst, const CUtensorMap *m, uint32_t bar_cluster_addr, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"((uint64_t)m), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t *smem_slot, uint32_t ncols) {   // whole warp, same warp in both CTAs
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_slot)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {      // whole warp, same warp in both CTAs
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Four K-slices (one 64-column stage) of a pair MMA, both operands in shared memory; issued by ONE thread of CTA 0.
template <class SA, class SB>
__device__ __forceinline__ void mma4_ss_pair(uint32_t d_tmem, uint64_t a0, uint64_t b0, uint32_t idesc, bool acc_first) {
    asm volatile(
        "{\n\t.reg .pred pf, pt;\n\t.reg .b64 a, b;\n\t"
        "setp.ne.b32 pf, %4, 0;\n\tsetp.eq.u32 pt, 0, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, pf;\n\t"
        "add.s64 a, %1, %5;\n\tadd.s64 b, %2, %6;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], a, b, %3, pt;\n\t"
        "add.s64 a, %1, %7;\n\tadd.s64 b, %2, %8;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], a, b, %3, pt;\n\t"
        "add.s64 a, %1, %9;\n\tadd.s64 b, %2, %10;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], a, b, %3, pt;\n\t"
        "}"
        ::"r"(d_tmem), "l"(a0), "l"(b0), "r"(idesc), "r"((uint32_t)acc_first),
          "n"(SA::at(1)), "n"(SB::at(1)), "n"(SA::at(2)), "n"(SB::at(2)), "n"(SA::at(3)), "n"(SB::at(3))
        : "memory");
}
// Arrive, once all pair MMAs issued so far by this thread have completed, on the mbarrier at this offset in each CTA
// of `cta_mask` (bit r = CTA r of the cluster).
__device__ __forceinline__ void mma_commit_pair(uint64_t *bar, uint16_t cta_mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(cta_mask)
                 : "memory");
}

// TMEM -> registers: 32 lanes x 32-bit, 32 consecutive columns; thread i of the warp reads lane
// (lane_base + i).  The warp may only touch the lane quadrant 32*(warp_id % 4).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
// 16 consecutive 32-bit columns of this thread's lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
// 8 consecutive 32-bit columns of this thread's lane
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&v)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "r"(taddr)
                 : "memory");
}
// Wait for this thread's tensor-memory loads; `v` (the registers of a load still in flight) is named as read and
// written so that no use of it can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait8(uint32_t (&v)[8]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7])
                 :
                 : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
          "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
          "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}
// registers -> TMEM, 16 consecutive 32-bit columns of this thread's lane
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&v)[8]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 2^x on the special-function unit (relative error about 2^-22; -inf and very negative inputs give +0).
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// log2(x) on the special-function unit (log2(0) = -inf).
__device__ __forceinline__ float lg2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

}  // namespace tc

// ---- host: tensor maps ------------------------------------------------------------------------
// 2-D row-major bf16 tensor [rows][cols] (cols contiguous), box [box_rows][box_cols], swizzle mode
// chosen so that box_cols * 2 bytes equals the swizzle span (128 B for 64 columns).
static inline int str_make_tmap_2d_bf16(str_ctx *ctx, CUtensorMap *map, const void *base, uint64_t rows,
                                        uint64_t cols, uint64_t row_stride_elems, uint32_t box_rows,
                                        uint32_t box_cols, CUtensorMapSwizzle swz) {
    typedef CUresult (*encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    if (!ctx->encode_tiled) return STR_ERR_CUDA;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {row_stride_elems * 2};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = ((encode_fn)ctx->encode_tiled)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims,
                                                strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? STR_OK : STR_ERR_CUDA;
}

// 3-D bf16 tensor [outer][rows][inner] (inner contiguous, rows stride = inner, outer stride = rows * inner),
// box [1][box_rows][64] with 128-byte swizzle: one box is a 64-column slice of box_rows rows.
static inline int str_make_tmap_3d_bf16_sw128(str_ctx *ctx, CUtensorMap *map, const void *base, uint64_t inner,
                                              uint64_t rows, uint64_t outer, uint32_t box_rows) {
    typedef CUresult (*encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    if (!ctx->encode_tiled) return STR_ERR_CUDA;
    cuuint64_t dims[3] = {inner, rows, outer};
    cuuint64_t strides[2] = {inner * 2, inner * rows * 2};
    cuuint32_t box[3] = {64, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = ((encode_fn)ctx->encode_tiled)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims,
                                                strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? STR_OK : STR_ERR_CUDA;
}
