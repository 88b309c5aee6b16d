// tcgen05 / TMA / cluster PTX wrappers shared by the tensor-core kernels (the dense matcher and the
// fused gather-linear-scatter kernel).  Everything here is a thin wrapper around one instruction, or
// around one instruction block whose internal order matters.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace oc {

// ---- PTX wrappers ------------------------------------------------------------------------------
__device__ __forceinline__ void tma_prefetch_map(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" :: "l"(map) : "memory");
}
// arrive on a barrier given by its cluster-wide shared address (own CTA or the other CTA of a pair).
// What the arrival orders here are reads of tensor memory, which the tcgen05 fences around it cover; it
// publishes no ordinary memory to the other CTA, so the default (CTA-scope) release is enough, and a
// cluster-scope one would wait for the thread's outstanding global-memory traffic first.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" :: "r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared address of the same variable in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// In a CTA pair `bar` is the cluster address of the LEADER's barrier: both CTAs' copies report there.
template <bool PAIR>
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint32_t bar) {
    if (PAIR)
        asm volatile(
            "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
            :: "r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
    else
        asm volatile(
            "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
            :: "r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
// The same copy issued by the one lane whose `issue` is non-zero, from code that the whole warp runs:
// addresses and coordinates then stay warp-uniform values (a lone diverged lane would have them moved
// from per-thread to uniform registers before every instruction, which costs it hundreds of cycles).
template <bool PAIR>
__device__ __forceinline__ void tma_load_4d_elected(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                                    uint32_t bar, uint32_t issue) {
    if (PAIR)
        asm volatile(
            "{\n\t.reg .pred e;\n\tsetp.ne.b32 e, %7, 0;\n\t"
            "@e cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];\n\t}"
            :: "r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar), "r"(issue) : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred e;\n\tsetp.ne.b32 e, %7, 0;\n\t"
            "@e cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];\n\t}"
            :: "r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar), "r"(issue) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx_elected(uint32_t bar, uint32_t bytes, uint32_t issue) {
    asm volatile("{\n\t.reg .pred e;\n\tsetp.ne.b32 e, %2, 0;\n\t"
                 "@e mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n\t}" :: "r"(bar), "r"(bytes), "r"(issue) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// arrive on `bar` once every MMA issued so far by this thread has retired
// The MMA warp runs its loop with all 32 lanes (so that addresses and descriptors are warp-uniform
// values); `issue` is non-zero in the one elected lane that actually issues.
template <bool PAIR>
__device__ __forceinline__ void tc_commit(uint32_t bar, uint32_t issue = 1u) {
    if (PAIR)
        asm volatile("{\n\t.reg .pred e;\n\tsetp.ne.b32 e, %1, 0;\n\t"
                     "@e tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
                     :: "r"(bar), "r"(issue) : "memory");
    else
        asm volatile("{\n\t.reg .pred e;\n\tsetp.ne.b32 e, %1, 0;\n\t"
                     "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
                     :: "r"(bar), "r"(issue) : "memory");
}
__device__ __forceinline__ uint32_t elect_one() {
    uint32_t e;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xFFFFFFFF;\n\tselp.b32 %0, 1, 0, p;\n\t}" : "=r"(e));
    return e;
}
template <bool PAIR>
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate, uint32_t issue) {
    if (PAIR)
        asm volatile(
            "{\n\t.reg .pred p, e;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "setp.ne.b32 e, %5, 0;\n\t"
            "@e tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(issue) : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p, e;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "setp.ne.b32 e, %5, 0;\n\t"
            "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(issue) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// All MMAs of one 64-channel stage (4 steps of K = 16, for one or two candidate tiles), with a look at
// the NEXT stage's barrier folded in: the test is issued before the last MMAs and its answer read
// after them, so the ~150 cycles it takes to come back pass while those MMAs queue up instead of
// between two stages (the tensor pipe accepts an MMA only about when the previous one starts, so
// nothing else hides that gap).
// tile_stride: TMEM columns between the accumulators of the two candidate tiles.
// The commits that follow a stage's MMAs are part of the same block -- the one that frees the stage's
// ring slot, when a_empty_bar is non-zero the one that frees a resident candidate slot, and when
// acc_full_bar is non-zero (the piece's last stage) the one that hands the accumulators over -- so that
// nothing the compiler schedules comes between them: in a pair ONE commit with a CTA mask signals the
// barrier at the same address in both CTAs.
// Returns non-zero when the next stage was already full.
#define OC_COMMIT_CG1(bar, pred) "@" pred " tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [" bar "];\n\t"
#define OC_COMMIT_CG2(bar, pred) "@" pred " tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [" bar "], both;\n\t"
#define OC_MMA_STAGE_ASM(CG, TWO, COMMIT)                                                                \
    asm volatile(                                                                                       \
        "{\n\t"                                                                                         \
        ".reg .pred pa, pt, e, r, ea, ef;\n\t"                                                          \
        ".reg .b16 both;\n\t"                                                                           \
        "mov.b16 both, 3;\n\t"                                                                          \
        ".reg .b64 a0, a1, bb;\n\t"                                                                     \
        ".reg .b32 d1;\n\t"                                                                             \
        "setp.ne.b32 pa, %5, 0;\n\t"                                                                    \
        "setp.ne.b32 e, %6, 0;\n\t"                                                                     \
        "setp.eq.b32 pt, 0, 0;\n\t"                                                                     \
        "add.u32 d1, %1, %10;\n\t"                                                                      \
        "@e tcgen05.mma.cta_group::" CG ".kind::f16 [%1], %2, %4, %9, pa;\n\t"                          \
        TWO("@e tcgen05.mma.cta_group::" CG ".kind::f16 [d1], %3, %4, %9, pa;\n\t")                     \
        "add.u64 a0, %2, 2;\n\tadd.u64 a1, %3, 2;\n\tadd.u64 bb, %4, 2;\n\t"                          \
        "@e tcgen05.mma.cta_group::" CG ".kind::f16 [%1], a0, bb, %9, pt;\n\t"                          \
        TWO("@e tcgen05.mma.cta_group::" CG ".kind::f16 [d1], a1, bb, %9, pt;\n\t")                     \
        "add.u64 a0, %2, 4;\n\tadd.u64 a1, %3, 4;\n\tadd.u64 bb, %4, 4;\n\t"                          \
        "@e tcgen05.mma.cta_group::" CG ".kind::f16 [%1], a0, bb, %9, pt;\n\t"                          \
        TWO("@e tcgen05.mma.cta_group::" CG ".kind::f16 [d1], a1, bb, %9, pt;\n\t")                     \
        "mbarrier.test_wait.parity.shared::cta.b64 r, [%7], %8;\n\t"                                    \
        "add.u64 a0, %2, 6;\n\tadd.u64 a1, %3, 6;\n\tadd.u64 bb, %4, 6;\n\t"                          \
        "@e tcgen05.mma.cta_group::" CG ".kind::f16 [%1], a0, bb, %9, pt;\n\t"                          \
        TWO("@e tcgen05.mma.cta_group::" CG ".kind::f16 [d1], a1, bb, %9, pt;\n\t")                     \
        COMMIT("%11", "e")                                                                              \
        "setp.ne.b32 ea, %12, 0;\n\t"                                                                   \
        "and.pred ea, ea, e;\n\t"                                                                       \
        COMMIT("%12", "ea")                                                                             \
        "setp.ne.b32 ef, %13, 0;\n\t"                                                                   \
        "and.pred ef, ef, e;\n\t"                                                                       \
        COMMIT("%13", "ef")                                                                             \
        "selp.b32 %0, 1, 0, r;\n\t"                                                                     \
        "}"                                                                                             \
        : "=r"(ready)                                                                                   \
        : "r"(d_tmem), "l"(a0_desc), "l"(a1_desc), "l"(b_desc), "r"(accumulate), "r"(issue), "r"(next_bar), \
          "r"(next_parity), "r"(idesc), "r"(tile_stride), "r"(empty_bar), "r"(a_empty_bar), "r"(acc_full_bar) \
        : "memory")
#define OC_KEEP(x) x
#define OC_DROP(x)
template <bool PAIR>
__device__ __forceinline__ uint32_t tc_mma_stage(uint32_t d_tmem, uint64_t a0_desc, uint64_t a1_desc, uint64_t b_desc,
                                                 uint32_t idesc, uint32_t accumulate, uint32_t issue, bool two_tiles,
                                                 uint32_t next_bar, uint32_t next_parity, uint32_t tile_stride,
                                                 uint32_t empty_bar, uint32_t a_empty_bar, uint32_t acc_full_bar) {
    uint32_t ready;
    if (two_tiles) {
        if (PAIR) OC_MMA_STAGE_ASM("2", OC_KEEP, OC_COMMIT_CG2); else OC_MMA_STAGE_ASM("1", OC_KEEP, OC_COMMIT_CG1);
    } else {
        if (PAIR) OC_MMA_STAGE_ASM("2", OC_DROP, OC_COMMIT_CG2); else OC_MMA_STAGE_ASM("1", OC_DROP, OC_COMMIT_CG1);
    }
    return ready;
}

// K-major, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
    const uint32_t lo = ((addr >> 4) & 0x3FFFu) | (1u << 16);           // start address, LBO = 16 B (unused)
    const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);         // SBO = 1024 B, version 1, SWIZZLE_128B
    return ((uint64_t)hi << 32) | lo;
}


// ---- TMEM allocation (one warp, .sync.aligned) -------------------------------------------------------
__device__ __forceinline__ void tmem_alloc_cta1(uint32_t slot_smem_addr, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(slot_smem_addr), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_cta1(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(taddr), "r"(cols) : "memory");
}
// 2-D tiled TMA load (no cluster qualifiers): box at {c0 (innermost), c1}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 :: "r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

}  // namespace oc
