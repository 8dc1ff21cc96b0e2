// Inline-PTX wrappers for sm_100a: mbarrier, TMA (cp.async.bulk.tensor), tcgen05
// (TMEM allocation, MMA, commit, load) and cluster helpers.
#pragma once
#include <cuda_fp16.h>
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace kx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint64_t globaltimer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}


// ------------------------------------------------------------------ cluster
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cta address of this CTA -> shared::cluster address of the same offset in CTA `rank`
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_arrive() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
// arrival without memory ordering: for barriers that only keep the CTAs of a cluster alive, where no data
// is handed over
__device__ __forceinline__ void cluster_arrive_relaxed() {
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float4 ld_cluster_f32x4(uint32_t cluster_addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "r"(cluster_addr)
                 : "memory");
    return v;
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}

// ------------------------------------------------------------------ mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// arrive on a barrier that may live in another CTA of the cluster
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr)
                 : "memory");
}
// the same without ordering of its own (the caller has issued a fence at cluster scope)
__device__ __forceinline__ void mbar_arrive_cluster_relaxed(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// non-blocking test of a phase (no suspension): the result can be read long after the instruction was issued
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// the same test with acquire semantics at cluster scope: pairs with arrivals made by other CTAs of the cluster
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void fence_acq_rel_cluster() { asm volatile("fence.acq_rel.cluster;" ::: "memory"); }

// ------------------------------------------------------------------ fences
__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// ------------------------------------------------------------------ TMA
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* m) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
// 2-D tiled load global -> this CTA's shared memory, completion on this CTA's mbarrier
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* m, int x, int y,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(m)), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// same, inside a CTA pair: the mbarrier (a shared::cluster address) may be the peer's
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* m, int x, int y,
                                                 uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.cta_group::2 "
        "[%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(m)), "r"(x), "r"(y), "r"(bar_cluster)
        : "memory");
}
// Bulk copy from this CTA's shared memory into the shared memory of a CTA of the cluster (dst and bar are
// shared::cluster addresses of the destination CTA); the bytes are counted on the destination's mbarrier.
// Source, destination and size are multiples of 16 bytes.  The source must have been made visible to the
// asynchronous proxy (fence.proxy.async) and must stay intact until the destination's barrier completes.
__device__ __forceinline__ void bulk_copy_to_cta(uint32_t dst_cluster, uint32_t src_cta, uint32_t bytes,
                                                 uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            dst_cluster),
        "r"(src_cta), "r"(bytes), "r"(bar_cluster)
        : "memory");
}
// Untiled bulk copy global -> this CTA's shared memory (both 16-byte aligned, size a multiple of 16 bytes); the
// bytes are counted on `bar` (a barrier of this CTA).
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// Orders this thread's earlier generic-proxy accesses (here: an acquire load that made another CTA's global
// stores visible) before its later asynchronous-proxy operations.
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
// Ask for a 2-D tile to be brought into L2 (no shared-memory destination, no completion signal).
// L2 is the coherence point of the device, so a tile prefetched early still reflects any later
// write made through L2 before it is actually loaded.
__device__ __forceinline__ void tma_prefetch_l2_2d(const CUtensorMap* m, int x, int y) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(
                     reinterpret_cast<uint64_t>(m)),
                 "r"(x), "r"(y)
                 : "memory");
}
// Four binary32 values -> four E4M3 codes (b0 lowest): round to nearest even, saturate to +-448.
__device__ __forceinline__ uint32_t pack_e4m3x4(float b0, float b1, float b2, float b3) {
    uint16_t lo, hi;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(b1), "f"(b0));
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(b3), "f"(b2));
    return static_cast<uint32_t>(lo) | (static_cast<uint32_t>(hi) << 16);
}
// Four 32-bit integers -> four signed bytes (b0 lowest), each saturated to [-128, 127].
__device__ __forceinline__ uint32_t pack_s8x4_sat(int b0, int b1, int b2, int b3) {
    uint32_t hi, d;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, 0;" : "=r"(hi) : "r"(b3), "r"(b2));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(b1), "r"(b0), "r"(hi));
    return d;
}
// 2-D tiled store shared -> global (bulk async group)
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* m, int x, int y, uint32_t src) {
    asm volatile(
        "cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
            reinterpret_cast<uint64_t>(m)),
        "r"(x), "r"(y), "r"(src)
        : "memory");
}
__device__ __forceinline__ void tma_store_commit() {
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void tma_store_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void tma_store_wait_all() {
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}

// ------------------------------------------------------------------ TMEM
template <int CTAS>
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    if constexpr (CTAS == 1)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst),
                     "r"(ncols)
                     : "memory");
    else
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst),
                     "r"(ncols)
                     : "memory");
}
template <int CTAS>
__device__ __forceinline__ void tmem_relinquish() {
    if constexpr (CTAS == 1)
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    else
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
template <int CTAS>
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    if constexpr (CTAS == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
                     : "memory");
    else
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
                     : "memory");
}

// ------------------------------------------------------------------ MMA
// Shared-memory matrix descriptor, K-major operand tile whose rows are 64 BF16
// (128 bytes) written by TMA with the 128-byte swizzle: 8-row groups are 1024
// bytes apart (stride byte offset), descriptor version 1, layout = SWIZZLE_128B.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);       // start address
    d |= static_cast<uint64_t>(1) << 16;                           // leading byte offset (unused here)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;                   // stride byte offset
    d |= static_cast<uint64_t>(1) << 46;                           // descriptor version (sm_100)
    d |= static_cast<uint64_t>(2) << 61;                           // SWIZZLE_128B
    return d;
}
// Instruction descriptor: BF16 x BF16 -> FP32, both operands K-major, dense.
__host__ __device__ constexpr uint32_t idesc_bf16_f32(int mma_m, int mma_n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(mma_n >> 3) << 17) |
           (static_cast<uint32_t>(mma_m >> 4) << 24);
}
// Instruction descriptor: S8 x S8 -> S32 (integer accumulate), both operands K-major, dense.
__host__ __device__ constexpr uint32_t idesc_s8_s32(int mma_m, int mma_n) {
    return (2u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(mma_n >> 3) << 17) |
           (static_cast<uint32_t>(mma_m >> 4) << 24);
}
// One K = 32 step of signed 8-bit operands into 32-bit integer accumulators in tensor memory.
template <int CTAS>
__device__ __forceinline__ void mma_s8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
    if constexpr (CTAS == 1)
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
            "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
            "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
}
// Instruction descriptor: E4M3 x E4M3 -> FP32, both operands K-major, dense.
__host__ __device__ constexpr uint32_t idesc_e4m3_f32(int mma_m, int mma_n) {
    return (1u << 4) | (static_cast<uint32_t>(mma_n >> 3) << 17) | (static_cast<uint32_t>(mma_m >> 4) << 24);
}
// One K = 32 step of FP8 operands (byte-packed) into FP32 accumulators in tensor memory.
template <int CTAS>
__device__ __forceinline__ void mma_f8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
    if constexpr (CTAS == 1)
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
            "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
            "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
}
template <int CTAS>
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                         uint32_t accumulate) {
    if constexpr (CTAS == 1)
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
            "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
            "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
}
// One k-block (128 bytes of K per operand row) from a single inline block, in the order that keeps
// the issuing lane busy: (1) a non-blocking test of the NEXT stage's `full` barrier, whose latency
// then overlaps everything below; (2) the four K steps, their shared-memory descriptors assembled
// from low words: `a_lo` / `b_lo` are the low 32 bits of the K-major SWIZZLE_128B descriptors of
// the stage's A and B tiles (start address >> 4, leading byte offset field), `desc_hi` the
// constant high word, and a K step advances the start address by 32 bytes = 2 in the low word
// (shared-memory addresses are below 2^18, so the 14-bit field never carries); (3) the commit
// that releases the stage (to both CTAs of a pair); (4) only now the test's result is read.
// `acc_first` = 0 makes the first step overwrite the accumulator.  Returns 1 if the next stage was
// already full.
#define KX_MMA_STEPS(GROUP, KINDSTR, A, B, P0)                                                              \
        "mov.b64 da, {" A ", %6};\n\t"                                                                      \
        "mov.b64 db, {" B ", %6};\n\t"                                                                      \
        "tcgen05.mma.cta_group::" GROUP ".kind::" KINDSTR " [%1], da, db, %4, " P0 ";\n\t"                  \
        "add.u32 al, " A ", 2;\n\tadd.u32 bl, " B ", 2;\n\tmov.b64 da, {al, %6};\n\tmov.b64 db, {bl, %6};\n\t" \
        "tcgen05.mma.cta_group::" GROUP ".kind::" KINDSTR " [%1], da, db, %4, q;\n\t"                      \
        "add.u32 al, " A ", 4;\n\tadd.u32 bl, " B ", 4;\n\tmov.b64 da, {al, %6};\n\tmov.b64 db, {bl, %6};\n\t" \
        "tcgen05.mma.cta_group::" GROUP ".kind::" KINDSTR " [%1], da, db, %4, q;\n\t"                      \
        "add.u32 al, " A ", 6;\n\tadd.u32 bl, " B ", 6;\n\tmov.b64 da, {al, %6};\n\tmov.b64 db, {bl, %6};\n\t" \
        "tcgen05.mma.cta_group::" GROUP ".kind::" KINDSTR " [%1], da, db, %4, q;\n\t"
#define KX_MMA_HEAD                                                                                        \
        "{\n\t.reg .pred p, q, r;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"                          \
        "mbarrier.test_wait.parity.shared::cta.b64 r, [%7], %8;\n\t"                                       \
        "setp.ne.b32 p, %5, 0;\n\t"                                                                        \
        "setp.eq.b32 q, %1, %1;\n\t"
#define KX_MMA_TAIL1 \
        "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%9];\n\t"                  \
        "selp.u32 %0, 1, 0, r;\n\t}"
#define KX_MMA_TAIL2 \
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%9];\n\t"                  \
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%10];\n\t"                 \
        "selp.u32 %0, 1, 0, r;\n\t}"
#define KX_MMA_OPERANDS                                                                                    \
        : "=r"(next_ok)                                                                                    \
        : "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(acc_first), "r"(desc_hi), "r"(next_full),     \
          "r"(next_parity), "r"(empty0), "r"(empty1), "r"(a_lo2), "r"(b_lo2)                               \
        : "memory"
// one k-block per stage
#define KX_MMA_KBLOCK(GROUP, KINDSTR, TAIL)                                                                \
    asm volatile(KX_MMA_HEAD KX_MMA_STEPS(GROUP, KINDSTR, "%2", "%3", "p") TAIL KX_MMA_OPERANDS)
// two k-blocks per stage: eight K steps between one barrier test and one commit
#define KX_MMA_KBLOCK_X2(GROUP, KINDSTR, TAIL)                                                             \
    asm volatile(KX_MMA_HEAD KX_MMA_STEPS(GROUP, KINDSTR, "%2", "%3", "p")                                 \
                 KX_MMA_STEPS(GROUP, KINDSTR, "%11", "%12", "q") TAIL KX_MMA_OPERANDS)
constexpr uint32_t kDescHiSw128 = (1024u >> 4) | (1u << 14) | (2u << 29);   // SBO 1024 B, version 1, SWIZZLE_128B
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t smem_addr) {
    return ((smem_addr & 0x3FFFFu) >> 4) | (1u << 16);
}
// KIND: 0 = BF16 (kind::f16), 1 = signed 8-bit (kind::i8), 2 = FP8 E4M3 (kind::f8f6f4).
// empty0 / empty1: shared::cluster addresses of the stage's `empty` barrier in CTA 0 / CTA 1 of
// the pair (empty1 unused for CTAS == 1); next_full / next_parity: the next stage's `full` barrier.
// TWO: the stage holds a second k-block whose descriptors' low words are a_lo2 / b_lo2.
template <int CTAS, int KIND, bool TWO>
__device__ __forceinline__ uint32_t mma_kblock(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                               uint32_t acc_first, uint32_t next_full, uint32_t next_parity,
                                               uint32_t empty0, uint32_t empty1, uint32_t a_lo2 = 0,
                                               uint32_t b_lo2 = 0) {
    const uint32_t desc_hi = kDescHiSw128;
    uint32_t next_ok;
#define KX_MMA_DISPATCH(GROUP, TAIL)                                                                       \
    if constexpr (TWO) {                                                                                   \
        if constexpr (KIND == 1) KX_MMA_KBLOCK_X2(GROUP, "i8", TAIL);                                      \
        else if constexpr (KIND == 2) KX_MMA_KBLOCK_X2(GROUP, "f8f6f4", TAIL);                             \
        else KX_MMA_KBLOCK_X2(GROUP, "f16", TAIL);                                                         \
    } else {                                                                                               \
        if constexpr (KIND == 1) KX_MMA_KBLOCK(GROUP, "i8", TAIL);                                         \
        else if constexpr (KIND == 2) KX_MMA_KBLOCK(GROUP, "f8f6f4", TAIL);                                \
        else KX_MMA_KBLOCK(GROUP, "f16", TAIL);                                                            \
    }
    if constexpr (CTAS == 1) {
        KX_MMA_DISPATCH("1", KX_MMA_TAIL1)
    } else {
        KX_MMA_DISPATCH("2", KX_MMA_TAIL2)
    }
#undef KX_MMA_DISPATCH
    return next_ok;
}
#undef KX_MMA_KBLOCK
#undef KX_MMA_KBLOCK_X2
#undef KX_MMA_OPERANDS
#undef KX_MMA_TAIL1
#undef KX_MMA_TAIL2
#undef KX_MMA_HEAD
#undef KX_MMA_STEPS
// ------------------------------------------------------------------ block-scaled FP8 (kind::mxf8f6f4)
// Instruction descriptor of the block-scaled kind: E4M3 A and B (format 0), both K-major, E8M0
// scales (bit 23), N >> 3 at bit 17, M >> 4 at bit 24.  The byte of the scale column that a K = 32
// step uses (0..3 = which 32-element block of the 128-element k-block) goes into bits 4..5 (B) and
// 29..30 (A).
__host__ __device__ constexpr uint32_t idesc_mxf8(int m, int n) {
    return (1u << 23) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}
// One k-block (128 FP8 elements) of the block-scaled kind in a single instruction block: the scale
// chunks (A, then CHUNKS of B, 512 bytes apart in shared memory; each 32 rows x 16 bytes, described
// K-major without swizzle, 8-row core matrices 128 bytes apart) are copied to TMEM columns cols,
// cols + 4 (, cols + 8) - 4 columns each, the same data in every 32-lane quarter; with a CTA pair
// each CTA copies from its own shared memory into its own tensor memory - then four K = 32 steps, step i reading byte i of the scale columns (sfb = first
// scale column of the tile's B rows).  a_lo / b_lo / sf_lo are the low words of the shared-memory
// descriptors; acc_first = 0 makes step 0 overwrite the accumulator.
#define KX_MX_CP(G, OFFS, OFFT)                                                                            \
        "add.u32 t, %6, " OFFS ";\n\tmov.b64 ds, {t, %7};\n\tadd.u32 sa, %8, " OFFT ";\n\t"               \
        "tcgen05.cp.cta_group::" G ".32x128b.warpx4 [sa], ds;\n\t"
#define KX_MX_STEP(G, KOFF, IDOFF, SFOFF, P)                                                               \
        "add.u32 al, %1, " KOFF ";\n\tadd.u32 bl, %2, " KOFF ";\n\tmov.b64 da, {al, %4};\n\tmov.b64 db, {bl, %4};\n\t" \
        "add.u32 id, %3, " IDOFF ";\n\tadd.u32 sa, %8, " SFOFF ";\n\tadd.u32 sb, %9, " SFOFF ";\n\t"         \
        "tcgen05.mma.cta_group::" G ".kind::mxf8f6f4.block_scale [%0], da, db, id, [sa], [sb], " P ";\n\t"
#define KX_MX_BODY(G, CP2)                                                                                 \
    asm volatile(                                                                                          \
        "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db, ds;\n\t.reg .b32 al, bl, t, sa, sb, id;\n\t"          \
        "setp.ne.b32 p, %5, 0;\n\tsetp.eq.b32 q, %0, %0;\n\t"                                             \
        KX_MX_CP(G, "0", "0") KX_MX_CP(G, "32", "4") CP2                                                   \
        KX_MX_STEP(G, "0", "0", "0", "p")                                                                  \
        KX_MX_STEP(G, "2", "0x20000010", "0x40000000", "q")                                                \
        KX_MX_STEP(G, "4", "0x40000020", "0x80000000", "q")                                                \
        KX_MX_STEP(G, "6", "0x60000030", "0xC0000000", "q")                                                \
        "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(desc_hi), "r"(acc_first), "r"(sf_lo),     \
        "r"(sf_hi), "r"(cols), "r"(sfb)                                                                    \
        : "memory")
template <int CTAS, int CHUNKS>
__device__ __forceinline__ void mma_kblock_mx(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                              uint32_t acc_first, uint32_t sf_lo, uint32_t cols, uint32_t sfb) {
    const uint32_t desc_hi = kDescHiSw128;
    const uint32_t sf_hi = (128u >> 4) | (1u << 14);
    if constexpr (CTAS == 1) {
        if constexpr (CHUNKS == 2) KX_MX_BODY("1", KX_MX_CP("1", "64", "8"));
        else KX_MX_BODY("1", "");
    } else {
        if constexpr (CHUNKS == 2) KX_MX_BODY("2", KX_MX_CP("2", "64", "8"));
        else KX_MX_BODY("2", "");
    }
}

#undef KX_MX_BODY
#undef KX_MX_STEP
#undef KX_MX_CP

// ------------------------------------------------------------------ 4-bit block-scaled kind (kind::mxf4nvf4)
// E2M1 elements packed two per byte (a 128-byte swizzle row holds 256 of them = four K = 64 steps), one
// E4M3 scale per 16 elements: a K = 64 step reads all four bytes of a 32-bit scale column per row.
// Instruction descriptor: A = B = E2M1 (format 1), K-major, E4M3 scales (bit 23 clear).
__host__ __device__ constexpr uint32_t idesc_nvf4(int m, int n) {
    return (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}
// One k-block: for each of its four K = 64 steps, the step's scale chunks (A, then CHUNKS of B; the four
// steps' chunks of one operand are contiguous, 512 bytes each, operands 2048 bytes apart) are copied to 12
// TMEM columns of their own, then the step is issued.  sfb_off = first scale column of the tile's B rows
// inside the B chunks.
template <int CHUNKS>
__device__ __forceinline__ void mma_kblock_nv(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                              uint32_t acc_first, uint32_t sf_lo, uint32_t cols, uint32_t sfb_off) {
    const uint64_t hi = static_cast<uint64_t>(kDescHiSw128) << 32;
    const uint64_t sf_hi = static_cast<uint64_t>((128u >> 4) | (1u << 14)) << 32;
#pragma unroll
    for (uint32_t i = 0; i < 4; ++i) {
        const uint32_t c = cols + 12u * i;
        asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(c), "l"(sf_hi | (sf_lo + 32u * i)) : "memory");
        asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(c + 4u), "l"(sf_hi | (sf_lo + 128u + 32u * i))
                     : "memory");
        if constexpr (CHUNKS == 2)
            asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(c + 8u),
                         "l"(sf_hi | (sf_lo + 256u + 32u * i))
                         : "memory");
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.scale_vec::4X [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
            ::"r"(d_tmem), "l"(hi | (a_lo + 2u * i)), "l"(hi | (b_lo + 2u * i)), "r"(idesc),
              "r"((acc_first != 0u || i > 0u) ? 1u : 0u), "r"(c), "r"(c + 4u + sfb_off)
            : "memory");
    }
}
// The two halves of the above for kernels in which another thread copies the scales: all copies of a k-block
// (step i: A chunk and CHUNKS of B into columns cols + 12 i ...) and the four K = 64 steps alone.
template <int CHUNKS>
__device__ __forceinline__ void sf_copy_nv(uint32_t sf_lo, uint32_t cols, uint32_t step0, uint32_t step1) {
    const uint64_t sf_hi = static_cast<uint64_t>((128u >> 4) | (1u << 14)) << 32;
#pragma unroll
    for (uint32_t i = step0; i < step1; ++i) {
        const uint32_t c = cols + 12u * i;
        asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(c), "l"(sf_hi | (sf_lo + 32u * i)) : "memory");
        asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(c + 4u), "l"(sf_hi | (sf_lo + 128u + 32u * i))
                     : "memory");
        if constexpr (CHUNKS == 2)
            asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(c + 8u),
                         "l"(sf_hi | (sf_lo + 256u + 32u * i))
                         : "memory");
    }
}
__device__ __forceinline__ void mma_kblock_nv_steps(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                                    uint32_t acc_first, uint32_t cols, uint32_t sfb_off) {
    const uint64_t hi = static_cast<uint64_t>(kDescHiSw128) << 32;
#pragma unroll
    for (uint32_t i = 0; i < 4; ++i) {
        const uint32_t c = cols + 12u * i;
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.scale_vec::4X [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
            ::"r"(d_tmem), "l"(hi | (a_lo + 2u * i)), "l"(hi | (b_lo + 2u * i)), "r"(idesc),
              "r"((acc_first != 0u || i > 0u) ? 1u : 0u), "r"(c), "r"(c + 4u + sfb_off)
            : "memory");
    }
}
// two binary32 values -> one byte of two E2M1 codes (nearest, ties to even, saturating): `lo` in the low nibble
__device__ __forceinline__ uint32_t pack_e2m1x8(const float (&z)[8]) {
    uint32_t r;
    asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
        "mov.b32 %0, {b0, b1, b2, b3};\n\t}"
        : "=r"(r)
        : "f"(z[0]), "f"(z[1]), "f"(z[2]), "f"(z[3]), "f"(z[4]), "f"(z[5]), "f"(z[6]), "f"(z[7]));
    return r;
}
// one E4M3 byte -> binary32 (exact)
__device__ __forceinline__ float e4m3_to_f32(uint32_t byte) {
    uint32_t h2;
    asm("{\n\t.reg .b16 t;\n\tcvt.u16.u32 t, %1;\n\tcvt.rn.f16x2.e4m3x2 %0, t;\n\t}" : "=r"(h2) : "r"(byte & 0xFFu));
    return __half2float(__ushort_as_half(static_cast<unsigned short>(h2 & 0xFFFFu)));
}

// Arrive on an mbarrier once every MMA issued so far by this thread has finished.
// `bar` is a shared::cluster address (this CTA's own shared::cta address is one).
template <int CTAS>
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    if constexpr (CTAS == 1)
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                     : "memory");
    else
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                     : "memory");
}

// TMEM -> registers: this warp's 32 lanes x 32 consecutive FP32 columns.
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
          "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
          "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
          "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
          "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
// registers -> TMEM: this warp's 32 lanes x 32 consecutive FP32 columns
__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]),
        "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]),
        "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() {
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ------------------------------------------------------------------ programmatic dependent launch
// Block until the kernel(s) this launch depends on have completed and their writes are
// visible.  A no-op when the kernel was launched without programmatic serialization.
__device__ __forceinline__ void pdl_wait_prior() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Allow the next kernel in the stream to start its own prologue.
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ------------------------------------------------------------------ misc
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xFFFF0000u); }

}  // namespace kx
