// Shared-memory staging of 32-token tiles with bulk-async (TMA, 1-D) copies and mbarriers.
//
// Each warp owns a small ring of stage buffers.  Lane 0 issues, for one tile, one bulk copy: a page
// block is two 32-token halves, each holding its code chunks, mantissa planes, metadata and value
// chunks one after another exactly as the stage buffer does.  It completes on the stage's
// mbarrier, which the whole warp then polls.  Every wait is bounded: after kWaitLimit unsuccessful
// polls the caller poisons its result with NaN and leaves its loop instead of spinning on.
// Copies are plain (no cluster qualifier): every block stages its own tiles.
#pragma once
#include "sa_common.cuh"

namespace sa {

constexpr int kStages = 2;                    // stage buffers per warp
constexpr uint32_t kWaitLimit = 1u << 18;     // polls of one mbarrier phase before giving up

SA_D uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

SA_D void mbar_init(uint32_t mbar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(count) : "memory");
}
SA_D void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
SA_D void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// orders this thread's earlier plain global stores before bulk-async copies that read them
SA_D void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
// one arrival that also announces `bytes` of pending copy traffic
SA_D void mbar_arrive_expect_tx(uint32_t mbar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(bytes) : "memory");
}
SA_D void mbar_arrive(uint32_t mbar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(mbar) : "memory");
}
SA_D bool mbar_try_wait(uint32_t mbar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(mbar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait for a phase; false if it did not complete within `limit` polls.
SA_D bool mbar_wait_bounded(uint32_t mbar, uint32_t parity, uint32_t limit = kWaitLimit) {
    for (uint32_t it = 0; it < limit; ++it)
        if (mbar_try_wait(mbar, parity)) return true;
    return false;
}
// The 16 bytes of key codes of this lane's key in one chunk of a staged tile (one 128-bit load; with
// SA_ABLATE_WORD_STAGING four 32-bit loads that the compiler may not merge).
SA_D uint4 load_code_chunk(const uint32_t* p) {
#ifndef SA_ABLATE_WORD_STAGING
    return *reinterpret_cast<const uint4*>(p);
#else
    uint4 v;
    const uint32_t addr = smem_addr(p);
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v.x) : "r"(addr));
    asm volatile("ld.shared.u32 %0, [%1+4];" : "=r"(v.y) : "r"(addr));
    asm volatile("ld.shared.u32 %0, [%1+8];" : "=r"(v.z) : "r"(addr));
    asm volatile("ld.shared.u32 %0, [%1+12];" : "=r"(v.w) : "r"(addr));
    return v;
#endif
}
// global -> shared bulk copy; size and both addresses are multiples of 16 bytes
SA_D void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t mbar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(mbar)
                 : "memory");
}

// Ask for `bytes` (a multiple of 16) at src to be brought into L2; a hint that changes no state the
// program can observe.
SA_D void bulk_prefetch_l2(const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}

// Layout of one stage buffer: [code chunks: CHUNKS x 512 B][mantissa bit planes: PLANES x 32 rows of
// PLANE_ROW bytes (dense planar container only)][metadata: 128 B or none][value chunks: VROW_BYTES / 16 x 512 B,
// chunk c = 16 dims of the 32 tokens after one another, as in the page].
template <int CHUNKS, bool HAS_META, int VROW_BYTES, int PLANES = 0, int PLANE_ROW = 0>
struct TileStage {
    static constexpr int kCodeBytes = CHUNKS * 512;
    static constexpr int kPlaneOff = kCodeBytes;
    static constexpr int kPlaneBytes = 32 * PLANE_ROW;          // one plane of one tile
    static constexpr int kMetaOff = kPlaneOff + PLANES * kPlaneBytes;
    static constexpr int kMetaBytes = HAS_META ? 128 : 0;
    static constexpr int kVOff = kMetaOff + kMetaBytes;
    static constexpr int kVBytes = 32 * VROW_BYTES;
    static constexpr int kBytes = kVOff + kVBytes;            // a multiple of 128

    // Issued by one lane.  `block` is the (page, KV head) block, tk0 the tile's first token (0 or 32): the
    // tile is that half of the block, which is laid out exactly like the stage buffer, so it is one copy.
    // with_codes / with_values: which parts of the tile the caller needs (at least one of them); the
    // metadata sits between the two and comes with either.
    SA_D static void issue(uint32_t dst, const uint8_t* block, int tk0, uint32_t mbar, bool with_codes = true,
                           bool with_values = true) {
        const uint8_t* half = block + (size_t)(tk0 >> 5) * kBytes;
        const uint32_t lo = with_codes ? 0u : (uint32_t)kMetaOff;
        const uint32_t hi = with_values ? (uint32_t)kBytes : (uint32_t)kVOff;
        mbar_arrive_expect_tx(mbar, hi - lo);
        bulk_g2s(dst + lo, half + lo, hi - lo, mbar);
    }
    // Metadata and values only, for a stage plan without code chunks (CHUNKS = 0, PLANES = 0) reading a block
    // whose halves do hold codes: the two parts follow one another from meta_off to the end of the half.
    SA_D static void issue_values(uint32_t dst, const uint8_t* block, size_t page_bytes, size_t meta_off, int tk0,
                                  uint32_t mbar) {
        static_assert(CHUNKS == 0 && PLANES == 0, "the stage holds metadata and values only");
        mbar_arrive_expect_tx(mbar, (uint32_t)kBytes);
        bulk_g2s(dst, block + (size_t)(tk0 >> 5) * (page_bytes >> 1) + meta_off, (uint32_t)kBytes, mbar);
    }
    // The same range as issue(), as an L2 prefetch hint.
    SA_D static void prefetch(const uint8_t* block, int tk0, bool with_values) {
        bulk_prefetch_l2(block + (size_t)(tk0 >> 5) * kBytes, with_values ? (uint32_t)kBytes : (uint32_t)kVOff);
    }
};

}  // namespace sa
