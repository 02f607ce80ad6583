// Building blocks of the shared-memory tile ring used by the streaming kernels: a thread issues 1-D bulk
// asynchronous copies (cp.async.bulk) of 16 KB tiles into a small ring of stages; each stage has an mbarrier
// that completes when the tile's bytes have landed (complete_tx).  No cluster: every copy goes
// into the issuing CTA's own shared memory.  Every wait is bounded.
#pragma once
#include "common.cuh"

namespace cadd {

constexpr int kTopkUnroll = 4;            // chunks per thread per tile
constexpr int kTileChunks = kTopkUnroll * kThreads;   // 16-byte chunks per tile (16 KB)
constexpr int kStages = 3;                // tiles in flight per CTA
constexpr int kRunChunks = kTileChunks / (kThreads / 32);   // a warp's share of a tile when each warp takes a contiguous run: 128 chunks = 2 KB
constexpr int kSpinLimit = 1 << 16;       // bounded waits: tries of up to ~2 us each (mbarrier), or plain polls

// First statement of a kernel that may be launched while the previous kernel of its stream still runs (programmatic
// stream serialization): returns when that kernel has completed and its writes are visible; a no-op otherwise.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel of the stream be dispatched from now on (it still waits, in its own first statement, for this
// kernel to complete).  Only worth calling where the next kernel is tiny: its CTAs hold their resources while they wait.
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One try: the hardware may park the thread for up to `hint_ns` while the phase is incomplete, so a waiting
// warp does not burn issue slots.
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity, unsigned hint_ns = 2000u) {
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns) : "memory");
    return ok != 0;
}
// Wait for a phase with an iteration limit; false = gave up (the caller flags an error and leaves).
__device__ __forceinline__ bool mbar_wait_limited(uint64_t* bar, unsigned parity, int limit) {
    for (int it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(200);          // a waiting warp must not take issue slots from the warps that still work
    }
    return false;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, unsigned parity) { return mbar_wait_limited(bar, parity, kSpinLimit); }

// Test hook of the streaming kernels (the TEST_DROP_TILE flags of the C ABI): the copy of one tile per row is never
// issued, and the wait for that tile alone gives up after kTestSpinLimit tries, so that the time-out path runs with
// nothing in flight for the barrier that is given up on.  Every other wait keeps the full limit.
constexpr int kTestSpinLimit = 4;
__device__ __forceinline__ int tile_wait_limit(int t, int fault_tile) { return t == fault_tile ? kTestSpinLimit : kSpinLimit; }

// Ring bookkeeping for the exit path after a wait ran out: last_seq[s] is the sequence number g of the last tile issued
// into stage s (tile g goes to stage g % kStages and completes phase (g / kStages) & 1 of that stage's barrier), kNoTile
// if none.  ring_drain, called by ONE thread once every warp of the CTA has left its tile loop, waits (with the full
// limit per stage) until every issued copy has landed, so that the CTA never exits with a bulk copy still writing into
// its shared memory.  A tile that has landed already, consumed or not, costs one successful try.
constexpr unsigned kNoTile = 0xffffffffu;
__device__ __forceinline__ void ring_drain(uint64_t* full, const volatile unsigned* last_seq) {
    for (int s = 0; s < kStages; ++s) {
        const unsigned g = last_seq[s];
        if (g != kNoTile) mbar_wait_bounded(&full[s], (g / kStages) & 1u);
    }
}
// 1-D bulk copy global -> this CTA's shared memory; both addresses 16-byte aligned, bytes % 16 == 0.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}


}  // namespace cadd
