// Thin wrappers over the PTX this library uses for asynchronous copies and
// mbarrier pipelines (shared by the two GEMM kernels).  Every wait is bounded:
// after WAIT_LIMIT_NS of %globaltimer the waiter raises the CTA's abort flag,
// latches MOQE_ERR_TIMEOUT and returns false, and every other waiter of the CTA
// returns false at its next poll, so a pipeline that stops moving ends the
// kernel instead of hanging the device.
#pragma once
#include "common.cuh"

namespace moqe {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;

// A flag in global memory that one CTA raises and another polls.  The release orders every write that happens
// before it -- the raising thread's own and, through a CTA barrier, those of the threads that arrived there before it
// -- ahead of the flag; a thread that reads the flag with the acquire load sees them all afterwards.
__device__ __forceinline__ void st_release_gpu(unsigned* p, unsigned v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// try_wait with a suspend-time hint parks the thread in hardware until the phase completes or the hint (1 ms)
// has passed, so a waiting warp does not compete for issue slots; without the hint the wait returns after a short
// system-defined time and a waiting warp spins, which costs the working warps of the same scheduler their slots.
constexpr uint32_t TRY_WAIT_HINT_NS = 1000000u;
// (kernels whose waits are short and on the critical path use the plain form: waking up from the hinted sleep is
// slower than coming round a short spin)
__device__ __forceinline__ bool mbar_try_short(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(TRY_WAIT_HINT_NS) : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false if the CTA is aborting (someone's wait ran out).  A failed try has already slept
// for up to the hint, so the clock and the abort flag are consulted after every few of them.
__device__ __forceinline__ bool mbar_wait_limit(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                                unsigned long long limit_ns) {
    if (mbar_try(bar, parity)) return true;
    unsigned long long t0 = 0;
    for (unsigned it = 1;; ++it) {
        if (mbar_try(bar, parity)) return true;
        if ((it & 3u) == 0) {
            if (*abort_flag) return false;
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) {
                *abort_flag = 1;
                latch_status(status, (int)MOQE_ERR_TIMEOUT);
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
    return mbar_wait_limit(bar, parity, abort_flag, status, WAIT_LIMIT_NS);
}

// the same bounded wait on the plain try_wait: the clock is consulted every 256 failed tries
__device__ __forceinline__ bool mbar_wait_short(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
    if (mbar_try_short(bar, parity)) return true;
    unsigned long long t0 = 0;
    for (unsigned it = 1;; ++it) {
        if (mbar_try_short(bar, parity)) return true;
        if ((it & 255u) == 0) {
            if (*abort_flag) return false;
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > WAIT_LIMIT_NS) {
                *abort_flag = 1;
                latch_status(status, (int)MOQE_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// the same copy for data that is read once: its lines are the first to leave L2, so what every CTA keeps re-reading
// (token rows, tables) stays there
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_load_once(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}
// 16-byte asynchronous global->shared copy; src_bytes (0..16) are read, the rest of the 16 is zero-filled
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// arrive on the mbarrier once all of this thread's earlier cp.async copies have landed (the arrival must be
// part of the barrier's expected count)
__device__ __forceinline__ void cp_async_arrive_noinc(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

struct Ring {
    int stage = 0;
    uint32_t phase = 0;
    __device__ __forceinline__ void advance(int n) { if (++stage == n) { stage = 0; phase ^= 1u; } }
};

}  // namespace moqe
