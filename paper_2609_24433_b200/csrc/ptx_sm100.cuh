// Thin inline-PTX wrappers shared by the kernels: mbarrier, bounded waits, proxy fences.
#pragma once

#include <stdint.h>

namespace fq {

constexpr uint64_t kWaitLimitNs = 2000000000ull;   // every device-side wait gives up after 2 s

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
// One lane of a fully converged warp.  Issue work placed under `if (elect_one())` was measured
// much cheaper than under `if (lane == 0)`: the compiler then knows that a single thread runs it.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Same, but the thread may stay suspended for up to `hint_ns` before the instruction returns:
// long waits then cost far fewer issue slots (and less power) than a tight polling loop.
__device__ __forceinline__ bool mbar_try_wait_hint(uint32_t bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Non-blocking test of a phase (never suspends the thread): used to look one stage ahead, so that
// the ~100-cycle latency of a barrier test overlaps with the work issued in between.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false if the CTA is aborting or the limit expired
// (in which case the abort flag and the watchdog word are set).  The clock is read only after a
// few thousand failed tries (each try may itself suspend the thread for a while), so that the
// common short wait pays for nothing but the tries.
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                            uint32_t* watchdog, uint32_t code, uint64_t limit_ns = kWaitLimitNs) {
    uint64_t t0 = 0;
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 0xfff) == 0) {
            if (*abort_flag) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > limit_ns) {
                *abort_flag = 1;
                atomicOr(watchdog, code);
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          uint32_t* watchdog, uint32_t code, uint64_t limit_ns = kWaitLimitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, watchdog, code, limit_ns);
}
// Warp-converged wait: every lane polls the same barrier, the result is made warp-uniform.
// Roles that hand work over through barriers run their loops with the whole warp converged and
// elect a lane only for the issue itself: a lone lane looping while its warp-mates are parked at a
// CTA barrier was measured 2-3x slower per dependent wait/arrive pair.
// `peeked` is the result of an earlier mbar_test_wait on the same phase: when it was already true
// the wait costs nothing.
__device__ __forceinline__ bool mbar_wait_all(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                              uint32_t* watchdog, uint32_t code, bool peeked = false,
                                              uint64_t limit_ns = kWaitLimitNs) {
    if (__all_sync(0xffffffffu, peeked)) return true;
    const bool ok = mbar_wait(bar, parity, abort_flag, watchdog, code, limit_ns);
    return __all_sync(0xffffffffu, ok);
}
// Converged wait for roles that run far ahead of their consumer (TMA producers behind a full ring): between
// tries the warp sleeps, so that it does not take issue slots from the warps on the critical path.
__device__ __forceinline__ bool mbar_wait_all_lazy(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                   uint32_t* watchdog, uint32_t code, bool peeked = false) {
    if (__all_sync(0xffffffffu, peeked)) return true;
    bool ok = true;
    if (!mbar_try_wait(bar, parity)) {
        const uint64_t t0 = global_timer_ns();
        for (uint32_t spin = 1; !mbar_try_wait(bar, parity); ++spin) {
            __nanosleep(100);
            if ((spin & 0x3ff) == 0) {
                if (*abort_flag) { ok = false; break; }
                if (global_timer_ns() - t0 > kWaitLimitNs) {
                    *abort_flag = 1;
                    atomicOr(watchdog, code);
                    ok = false;
                    break;
                }
            }
        }
    }
    return __all_sync(0xffffffffu, ok);
}
// Wait for latency-tolerant roles (epilogue): lane 0 polls with a short sleep between tries so that
// an idle warp does not compete for issue slots with the warps feeding the tensor core.
__device__ __forceinline__ bool mbar_wait_warp_relaxed(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                       uint32_t* watchdog, uint32_t code) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) {
        const uint64_t t0 = global_timer_ns();
        for (uint32_t spin = 1; !mbar_try_wait(bar, parity); ++spin) {
            __nanosleep(200);
            if ((spin & 0x3f) == 0) {
                if (*abort_flag) { ok = 0; break; }
                if (global_timer_ns() - t0 > kWaitLimitNs) {
                    *abort_flag = 1;
                    atomicOr(watchdog, code);
                    ok = 0;
                    break;
                }
            }
        }
    }
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
// Warp-collective wait: lane 0 waits, the result is broadcast (one poller per warp instead of 32).
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                               uint32_t* watchdog, uint32_t code) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, abort_flag, watchdog, code) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// Programmatic dependent launch.  A kernel launched with the programmatic-serialization attribute
// may start while the kernel before it in the stream is still running; griddep_wait() returns once
// that kernel has completed and its writes are visible, so everything that touches global memory
// comes after it and only on-chip setup (barriers, TMEM, descriptor prefetch) runs ahead.
// griddep_launch_dependents() lets the NEXT kernel in the stream begin its own setup early.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void fence_mbarrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// 1-D bulk copy global -> shared (16-byte aligned addresses, size a multiple of 16 bytes).
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

}  // namespace fq
