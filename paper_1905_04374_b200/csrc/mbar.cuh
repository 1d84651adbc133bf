// mbarrier helpers shared by the kernels that hand shared-memory tiles from one role to another
// (bulk copies -> compute threads, producers -> tensor core, tensor core -> flush warps).
// Every wait is bounded: after `limit` suspended waits it raises the caller's error flag and
// returns false, so that a kernel can drain its copies, free what it holds and leave with a status
// instead of hanging.
#pragma once

namespace gar {

// Suspended waits before a wait gives up.  One mbarrier.try_wait on a barrier that does not
// complete returns after the hardware's own time limit, 4.0 microseconds on B200 (measured with
// gar_selftest_bounded_wait); 2^20 of them bound the time a kernel can be stuck by 4.2 seconds.
constexpr unsigned KB_SPIN_LIMIT = 1u << 20;

__device__ __forceinline__ unsigned kb_smem_u32(const void* p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }

// One wait for the phase with the given parity: the thread is suspended in the barrier unit until the
// phase completes or a hardware time limit passes, whichever comes first; true if it completed.
__device__ __forceinline__ bool kb_try_wait(unsigned bar, unsigned parity) {
    unsigned done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
// Non-suspending test of the same.
__device__ __forceinline__ bool kb_test(unsigned bar, unsigned parity) {
    unsigned done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
// Bounded wait for the phase with the given parity; a waiting warp sleeps in the barrier unit and
// leaves the issue slots to the computing ones.  False: the wait gave up (error flag raised) or,
// unless `ignore_flag`, somebody else raised the flag.
__device__ __forceinline__ bool kb_wait(unsigned bar, unsigned parity, volatile int* error, bool ignore_flag = false,
                                        unsigned limit = KB_SPIN_LIMIT) {
    for (unsigned spin = 0; spin < limit; ++spin) {
        if (kb_try_wait(bar, parity)) return true;
        if (!ignore_flag && *error) return false;
    }
    *error = 1;
    return false;
}
// The same with the answer agreed over the warp, and `polls` quick tests first: a hand-off that is
// about to happen is seen soonest that way, which matters when a kernel is a few dozen tiles long.
__device__ __forceinline__ bool kb_wait_warp(unsigned bar, unsigned parity, volatile int* error, unsigned polls = 64,
                                             unsigned limit = KB_SPIN_LIMIT) {
    bool ok = false;
    for (unsigned spin = 0; spin < polls; ++spin) {
        if (kb_test(bar, parity)) { ok = true; break; }
    }
    if (!ok) ok = kb_wait(bar, parity, error, false, limit);
    return __all_sync(0xffffffffu, ok);
}
__device__ __forceinline__ void kb_init(unsigned long long* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(kb_smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void kb_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void kb_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(kb_smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void kb_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// bytes from global memory to this CTA's shared memory (both 16-byte aligned, a multiple of 16), counted in on `bar`
__device__ __forceinline__ void kb_bulk_load(unsigned dst, const void* src, unsigned bytes, unsigned bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

}  // namespace gar
