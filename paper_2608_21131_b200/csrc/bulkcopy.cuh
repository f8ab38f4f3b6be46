// Bulk asynchronous global -> shared copies with mbarrier completion (the asynchronous copy path of sm_90 and later),
// as used by the transform's pass B and by the multiply-accumulate.  Every copy is private to one CTA: it lands in the
// issuing CTA's own shared memory.  Every wait is bounded in wall-clock time.
#pragma once
#include <cstdint>

namespace {

constexpr unsigned long long kWaitLimitNs = 1000000000ULL;

__device__ __forceinline__ unsigned smem_addr(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(unsigned dst, const void* src, unsigned bytes, unsigned bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src),
                 "r"(bytes), "r"(bar)
                 : "memory");
}
// one box of a 2-D tiled tensor map (x = innermost coordinate in elements: x times the element size must be a multiple of
// 16 bytes; y = row) into shared memory (128-byte aligned destination)
__device__ __forceinline__ void tensor_load_2d(unsigned dst, const void* tmap, int x, int y, unsigned bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
                 "l"(tmap), "r"(x), "r"(y), "r"(bar)
                 : "memory");
}
// the context's error word lives in mapped host memory: a plain store, made visible to the host before the kernel ends
__device__ __forceinline__ void raise_flag(int* kflag) {
    *(volatile int*)kflag = 1;
    __threadfence_system();
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// bounded: gives up (false) limit_ns (default: one second) after the first unsuccessful probe
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, unsigned long long limit_ns = kWaitLimitNs) {
    unsigned long long t0 = 0;
    for (unsigned it = 0;; it++) {
        unsigned ok;
        asm volatile(
            "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
        if ((it & 63) == 0) {
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) return false;
        }
    }
}


}  // namespace
