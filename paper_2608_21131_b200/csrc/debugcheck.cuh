// Index range checks of the -DHANN_DEBUG build (the stand-in for a memory checker: nothing here ever traps).
//
// HANN_CHECK_INDEX(idx, limit) evaluates to true when 0 <= idx < limit.  In a debug build a failing check records the
// source line in the context's error word (the one a kernel raises when it gives up a bounded wait: mapped host memory,
// read and cleared by the synchronisation that ends every host-pointer call and hann_sync, which then return HANN_ECUDA
// naming the line) and evaluates to false, so that the caller SKIPS the access; in a release build it is the constant
// true and costs nothing.  The word's address reaches the kernels through a device-global pointer (one copy per
// translation unit, bound by hann_ctx_create through HANN_DEBUG_DEFINE_BIND's function; debug builds only), which keeps
// every kernel signature as it is.  The most recently created context owns the word.
#pragma once

#ifdef HANN_DEBUG
#include <cuda_runtime.h>
static __device__ int* g_hann_debug_word = nullptr;
// defines `int NAME(int* word)`, which points this translation unit's copy at the context's error word
#define HANN_DEBUG_DEFINE_BIND(NAME) \
    int NAME(int* word) { return cudaMemcpyToSymbol(g_hann_debug_word, &word, sizeof(word)) == cudaSuccess ? 0 : -1; }
__device__ __forceinline__ bool hann_debug_fail(int line) {
    int* w = g_hann_debug_word;
    if (w) {
        *(volatile int*)w = 0x10000 | line;   // bit 16 marks a range check (a plain 1 is a bounded wait that ran out)
        __threadfence_system();
    }
    return false;
}
#define HANN_CHECK_INDEX(idx, limit) \
    (((long long)(idx) >= 0 && (long long)(idx) < (long long)(limit)) ? true : hann_debug_fail(__LINE__))
#else
#define HANN_CHECK_INDEX(idx, limit) true
#define HANN_DEBUG_DEFINE_BIND(NAME) \
    int NAME(int*) { return 0; }
#endif
