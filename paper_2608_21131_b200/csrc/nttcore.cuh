// Arithmetic policies and register rounds shared by the transform kernels (ntt.cu) and the fused encoder
// (encode.cu).  See ntt.cu for the description of the three arithmetic classes and their range discipline.
#pragma once
#include "modarith.cuh"

#ifndef HANN_F64_MINBLOCKS
#define HANN_F64_MINBLOCKS 2
#endif
#ifndef HANN_NTT_MINBLOCKS
#define HANN_NTT_MINBLOCKS 2
#endif

// ---- arithmetic policies ---------------------------------------------------------------------------------------

struct ArithF64 {
    typedef double T;
    typedef double2 TW;
    double q, qinv, half;
    long long qi;
    static constexpr int kMinBlocks = HANN_F64_MINBLOCKS;
    static constexpr double kRound = 6755399441055744.0;  // 1.5 * 2^52: fl(v + kRound) - kRound = rint(v) for |v| < 2^51
    static constexpr double kTwo52 = 4503599627370496.0;
    TW ninv;
    __device__ __forceinline__ ArithF64(const LimbConst* lc)
        : q((double)lc->q), qinv(1.0 / (double)lc->q), half((double)lc->half), qi((long long)lc->q), ninv(make_double2(lc->ninv_bal, lc->ninv_q)) {}
    // x - round(x/q) q; the quotient (at most 8 in magnitude) is rounded by adding 1.5 * 2^52
    __device__ __forceinline__ T reduce(T x) const {
        return __fma_rn(-__dsub_rn(__fma_rn(x, qinv, kRound), kRound), q, x);
    }
    __device__ __forceinline__ T mulmod(T y, TW w) const {
        const double h = __dmul_rn(y, w.x);
        const double l = __fma_rn(y, w.x, -h);
        const double c = rint(__dmul_rn(y, w.y));
        return __dadd_rn(__fma_rn(-c, q, h), l);
    }
    // the same product for |y| < 4q: |y * w/q| < 2^51, so the quotient can be rounded on the FP64 pipe by adding
    // 1.5 * 2^52 inside the multiply-add (one rounding less than above, and no trip through the conversion unit)
    __device__ __forceinline__ T mulmod_small(T y, TW w) const {
        const double h = __dmul_rn(y, w.x);
        const double l = __fma_rn(y, w.x, -h);
        const double c = __dsub_rn(__fma_rn(y, w.y, kRound), kRound);
        return __dadd_rn(__fma_rn(-c, q, h), l);
    }
    // integers below 2^52 <-> binary64 through the mantissa of 2^52 + v (one add and one logic operation)
    __device__ __forceinline__ T from_canonical(u64 v) const {
        return __dsub_rn(__longlong_as_double((long long)(v | 0x4330000000000000ULL)), kTwo52);
    }
    __device__ __forceinline__ T from_mid(u64 v) const { return __longlong_as_double((long long)v); }
    __device__ __forceinline__ u64 to_mid(T x) const { return (u64)__double_as_longlong(reduce(x)); }
    // exchange between the two rounds of a forward pass that started from reduced values: no reduction (eight stages
    // stay below 8q, see ntt.cu)
    __device__ __forceinline__ u64 to_exch(T x) const { return (u64)__double_as_longlong(x); }
    __device__ __forceinline__ u64 to_canonical(T x) const {
        x = reduce(x);
        // balanced integer -> two's complement through the mantissa of 1.5 * 2^52 + x; the sign fix runs on the integer
        // pipe, which is idle beside the FP64 pipe
        const long long r = __double_as_longlong(__dadd_rn(x, kRound)) - 0x4338000000000000LL;
        return (u64)(r + ((r >> 63) & qi));
    }
    __device__ __forceinline__ void fwd(T& X, T& Y, TW w) const {
        const T t = mulmod(Y, w);
        Y = __dsub_rn(X, t);
        X = __dadd_rn(X, t);
    }
    __device__ __forceinline__ void fwd_small(T& X, T& Y, TW w) const {  // |Y| < 4q
        const T t = mulmod_small(Y, w);
        Y = __dsub_rn(X, t);
        X = __dadd_rn(X, t);
    }
    __device__ __forceinline__ void inv(T& X, T& Y, TW w) const {
        const T d = __dsub_rn(X, Y);
        X = __dadd_rn(X, Y);
        Y = mulmod(d, w);
    }
    // inverse transforms start from balanced values so that four doubling stages stay below 2^53
    __device__ __forceinline__ T inv_input(u64 v) const {
        const double x = from_canonical(v);
        return x > half ? x - q : x;
    }
    __device__ __forceinline__ u64 scaled_output(T x, TW ninv_pair) const { return to_canonical(mulmod(reduce(x), ninv_pair)); }
};

template <bool SMALLQ>
struct ArithInt {
    typedef u64 T;
    typedef ulonglong2 TW;
    u64 q, q2;
    static constexpr int kMinBlocks = HANN_NTT_MINBLOCKS;
    TW ninv;
    __device__ __forceinline__ ArithInt(const LimbConst* lc) : q(lc->q), q2(2 * lc->q), ninv(make_ulonglong2(lc->ninv, lc->ninv_s)) {}
    __device__ __forceinline__ T from_canonical(u64 v) const { return v; }
    __device__ __forceinline__ T from_mid(u64 v) const { return v; }
    __device__ __forceinline__ u64 to_mid(T x) const { return x; }
    __device__ __forceinline__ u64 to_exch(T x) const { return x; }
    __device__ __forceinline__ u64 to_canonical(T v) const {  // forward results: [0, 33q) or [0, 4q)
        if (SMALLQ) {
            v = csub(v, 32 * q);
            v = csub(v, 16 * q);
            v = csub(v, 8 * q);
            v = csub(v, 4 * q);
        }
        v = csub(v, q2);
        return csub(v, q);
    }
    __device__ __forceinline__ void fwd(T& X, T& Y, TW w) const {
        u64 x = X;
        if (!SMALLQ) x = csub(x, q2);
        const u64 t = shoup_mul(Y, w.x, w.y, q);
        X = x + t;
        Y = x - t + q2;
    }
    __device__ __forceinline__ void fwd_small(T& X, T& Y, TW w) const { fwd(X, Y, w); }
    __device__ __forceinline__ void inv(T& X, T& Y, TW w) const {  // [0, 2q) in and out
        const u64 x = X, y = Y;
        X = csub(x + y, q2);
        Y = shoup_mul(x - y + q2, w.x, w.y, q);
    }
    __device__ __forceinline__ T inv_input(u64 v) const { return v; }
    __device__ __forceinline__ u64 scaled_output(T x, TW ninv_pair) const { return csub(shoup_mul(x, ninv_pair.x, ninv_pair.y, q), q); }
};

// ---- register rounds -----------------------------------------------------------------------------------------

// NS: the first NS stages of the round see inputs below 4q (binary64 arithmetic then rounds its quotients on the FP64
// pipe instead of the conversion unit); 0 is always correct
template <int R, class AR, int NS = 0>
__device__ __forceinline__ void fwd_round(const AR& ar, typename AR::T (&x)[1 << R], const typename AR::TW* __restrict__ tw,
                                          unsigned base) {
#pragma unroll
    for (int s = 0; s < R; s++) {
        const int span = 1 << (R - 1 - s);
#pragma unroll
        for (int il = 0; il < (1 << s); il++) {
            const typename AR::TW w = tw[(base << s) + il];
#pragma unroll
            for (int jj = 0; jj < span; jj++) {
                const int e = il * 2 * span + jj;
                if (s < NS) ar.fwd_small(x[e], x[e + span], w);
                else ar.fwd(x[e], x[e + span], w);
            }
        }
    }
}

// the same round with the twiddle of (stage s, group il) supplied by a functor (shared-memory caches with their own
// layout)
template <int R, class AR, int NS = 0, class TWF>
__device__ __forceinline__ void fwd_round_f(const AR& ar, typename AR::T (&x)[1 << R], const TWF& twf) {
#pragma unroll
    for (int s = 0; s < R; s++) {
        const int span = 1 << (R - 1 - s);
#pragma unroll
        for (int il = 0; il < (1 << s); il++) {
            const typename AR::TW w = twf(s, il);
#pragma unroll
            for (int jj = 0; jj < span; jj++) {
                const int e = il * 2 * span + jj;
                if (s < NS) ar.fwd_small(x[e], x[e + span], w);
                else ar.fwd(x[e], x[e + span], w);
            }
        }
    }
}

// (flat butterfly index t = il * span + jj: with the nested (il, jj) loops of the forward round the compiler left x[] in
// local memory)
template <int R, class AR>
__device__ __forceinline__ void inv_round(const AR& ar, typename AR::T (&x)[1 << R], const typename AR::TW* __restrict__ tw,
                                          unsigned base) {
#pragma unroll
    for (int s = 0; s < R; s++) {
#pragma unroll
        for (int t = 0; t < (1 << (R - 1)); t++) {
            const int il = t >> s, jj = t & ((1 << s) - 1);
            const int e = (il << (s + 1)) + jj;
            ar.inv(x[e], x[e + (1 << s)], tw[(base << (R - 1 - s)) + il]);
        }
    }
}

// the inverse round with the twiddle of (stage s, group il) supplied by a functor
template <int R, class AR, class TWF>
__device__ __forceinline__ void inv_round_f(const AR& ar, typename AR::T (&x)[1 << R], const TWF& twf) {
#pragma unroll
    for (int s = 0; s < R; s++) {
#pragma unroll
        for (int t = 0; t < (1 << (R - 1)); t++) {
            const int il = t >> s, jj = t & ((1 << s) - 1);
            const int e = (il << (s + 1)) + jj;
            ar.inv(x[e], x[e + (1 << s)], twf(s, il));
        }
    }
}

template <int R2>
__device__ __forceinline__ int pad(int pos) { return R2 == 0 ? pos : pos + (pos >> R2); }

