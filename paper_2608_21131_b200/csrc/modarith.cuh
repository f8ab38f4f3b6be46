// Device-side modular arithmetic on 64-bit residues (moduli below 2^62).
//
// Three reductions are used:
//   * Shoup multiplication by a known constant w with precomputed w' = floor(w * 2^64 / q):
//     a*w - hi64(a*w')*q lies in [0, 2q) for every 64-bit a (lazy range, no correction);
//   * single-word Barrett with mu = floor(2^64 / q): v - hi64(v*mu)*q lies in [0, 2q);
//   * a 128-bit value hi*2^64 + lo is folded as (hi mod q)*(2^64 mod q) + (lo mod q), the middle product
//     again by Shoup, giving a residue in [0, q) after two conditional subtractions.
#pragma once
#include <cstdint>

typedef uint64_t u64;
typedef int64_t i64;

struct LimbConst {
    u64 q;       // modulus
    u64 mu;      // floor(2^64 / q)
    u64 c64;     // 2^64 mod q
    u64 c64s;    // floor(c64 * 2^64 / q)
    u64 ninv;    // N^{-1} mod q
    u64 ninv_s;  // Shoup companion of ninv
    u64 pinv;    // p^{-1} mod q          (ciphertext primes only)
    u64 pinv_s;
    u64 pmod;    // p mod q               (ciphertext primes only)
    u64 half;    // floor(q / 2): residues above it lift to negative integers
    double ninv_bal;  // N^{-1} mod q as a balanced integer (binary64 transform path)
    double ninv_q;    // fl(ninv_bal / q)
};

#define HANN_MAXL1 16  // up to 15 ciphertext primes + the special prime (limb numbers travel in 4-bit fields)

struct LimbTable {
    LimbConst c[HANN_MAXL1];
};

// which modulus each polynomial of a batch uses: limb[p % period]
struct LimbMap {
    int period;
    signed char limb[32];
};

#ifdef __CUDACC__  // device functions: only for translation units compiled by nvcc

__device__ __forceinline__ u64 shoup_mul(u64 a, u64 w, u64 ws, u64 q) {
    u64 t = __umul64hi(a, ws);
    return a * w - t * q;  // [0, 2q)
}

__device__ __forceinline__ u64 csub(u64 a, u64 q) { return a >= q ? a - q : a; }

// v mod q for any 64-bit v
__device__ __forceinline__ u64 barrett64(u64 v, const LimbConst& c) {
    u64 r = v - __umul64hi(v, c.mu) * c.q;  // [0, 2q)
    return csub(r, c.q);
}

// (hi * 2^64 + lo) mod q
__device__ __forceinline__ u64 reduce128(u64 hi, u64 lo, const LimbConst& c) {
    u64 h = hi - __umul64hi(hi, c.mu) * c.q;      // [0, 2q), congruent to hi
    u64 a = shoup_mul(h, c.c64, c.c64s, c.q);     // [0, 2q), congruent to hi * 2^64
    u64 l = lo - __umul64hi(lo, c.mu) * c.q;      // [0, 2q)
    u64 r = a + l;                                // [0, 4q)
    r = csub(r, 2 * c.q);
    return csub(r, c.q);
}

__device__ __forceinline__ u64 mulmod(u64 a, u64 b, const LimbConst& c) {
    return reduce128(__umul64hi(a, b), a * b, c);
}

__device__ __forceinline__ u64 addmod(u64 a, u64 b, u64 q) { return csub(a + b, q); }
__device__ __forceinline__ u64 submod(u64 a, u64 b, u64 q) { return a >= b ? a - b : a + q - b; }

// signed integer -> residue in [0, q)
__device__ __forceinline__ u64 reduce_signed(i64 v, const LimbConst& c) {
    u64 mag = v < 0 ? (u64)0 - (u64)v : (u64)v;
    u64 r = barrett64(mag, c);
    return (v < 0 && r) ? c.q - r : r;
}

// 128-bit accumulator: (hi, lo) += a * b
__device__ __forceinline__ void mac128(u64& hi, u64& lo, u64 a, u64 b) {
    u64 pl = a * b, ph = __umul64hi(a, b);
    lo += pl;
    hi += ph + (lo < pl ? 1 : 0);
}

// ---- exact sums of products on the FP64 pipe (moduli below 2^50) --------------------------------------------------------------
// The GPU has no native 64-bit integer multiplier (a product of two residues costs three or four 32 x 32 -> 64 multiply-adds
// plus additions) but a full-rate binary64 multiply-add.  A sum of at most EIGHT products w * p, w a balanced residue
// (|w| < 2^49) and p a residue in [0, 2^50), is kept exactly in two binary64 words:
//   ah starts at 1.5 * 2^103, so every ah = fma(p, w, ah) is rounded to a multiple of 2^51 (the partial sums stay below 2^102
//      in magnitude: ah never leaves its binade);
//   what that rounding dropped, p w + (ah_old - ah_new), is an integer of magnitude at most 2^50, which a second fma yields
//      exactly; eight of them sum exactly in al (|al| <= 2^53).
// Four FP64 operations per product.  sum = (ah - 1.5 * 2^103) + al.
constexpr double kAcc2Start = 0x1.8p103;

// residue below 2^52 -> binary64 through the mantissa of 2^52 + x (one logic operation, one addition)
__device__ __forceinline__ double residue_to_f64(u64 x) {
    return __dsub_rn(__longlong_as_double((long long)(x | 0x4330000000000000ULL)), 4503599627370496.0);
}
__device__ __forceinline__ double residue_to_balanced_f64(u64 x, double q, double half) {
    const double d = residue_to_f64(x);
    return d > half ? __dsub_rn(d, q) : d;
}
__device__ __forceinline__ void acc2_fma(double& ah, double& al, double p, double w) {
    const double nh = __fma_rn(p, w, ah);
    al = __dadd_rn(al, __fma_rn(p, w, __dsub_rn(ah, nh)));
    ah = nh;
}
// the two words as integers: high word as a count of 2^51 (below 2^51 in magnitude), low word as it is; both can be added up
// over several partial sums in 64-bit integers
__device__ __forceinline__ long long acc2_high(double ah) { return __double2ll_rn(__dmul_rn(__dsub_rn(ah, kAcc2Start), 0x1p-51)); }
__device__ __forceinline__ long long acc2_low(double al) { return __double2ll_rn(al); }
// (m 2^51 + sl) mod q for the integer sums of the words of n <= 128 products: |m 2^51 + sl| < n q^2 / 2 < q 2^57 (q < 2^50),
// so adding q 2^57 makes it a non-negative 128-bit integer
__device__ __forceinline__ u64 acc2_reduce(long long m, long long sl, const LimbConst& c) {
    u64 lo = (u64)m << 51, hi = (u64)(m >> 13);
    const u64 s_lo = (u64)sl, s_hi = (u64)(sl >> 63);
    lo += s_lo;
    hi += s_hi + (lo < s_lo ? 1 : 0);
    const u64 o_lo = c.q << 57, o_hi = c.q >> 7;
    lo += o_lo;
    hi += o_hi + (lo < o_lo ? 1 : 0);
    return reduce128(hi, lo, c);
}

// swap the two low nibbles of a position (an involution inside every aligned chunk of 256 positions)
__device__ __forceinline__ int swap_nibbles(int t) { return (t & ~255) | ((t & 15) << 4) | ((t >> 4) & 15); }

// Position t of a transformed polynomial holds the value at psi^(2*brev(t)+1); the automorphism X -> X^k reads position
// brev(((2*brev(t)+1)*k mod 2N - 1) / 2).  Rings of 2^10 points and more store every chunk of 256 positions with its
// two low nibbles swapped (`tau`: the last forward round then writes, and the first inverse round reads, coalesced
// words straight from registers), so the map is conjugated by that swap.
__device__ __forceinline__ int galois_src(int t, unsigned k, int logN, int tau) {
    if (tau) t = swap_nibbles(t);
    unsigned br = __brev((unsigned)t) >> (32 - logN);
    unsigned e = ((2u * br + 1u) * k) & ((2u << logN) - 1u);
    int s = (int)(__brev((e - 1u) >> 1) >> (32 - logN));
    return tau ? swap_nibbles(s) : s;
}

#endif  // __CUDACC__
