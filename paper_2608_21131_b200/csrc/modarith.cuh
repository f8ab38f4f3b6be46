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
