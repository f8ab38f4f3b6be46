// Host-side mathematics of the library: parameter validation, roots of unity, table values, and the client's
// CRT reconstruction and slot decoding.  None of this is on the per-query device path.
#include <cmath>
#include <cstring>
#include <vector>

#include "internal.h"

namespace hm {

typedef unsigned __int128 u128;

u64 mulmod(u64 a, u64 b, u64 q) { return (u64)(((u128)a * b) % q); }

u64 powmod(u64 a, u64 e, u64 q) {
    u64 r = 1 % q;
    a %= q;
    for (; e; e >>= 1) {
        if (e & 1) r = mulmod(r, a, q);
        a = mulmod(a, a, q);
    }
    return r;
}

u64 invmod(u64 a, u64 q) { return powmod(a, q - 2, q); }

u64 shoup(u64 w, u64 q) { return (u64)((((u128)w) << 64) / q); }

int bitrev(int x, int bits) {
    int r = 0;
    for (int i = 0; i < bits; i++) {
        r = (r << 1) | (x & 1);
        x >>= 1;
    }
    return r;
}

// Miller-Rabin with the first twelve primes as bases: deterministic below 3.3e24
bool is_prime(u64 n) {
    const u64 bases[12] = {2, 3, 5, 7, 11, 13, 17, 19, 23, 29, 31, 37};
    if (n < 2) return false;
    for (u64 b : bases) {
        if (n == b) return true;
        if (n % b == 0) return false;
    }
    u64 d = n - 1;
    int r = 0;
    while (!(d & 1)) {
        d >>= 1;
        r++;
    }
    for (u64 b : bases) {
        u64 x = powmod(b, d, n);
        if (x == 1 || x == n - 1) continue;
        bool witness = true;
        for (int i = 1; i < r && witness; i++) {
            x = mulmod(x, x, n);
            if (x == n - 1) witness = false;
        }
        if (witness) return false;
    }
    return true;
}

// a primitive 2N-th root of unity: x^((q-1)/2N) for the first x that is a quadratic non-residue
u64 find_psi(u64 q, int N) {
    const u64 e = (q - 1) / (2 * (u64)N);
    for (u64 x = 2; x < q; x++) {
        u64 c = powmod(x, e, q);
        if (powmod(c, (u64)N, q) == q - 1) return c;
    }
    return 0;
}

// ---- unit roots, correctly rounded -------------------------------------------------------------------------
// sin and cos of an angle in [0, pi/4] by their Taylor series in binary128 (relative error ~2^-110), so that the
// single rounding to binary64 gives the correctly rounded value except with negligible probability.

static __float128 quad_pi() {
    // pi as the exact sum of three doubles (the first 159 bits of pi), added in binary128
    return (__float128)3.141592653589793116 + (__float128)1.2246467991473532072e-16 + (__float128)(-2.9947698097183396659e-33);
}

static void sincos_small(__float128 x, __float128* s, __float128* c) {
    __float128 x2 = x * x, ts = x, tc = 1, ss = x, cs = 1;
    for (int k = 1; k <= 24; k++) {
        tc = -tc * x2 / (__float128)((2 * k - 1) * (2 * k));
        ts = -ts * x2 / (__float128)((2 * k) * (2 * k + 1));
        cs += tc;
        ss += ts;
    }
    *s = ss;
    *c = cs;
}

// (c, s) = (cos, sin)(2 pi t / den).  The angle is reduced to the first octant with integer arithmetic, so the
// exact values 0 and +-1 come out exact and the eight-fold symmetry holds bit for bit.
void unit_root(long t, long den, double* c, double* s) {
    t %= den;
    if (t < 0) t += den;
    const long e8 = 8 * t, oct = e8 / den, rem = e8 % den;
    __float128 qs, qc;
    double dc, ds;
    if ((oct & 1) == 0) {
        sincos_small(quad_pi() / 4 * (__float128)rem / (__float128)den, &qs, &qc);
        dc = (double)qc;
        ds = (double)qs;
    } else {
        sincos_small(quad_pi() / 4 * (__float128)(den - rem) / (__float128)den, &qs, &qc);
        dc = (double)qs;
        ds = (double)qc;
    }
    switch (oct / 2) {
        case 0: *c = dc; *s = ds; break;
        case 1: *c = -ds; *s = dc; break;
        case 2: *c = -dc; *s = -ds; break;
        default: *c = ds; *s = -dc; break;
    }
    *c += 0.0;  // turn -0.0 into +0.0
    *s += 0.0;
}

// ---- CRT -------------------------------------------------------------------------------------------------
// Garner's mixed-radix digits, then Horner evaluation in multi-word integers, centring against Q/2 and
// conversion to long double.

namespace {
struct Big {
    u64 w[HANN_MAXL1 + 1];
    int n;
};
void big_zero(Big& b, int n) {
    b.n = n;
    memset(b.w, 0, sizeof(b.w));
}
void big_mul_add(Big& b, u64 m, u64 a) {  // b = b*m + a
    u128 carry = a;
    for (int i = 0; i < b.n; i++) {
        u128 t = (u128)b.w[i] * m + carry;
        b.w[i] = (u64)t;
        carry = t >> 64;
    }
}
int big_cmp(const Big& a, const Big& b) {
    for (int i = a.n - 1; i >= 0; i--)
        if (a.w[i] != b.w[i]) return a.w[i] < b.w[i] ? -1 : 1;
    return 0;
}
void big_sub(Big& a, const Big& b) {  // a -= b (a >= b)
    u64 borrow = 0;
    for (int i = 0; i < a.n; i++) {
        u64 bi = b.w[i], ai = a.w[i];
        u64 d = ai - bi - borrow;
        borrow = (ai < bi || (ai == bi && borrow)) ? 1 : 0;
        a.w[i] = d;
    }
}
void big_half(Big& a) {
    for (int i = 0; i < a.n; i++) a.w[i] = (a.w[i] >> 1) | (i + 1 < a.n ? a.w[i + 1] << 63 : 0);
}
long double big_to_ld(const Big& a) {
    long double v = 0;
    for (int i = a.n - 1; i >= 0; i--) v = v * 18446744073709551616.0L + (long double)a.w[i];
    return v;
}
}  // namespace

void crt_to_real(const u64* res, int L, int N, const u64* q, long double* out) {
    // inv[i][k] = q_k^{-1} mod q_i for k < i
    std::vector<u64> inv((size_t)L * L, 0);
    for (int i = 0; i < L; i++)
        for (int k = 0; k < i; k++) inv[(size_t)i * L + k] = invmod(q[k] % q[i], q[i]);
    Big Q, halfQ;
    big_zero(Q, L + 1);
    Q.w[0] = 1;
    for (int i = 0; i < L; i++) big_mul_add(Q, q[i], 0);
    halfQ = Q;
    big_half(halfQ);
    for (int x = 0; x < N; x++) {
        u64 v[HANN_MAXL1];
        for (int i = 0; i < L; i++) {
            // v_i = (((r_i - v_0) / q_0 - v_1) / q_1 - ...) mod q_i
            u64 t = res[(size_t)i * N + x] % q[i];
            for (int k = 0; k < i; k++) {
                u64 vk = v[k] % q[i];
                t = t >= vk ? t - vk : t + q[i] - vk;
                t = mulmod(t, inv[(size_t)i * L + k], q[i]);
            }
            v[i] = t;
        }
        Big X;
        big_zero(X, L + 1);
        for (int i = L - 1; i >= 0; i--) big_mul_add(X, q[i], v[i]);  // X = v_0 + q_0 (v_1 + q_1 (v_2 + ...))
        if (big_cmp(X, halfQ) > 0) {
            Big D = Q;
            big_sub(D, X);
            out[x] = -big_to_ld(D);
        } else {
            out[x] = big_to_ld(X);
        }
    }
}

// plain radix-2 complex FFT (decode only; its result is compared within a tolerance, never bit for bit)
void fft_inplace(double* re, double* im, int n, int logn, int sign) {
    for (int i = 0; i < n; i++) {
        int j = bitrev(i, logn);
        if (i < j) {
            std::swap(re[i], re[j]);
            std::swap(im[i], im[j]);
        }
    }
    for (int len = 2; len <= n; len <<= 1) {
        std::vector<double> wr(len / 2), wi(len / 2);
        for (int t = 0; t < len / 2; t++) {
            const double ang = 2.0 * M_PI * t / len;
            wr[t] = std::cos(ang);
            wi[t] = sign * std::sin(ang);
        }
        for (int k0 = 0; k0 < n; k0 += len)
            for (int t = 0; t < len / 2; t++) {
                int a = k0 + t, b = a + len / 2;
                double yr = re[b] * wr[t] - im[b] * wi[t], yi = re[b] * wi[t] + im[b] * wr[t];
                re[b] = re[a] - yr;
                im[b] = im[a] - yi;
                re[a] += yr;
                im[a] += yi;
            }
    }
}

static u64 mix64(u64 x) {
    x ^= x >> 32;
    x *= 0x9E3779B97F4A7C15ULL;
    x ^= x >> 29;
    x *= 0xBB67AE8584CAA73BULL;
    x ^= x >> 32;
    return x;
}

u64 hash64(u64 seed, u64 stream, u64 ctr) {
    const u64 a = mix64(seed + 0x9E3779B97F4A7C15ULL);
    const u64 b = mix64(a ^ (stream * 0xBB67AE8584CAA73BULL));
    return mix64(b + ctr * 0x9E3779B97F4A7C15ULL);
}

void seeded_ternary(u64 seed, u64 stream, int N, int8_t* s) {
    // the top 32 bits times 3, shifted down: uniform on {0, 1, 2} up to 2^-32
    for (int x = 0; x < N; x++) s[x] = (int8_t)((int)(((hash64(seed, stream, (u64)x) >> 32) * 3) >> 32) - 1);
}

void seeded_gaussian(u64 seed, u64 stream, u64 ctr0, long count, double sigma, int8_t* e) {
    const double two_pi = 6.283185307179586476925286766559;
    for (long i = 0; i < count; i++) {
        // u1 in (0, 1], u2 in [0, 1): 53-bit uniforms from two sub-streams
        const double u1 = (double)((hash64(seed, stream, ctr0 + (u64)i) >> 11) + 1) * 0x1p-53;
        const double u2 = (double)(hash64(seed, stream + 1, ctr0 + (u64)i) >> 11) * 0x1p-53;
        double v = std::nearbyint(sigma * std::sqrt(-2.0 * std::log(u1)) * std::cos(two_pi * u2));
        if (v > 127) v = 127;
        if (v < -127) v = -127;
        e[i] = (int8_t)v;
    }
}

}  // namespace hm
