/*
 * hann_oracle.c -- plain, slow CPU RNS-CKKS reference for the encrypted scoring path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the checker the CUDA library is compared with.
 * It shares no code, header, table generator or constant with the CUDA path, and nothing
 * on the product path may call it.  Everything here is written for being checked by eye:
 * one modulus at a time, `unsigned __int128` products reduced with `%`, textbook
 * transforms, no blocking, no fusion, no lazy reduction.
 *
 * What it computes (paper sections in brackets):
 *   - a block of n = N/2 candidate rows is held as R "diagonals" of one slot vector each
 *     [Sec. 2, storage formula paragraph], the diagonals shifted in plaintext by the
 *     giant-step amount [Sec. 3.1, Detail: plaintext pre-rotation];
 *   - scores = diagonal matrix-vector product with baby-step/giant-step rotations
 *     [Sec. 3.1 "How", Detail], evaluated on an encrypted query and returned encrypted,
 *     the client decrypting and ranking [Sec. 2, The round trip];
 *   - the candidates are plaintext here (the measured prototype of Sec. 2 also held the
 *     database in plaintext), so the product is ciphertext x plaintext.
 * The paper names its CKKS primitives only through the libraries it used; the scheme
 * conventions below (slot order, canonical encode, symmetric encryption, hybrid key
 * switching with one special prime, centred lifts) are this build's stated readings.
 *
 * Layout of every polynomial crossing this API ("canonical"): coefficient domain, natural
 * order, residues in [0, q_i), uint64, index order [poly][limb][coeff].
 *
 * Pins (tests/test_oracle_pins.py): primes by independent primality test; NTT round trip and
 * NTT product == schoolbook product (python integers) for N <= 256; encode == exact cosine
 * sum evaluated in multi-precision; automorphism == slot roll; decrypt(encrypt(m)) - m == e;
 * key-switch error within the analytic noise bound and ModDown(p*x) == x; rotate via
 * "decompose then permute" == "permute then decompose"; BSGS/Horner == plain matvec;
 * decrypted scores == float64 dot products within the stated tolerance; the lazy giant steps: inner product + ModDown
 * == orc_keyswitch bit for bit, the result's decryption minus the exactly rotated decryptions of the terms inside the
 * analytic bound for G-1 key products and ONE rounding.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#include <quadmath.h>

typedef uint64_t u64;
typedef int64_t i64;
typedef unsigned __int128 u128;

#define ORC_MAX_LIMBS 17 /* up to 16 ciphertext primes + the special prime */

typedef struct {
    int logN, N, n;      /* ring degree N = 2^logN, n = N/2 slots */
    int L;               /* number of ciphertext primes q_0..q_{L-1}; limb index L is the special prime p */
    u64 mod[ORC_MAX_LIMBS];
    u64 psi[ORC_MAX_LIMBS];     /* primitive 2N-th root of unity mod each modulus */
    u64 psi_inv[ORC_MAX_LIMBS];
    u64 n_inv[ORC_MAX_LIMBS];   /* N^{-1} */
    int log_scale;       /* Delta = 2^log_scale */
    int R, B, G;         /* padded dimension, baby steps, giant steps (R = B*G) */
    int *g5;             /* g5[j] = 5^j mod 2N, j < n                    */
    int *uidx;           /* uidx[j] = (g5[j]-1)/4, a permutation of [0,n) */
    double *T_re, *T_im; /* T[t] = exp(-2 pi i t / n), t < n/2, correctly rounded */
    double *U_re, *U_im; /* U[k] = exp(-i pi k / N),  k < n,   correctly rounded */
} orc_ctx;

/* ------------------------------------------------------------------ modular arithmetic */

static u64 mulmod(u64 a, u64 b, u64 q) { return (u64)(((u128)a * b) % q); }
static u64 addmod(u64 a, u64 b, u64 q) { u64 c = a + b; return c >= q ? c - q : c; }
static u64 submod(u64 a, u64 b, u64 q) { return a >= b ? a - b : a + q - b; }
static u64 powmod(u64 a, u64 e, u64 q) {
    u64 r = 1 % q;
    a %= q;
    while (e) { if (e & 1) r = mulmod(r, a, q); a = mulmod(a, a, q); e >>= 1; }
    return r;
}
static u64 invmod(u64 a, u64 q) { return powmod(a, q - 2, q); } /* q prime */

/* signed integer -> residue in [0,q) */
static u64 reduce_signed(i64 v, u64 q) {
    if (v >= 0) return (u64)v % q;
    u64 r = ((u64)(-(v + 1)) + 1) % q; /* |v| mod q without overflow at INT64_MIN */
    return r ? q - r : 0;
}

/* centred lift of a residue x in [0,q) to the symmetric interval (-q/2, q/2] (q odd: +-(q-1)/2) */
static i64 centred(u64 x, u64 q) { return x > q / 2 ? (i64)x - (i64)q : (i64)x; }

/* deterministic Miller-Rabin for 64-bit integers */
int orc_is_prime(u64 n) {
    static const u64 bases[12] = {2, 3, 5, 7, 11, 13, 17, 19, 23, 29, 31, 37};
    if (n < 2) return 0;
    for (int i = 0; i < 12; i++) { if (n == bases[i]) return 1; if (n % bases[i] == 0) return 0; }
    u64 d = n - 1; int r = 0;
    while ((d & 1) == 0) { d >>= 1; r++; }
    for (int i = 0; i < 12; i++) {
        u64 x = powmod(bases[i], d, n);
        if (x == 1 || x == n - 1) continue;
        int comp = 1;
        for (int k = 1; k < r; k++) { x = mulmod(x, x, n); if (x == n - 1) { comp = 0; break; } }
        if (comp) return 0;
    }
    return 1;
}

/* The `count` largest primes below 2^bits that are 1 mod 2^logstep, in descending order.
 * (Parameter rule of this build: NTT-friendly primes just below a power of two.) */
int orc_find_primes(int bits, int logstep, int count, u64 *out) {
    u64 step = 1ULL << logstep;
    u64 c = (1ULL << bits) - step + 1; /* largest candidate == 1 mod step below 2^bits */
    int found = 0;
    while (found < count && c > step) { if (orc_is_prime(c)) out[found++] = c; c -= step; }
    return found;
}

/* smallest x >= 2 whose power x^((q-1)/2N) has order exactly 2N */
static u64 find_psi(u64 q, int N) {
    for (u64 x = 2; x < q; x++) {
        u64 c = powmod(x, (q - 1) / (2 * (u64)N), q);
        if (powmod(c, (u64)N, q) == q - 1) return c;
    }
    return 0;
}

/* ------------------------------------------------------------------ unit roots for encode */

/* (c, s) = (cos, sin)(2 pi t / den), correctly rounded to binary64: the angle is reduced to the
 * first octant by integer arithmetic, so exact values (0, +-1) come out exact; the octant value
 * is evaluated in binary128 and rounded once. */
static void unit_root(long t, long den, double *c, double *s) {
    t %= den; if (t < 0) t += den;
    long e8 = 8 * t, oct = e8 / den, rem = e8 % den;
    __float128 qc, qs;
    if ((oct & 1) == 0) {
        __float128 phi = M_PIq / 4 * (__float128)rem / (__float128)den;
        qc = cosq(phi); qs = sinq(phi);
    } else {
        __float128 phi = M_PIq / 4 * (__float128)(den - rem) / (__float128)den;
        qc = sinq(phi); qs = cosq(phi);
    }
    double dc = (double)qc, ds = (double)qs;
    switch (oct / 2) { /* rotate by quadrant */
        case 0: *c = dc;  *s = ds;  break;
        case 1: *c = -ds; *s = dc;  break;
        case 2: *c = -dc; *s = -ds; break;
        default: *c = ds; *s = -dc; break;
    }
    *c += 0.0; *s += 0.0; /* no negative zeros in the tables */
}

/* ------------------------------------------------------------------ context */

void orc_destroy(orc_ctx *c) {
    if (!c) return;
    free(c->g5); free(c->uidx); free(c->T_re); free(c->T_im); free(c->U_re); free(c->U_im);
    free(c);
}

/* mods = q_0..q_{L-1}, p.  Returns NULL on invalid parameters. */
orc_ctx *orc_create(int logN, int L, const u64 *mods, int log_scale, int R, int B) {
    if (logN < 2 || logN > 17 || L < 1 || L + 1 > ORC_MAX_LIMBS) return NULL;
    int N = 1 << logN, n = N / 2;
    if (R < 1 || B < 1 || R % B || n % R) return NULL;
    orc_ctx *c = (orc_ctx *)calloc(1, sizeof(orc_ctx));
    c->logN = logN; c->N = N; c->n = n; c->L = L; c->log_scale = log_scale;
    c->R = R; c->B = B; c->G = R / B;
    for (int i = 0; i <= L; i++) {
        u64 q = mods[i];
        if (!orc_is_prime(q) || (q - 1) % (2 * (u64)N)) { orc_destroy(c); return NULL; }
        c->mod[i] = q;
        c->psi[i] = find_psi(q, N);
        c->psi_inv[i] = invmod(c->psi[i], q);
        c->n_inv[i] = invmod((u64)N % q, q);
    }
    c->g5 = (int *)malloc(sizeof(int) * n);
    c->uidx = (int *)malloc(sizeof(int) * n);
    long g = 1;
    for (int j = 0; j < n; j++) { c->g5[j] = (int)g; c->uidx[j] = (int)((g - 1) / 4); g = (g * 5) % (2L * N); }
    int nh = n / 2 > 0 ? n / 2 : 1;
    c->T_re = (double *)malloc(sizeof(double) * nh); c->T_im = (double *)malloc(sizeof(double) * nh);
    c->U_re = (double *)malloc(sizeof(double) * n);  c->U_im = (double *)malloc(sizeof(double) * n);
    for (int t = 0; t < nh; t++) { double cs, sn; unit_root(t, n, &cs, &sn); c->T_re[t] = cs; c->T_im[t] = -sn; }
    for (int k = 0; k < n; k++) { double cs, sn; unit_root(k, 2L * N, &cs, &sn); c->U_re[k] = cs; c->U_im[k] = -sn; }
    return c;
}

u64 orc_get_psi(const orc_ctx *c, int limb) { return c->psi[limb]; }
void orc_get_tables(const orc_ctx *c, double *T_re, double *T_im, double *U_re, double *U_im, int *g5, int *uidx) {
    int nh = c->n / 2 > 0 ? c->n / 2 : 1;
    memcpy(T_re, c->T_re, sizeof(double) * nh); memcpy(T_im, c->T_im, sizeof(double) * nh);
    memcpy(U_re, c->U_re, sizeof(double) * c->n); memcpy(U_im, c->U_im, sizeof(double) * c->n);
    memcpy(g5, c->g5, sizeof(int) * c->n); memcpy(uidx, c->uidx, sizeof(int) * c->n);
}

/* ------------------------------------------------------------------ negacyclic NTT (textbook) */

static int bitrev(int x, int bits) { int r = 0; for (int i = 0; i < bits; i++) { r = (r << 1) | (x & 1); x >>= 1; } return r; }

/* in-place cyclic transform out[t] = sum_i a[i] w^(t i) mod q: bit-reversal, then radix-2
 * decimation-in-time stages. */
static void cyclic_ntt(u64 *a, int N, int logN, u64 w, u64 q) {
    for (int i = 0; i < N; i++) { int j = bitrev(i, logN); if (i < j) { u64 t = a[i]; a[i] = a[j]; a[j] = t; } }
    for (int len = 2; len <= N; len <<= 1) {
        u64 wl = powmod(w, (u64)(N / len), q);
        for (int k0 = 0; k0 < N; k0 += len) {
            u64 wp = 1;
            for (int t = 0; t < len / 2; t++) {
                u64 x = a[k0 + t], y = mulmod(a[k0 + t + len / 2], wp, q);
                a[k0 + t] = addmod(x, y, q);
                a[k0 + t + len / 2] = submod(x, y, q);
                wp = mulmod(wp, wl, q);
            }
        }
    }
}

/* forward: a_hat[t] = a(psi^(2t+1)) = sum_i a_i psi^((2t+1) i), natural order in and out */
void orc_ntt(const orc_ctx *c, int limb, u64 *a) {
    u64 q = c->mod[limb], pw = 1;
    for (int i = 0; i < c->N; i++) { a[i] = mulmod(a[i], pw, q); pw = mulmod(pw, c->psi[limb], q); }
    cyclic_ntt(a, c->N, c->logN, mulmod(c->psi[limb], c->psi[limb], q), q);
}

/* inverse of orc_ntt */
void orc_intt(const orc_ctx *c, int limb, u64 *a) {
    u64 q = c->mod[limb];
    u64 winv = mulmod(c->psi_inv[limb], c->psi_inv[limb], q);
    cyclic_ntt(a, c->N, c->logN, winv, q);
    u64 pw = c->n_inv[limb];
    for (int i = 0; i < c->N; i++) { a[i] = mulmod(a[i], pw, q); pw = mulmod(pw, c->psi_inv[limb], q); }
}

/* out = a * b in Z_q[X]/(X^N+1) through the transform */
void orc_negacyclic_mul(const orc_ctx *c, int limb, const u64 *a, const u64 *b, u64 *out) {
    int N = c->N; u64 q = c->mod[limb];
    u64 *fa = (u64 *)malloc(8 * N), *fb = (u64 *)malloc(8 * N);
    memcpy(fa, a, 8 * N); memcpy(fb, b, 8 * N);
    orc_ntt(c, limb, fa); orc_ntt(c, limb, fb);
    for (int i = 0; i < N; i++) fa[i] = mulmod(fa[i], fb[i], q);
    orc_intt(c, limb, fa);
    memcpy(out, fa, 8 * N);
    free(fa); free(fb);
}

/* ------------------------------------------------------------------ automorphism X -> X^k */

/* coefficient domain: coefficient i moves to position i*k mod N, negated when i*k mod 2N >= N */
void orc_automorphism(const orc_ctx *c, int limb, long k, const u64 *in, u64 *out) {
    int N = c->N; u64 q = c->mod[limb];
    for (long i = 0; i < N; i++) {
        long e = (i * k) % (2L * N);
        if (e < N) out[e] = in[i];
        else out[e - N] = in[i] ? q - in[i] : 0;
    }
}

/* Galois element of the left rotation by r slots: k = 5^r mod 2N */
long orc_galois(const orc_ctx *c, int r) {
    long k = 1; r %= c->n; if (r < 0) r += c->n;
    for (int i = 0; i < r; i++) k = (k * 5) % (2L * c->N);
    return k;
}

/* the same map on transform values: with t <-> psi^(2t+1), (phi_k a)^[t] = a^[((2t+1)k mod 2N - 1)/2] */
void orc_automorphism_ntt(const orc_ctx *c, long k, const u64 *in, u64 *out) {
    for (long t = 0; t < c->N; t++) out[t] = in[(((2 * t + 1) * k) % (2L * c->N) - 1) / 2];
}

/* ------------------------------------------------------------------ encode / decode */

/* Canonical encode of a real slot vector z[n] at scale 2^log_scale into integer coefficients m[N]:
 *   m_k = rint( (Delta/n) * sum_j z_j cos(pi g_j k / N) ),  ties to even,
 * evaluated by the pinned operation order: y[u_j] = z_j, radix-2 decimation-in-time FFT in
 * IEEE binary64 without fused multiply-add, twist by U[k], scale by the power of two Delta/n.
 * (Compile with -ffp-contract=off.) */
void orc_encode(const orc_ctx *c, const double *z, int log_scale, i64 *m) {
    int n = c->n, logn = c->logN - 1;
    double *are = (double *)malloc(sizeof(double) * n), *aim = (double *)malloc(sizeof(double) * n);
    for (int j = 0; j < n; j++) { int pos = bitrev(c->uidx[j], logn); are[pos] = z[j]; aim[pos] = 0.0; }
    for (int s = 1; s <= logn; s++) {
        int h = 1 << (s - 1);
        for (int k0 = 0; k0 < n; k0 += 2 * h)
            for (int t = 0; t < h; t++) {
                double wre = c->T_re[t * (n / (2 * h))], wim = c->T_im[t * (n / (2 * h))];
                double xre = are[k0 + t], xim = aim[k0 + t];
                double yre = are[k0 + t + h], yim = aim[k0 + t + h];
                double p1 = yre * wre, p2 = yim * wim, p3 = yre * wim, p4 = yim * wre;
                double vre = p1 - p2, vim = p3 + p4;
                are[k0 + t] = xre + vre;     aim[k0 + t] = xim + vim;
                are[k0 + t + h] = xre - vre; aim[k0 + t + h] = xim - vim;
            }
    }
    double sc = ldexp(1.0, log_scale - logn); /* Delta / n, a power of two */
    for (int k = 0; k < n; k++) {
        double p1 = are[k] * c->U_re[k], p2 = aim[k] * c->U_im[k], p3 = are[k] * c->U_im[k], p4 = aim[k] * c->U_re[k];
        double cre = p1 - p2, cim = p3 + p4;
        m[k] = (i64)rint(cre * sc);       /* default rounding mode: to nearest, ties to even */
        m[k + n] = (i64)rint(cim * sc);
    }
    free(are); free(aim);
}

/* plain complex FFT, sign = -1 forward / +1 inverse kernel, unscaled (decode only: toleranced) */
static void fft_inplace(double *re, double *im, int n, int logn, int sign) {
    for (int i = 0; i < n; i++) { int j = bitrev(i, logn); if (i < j) { double t = re[i]; re[i] = re[j]; re[j] = t; t = im[i]; im[i] = im[j]; im[j] = t; } }
    for (int len = 2; len <= n; len <<= 1)
        for (int k0 = 0; k0 < n; k0 += len)
            for (int t = 0; t < len / 2; t++) {
                double ang = sign * 2.0 * M_PI * t / len, wr = cos(ang), wi = sin(ang);
                double yr = re[k0 + t + len / 2] * wr - im[k0 + t + len / 2] * wi;
                double yi = re[k0 + t + len / 2] * wi + im[k0 + t + len / 2] * wr;
                double xr = re[k0 + t], xi = im[k0 + t];
                re[k0 + t] = xr + yr; im[k0 + t] = xi + yi;
                re[k0 + t + len / 2] = xr - yr; im[k0 + t + len / 2] = xi - yi;
            }
}

/* decode: slots z_j = mu(omega^{g_j}) / scale for a real coefficient vector mu[N] (already CRT'd and
 * converted to double by the caller).  Since omega^{g_j n} = i and
 * omega^{g_j k} = conj(U[k]) * exp(+2 pi i u_j k / n):
 *   a_k = (mu_k + i mu_{k+n}) * conj(U[k]);   z_j * scale = sum_{k<n} a_k exp(+2 pi i u_j k / n). */
void orc_decode(const orc_ctx *c, const double *mu, double scale, double *z_re, double *z_im) {
    int n = c->n, logn = c->logN - 1;
    double *re = (double *)malloc(sizeof(double) * n), *im = (double *)malloc(sizeof(double) * n);
    for (int k = 0; k < n; k++) {
        double ur = c->U_re[k], ui = -c->U_im[k]; /* conj(U[k]) */
        re[k] = mu[k] * ur - mu[k + n] * ui;
        im[k] = mu[k] * ui + mu[k + n] * ur;
    }
    fft_inplace(re, im, n, logn, +1);
    for (int j = 0; j < n; j++) { z_re[j] = re[c->uidx[j]] / scale; if (z_im) z_im[j] = im[c->uidx[j]] / scale; }
    free(re); free(im);
}

/* ------------------------------------------------------------------ encryption (symmetric) */

/* signed small/int64 polynomial -> residues of one limb */
static void lift_i64(const i64 *v, int N, u64 q, u64 *out) { for (int i = 0; i < N; i++) out[i] = reduce_signed(v[i], q); }
static void lift_i8(const int8_t *v, int N, u64 q, u64 *out) { for (int i = 0; i < N; i++) out[i] = reduce_signed(v[i], q); }

/* ct = (c0, c1) = (-a*s + e + m, a) over the L ciphertext primes.
 * s[N] ternary, m[N] integer message, a[L][N] uniform residues, e[N] small error; ct[2][L][N]. */
void orc_encrypt(const orc_ctx *c, const int8_t *s, const i64 *m, const u64 *a, const int8_t *e, u64 *ct) {
    int N = c->N, L = c->L;
    u64 *sq = (u64 *)malloc(8 * N), *t = (u64 *)malloc(8 * N);
    for (int l = 0; l < L; l++) {
        u64 q = c->mod[l];
        lift_i8(s, N, q, sq);
        orc_negacyclic_mul(c, l, a + (size_t)l * N, sq, t);
        for (int i = 0; i < N; i++) {
            u64 v = q - t[i]; if (v == q) v = 0;                 /* -a*s */
            v = addmod(v, reduce_signed(e[i], q), q);            /* + e  */
            v = addmod(v, reduce_signed(m[i], q), q);            /* + m  */
            ct[(size_t)(0 * L + l) * N + i] = v;
            ct[(size_t)(1 * L + l) * N + i] = a[(size_t)l * N + i];
        }
    }
    free(sq); free(t);
}

/* Seed-compressed ciphertexts (Sec. 7: the public-random half of a fresh ciphertext is regenerated from a short seed).
 * The uniform polynomial a is a pure function of (seed, stream): a[l][x] = h(seed, stream, l*N + x) mod q_l with the
 * 64-bit counter hash  mix(x): x ^= x>>32; x *= 0x9E3779B97F4A7C15; x ^= x>>29; x *= 0xBB67AE8584CAA73B; x ^= x>>32;
 * h = mix(mix(mix(seed + 0x9E3779B97F4A7C15) ^ (stream * 0xBB67AE8584CAA73B)) + ctr * 0x9E3779B97F4A7C15). */
static u64 mix64(u64 x) {
    x ^= x >> 32; x *= 0x9E3779B97F4A7C15ULL; x ^= x >> 29; x *= 0xBB67AE8584CAA73BULL; x ^= x >> 32;
    return x;
}
u64 orc_hash64(u64 seed, u64 stream, u64 ctr) {
    u64 a = mix64(seed + 0x9E3779B97F4A7C15ULL);
    u64 b = mix64(a ^ (stream * 0xBB67AE8584CAA73BULL));
    return mix64(b + ctr * 0x9E3779B97F4A7C15ULL);
}
void orc_expand_uniform(const orc_ctx *c, u64 seed, u64 stream, u64 *a) {
    int N = c->N, L = c->L;
    for (int l = 0; l < L; l++)
        for (int x = 0; x < N; x++) a[(size_t)l * N + x] = orc_hash64(seed, stream, (u64)l * N + x) % c->mod[l];
}

/* mu = c0 + c1*s, residues [L][N]; the caller reconstructs centred integers by CRT */
void orc_decrypt_residues(const orc_ctx *c, const int8_t *s, const u64 *ct, u64 *mu) {
    int N = c->N, L = c->L;
    u64 *sq = (u64 *)malloc(8 * N), *t = (u64 *)malloc(8 * N);
    for (int l = 0; l < L; l++) {
        u64 q = c->mod[l];
        lift_i8(s, N, q, sq);
        orc_negacyclic_mul(c, l, ct + (size_t)(1 * L + l) * N, sq, t);
        for (int i = 0; i < N; i++) mu[(size_t)l * N + i] = addmod(ct[(size_t)(0 * L + l) * N + i], t[i], q);
    }
    free(sq); free(t);
}

/* mu = c0 + c1*s over the first nl moduli of a ciphertext stored with nl limbs: ct[2][nl][N] */
void orc_decrypt_residues_limbs(const orc_ctx *c, const int8_t *s, const u64 *ct, int nl, u64 *mu) {
    int N = c->N;
    u64 *sq = (u64 *)malloc(8 * N), *t = (u64 *)malloc(8 * N);
    for (int l = 0; l < nl; l++) {
        u64 q = c->mod[l];
        lift_i8(s, N, q, sq);
        orc_negacyclic_mul(c, l, ct + (size_t)(1 * nl + l) * N, sq, t);
        for (int i = 0; i < N; i++) mu[(size_t)l * N + i] = addmod(ct[(size_t)(0 * nl + l) * N + i], t[i], q);
    }
    free(sq); free(t);
}

/* Output compaction (Sec. 7, storage and upload footprint: switch a ciphertext down to the minimal modulus the
 * remaining computation -- here only decryption -- needs).  On each of the two polynomials:
 *   rescale != 0: divide by the last prime q_{L-1} first:  r = centred lift of [c]_{q_{L-1}};
 *       c'_i = (c_i - r) * q_{L-1}^{-1} mod q_i, i.e. c' = (c - r) / q_{L-1} exactly; message and scale are divided by
 *       q_{L-1} and a rounding error (tau_0 + tau_1 s, |tau| <= 1/2 per coefficient) is added;
 *   then keep limbs 0..keep-1 (no division, no error: c_0 + c_1 s is the same integer mod q_0..q_{keep-1}; valid
 *       while |message + noise| < q_0..q_{keep-1} / 2).
 * ct[2][L][N] coefficient domain -> out[2][keep][N]; keep <= L-1 when rescaling, keep <= L otherwise. */
void orc_compact(const orc_ctx *c, const u64 *ct, int keep, int rescale, u64 *out) {
    int N = c->N, L = c->L; u64 ql = c->mod[L - 1];
    for (int poly = 0; poly < 2; poly++)
        for (int i = 0; i < keep; i++) {
            u64 q = c->mod[i], qlinv = invmod(ql % q, q);
            for (int x = 0; x < N; x++) {
                u64 v = ct[((size_t)poly * L + i) * N + x];
                if (rescale) {
                    i64 r = centred(ct[((size_t)poly * L + (L - 1)) * N + x], ql);
                    v = mulmod(submod(v, reduce_signed(r, q), q), qlinv, q);
                }
                out[((size_t)poly * keep + i) * N + x] = v;
            }
        }
}

/* ------------------------------------------------------------------ evaluation keys, key switching */

/* Evaluation key for the left rotation by r (k = 5^r, s' = phi_k(s)); one special prime, one digit per
 * ciphertext prime.  For digit j:  b_j = -a_j*s + e_j + F_j*s'  over the L+1 moduli, where
 * F_j = p * Qhat_j * [Qhat_j^{-1}]_{q_j}: F_j = p mod q_j on limb j and 0 on every other limb.
 * a[L][L+1][N] uniform, e[L][N] small; evk[L][2][L+1][N] with [j][0] = b_j, [j][1] = a_j. */
void orc_evk_gen(const orc_ctx *c, const int8_t *s, int r, const u64 *a, const int8_t *e, u64 *evk) {
    int N = c->N, L = c->L;
    long k = orc_galois(c, r);
    u64 *sq = (u64 *)malloc(8 * N), *sp = (u64 *)malloc(8 * N), *t = (u64 *)malloc(8 * N);
    for (int j = 0; j < L; j++)
        for (int i = 0; i <= L; i++) {
            u64 q = c->mod[i];
            const u64 *aj = a + ((size_t)j * (L + 1) + i) * N;
            u64 *bj = evk + (((size_t)j * 2 + 0) * (L + 1) + i) * N;
            u64 *ao = evk + (((size_t)j * 2 + 1) * (L + 1) + i) * N;
            lift_i8(s, N, q, sq);
            orc_automorphism(c, i, k, sq, sp);                    /* s' = phi_k(s) */
            orc_negacyclic_mul(c, i, aj, sq, t);
            u64 F = (i == j) ? c->mod[L] % q : 0;
            for (int x = 0; x < N; x++) {
                u64 v = t[x] ? q - t[x] : 0;                      /* -a_j*s   */
                v = addmod(v, reduce_signed(e[(size_t)j * N + x], q), q);   /* + e_j    */
                v = addmod(v, mulmod(F, sp[x], q), q);            /* + F_j*s' */
                bj[x] = v; ao[x] = aj[x];
            }
        }
    free(sq); free(sp); free(t);
}

/* Relinearisation key: the evaluation key of orc_evk_gen with s' = s*s (negacyclic square of the secret) in place of an
 * automorphism of s: b_j = -a_j*s + e_j + F_j*s^2.  Switching d2 with it gives (ks0, ks1) with ks0 + ks1*s ~ d2*s^2. */
void orc_rlk_gen(const orc_ctx *c, const int8_t *s, const u64 *a, const int8_t *e, u64 *evk) {
    int N = c->N, L = c->L;
    u64 *sq = (u64 *)malloc(8 * N), *s2 = (u64 *)malloc(8 * N), *t = (u64 *)malloc(8 * N);
    for (int j = 0; j < L; j++)
        for (int i = 0; i <= L; i++) {
            u64 q = c->mod[i];
            const u64 *aj = a + ((size_t)j * (L + 1) + i) * N;
            u64 *bj = evk + (((size_t)j * 2 + 0) * (L + 1) + i) * N;
            u64 *ao = evk + (((size_t)j * 2 + 1) * (L + 1) + i) * N;
            lift_i8(s, N, q, sq);
            orc_negacyclic_mul(c, i, sq, sq, s2);                 /* s' = s^2 */
            orc_negacyclic_mul(c, i, aj, sq, t);
            u64 F = (i == j) ? c->mod[L] % q : 0;
            for (int x = 0; x < N; x++) {
                u64 v = t[x] ? q - t[x] : 0;
                v = addmod(v, reduce_signed(e[(size_t)j * N + x], q), q);
                v = addmod(v, mulmod(F, s2[x], q), q);
                bj[x] = v; ao[x] = aj[x];
            }
        }
    free(sq); free(s2); free(t);
}

/* ModDown: u[L+1][N] over {q_0..q_{L-1}, p}  ->  out[L][N] = round(u / p):
 * rt = centred lift of [u]_p;  out_i = (u_i - rt) * p^{-1} mod q_i. */
void orc_moddown(const orc_ctx *c, const u64 *u, u64 *out) {
    int N = c->N, L = c->L; u64 p = c->mod[L];
    for (int i = 0; i < L; i++) {
        u64 q = c->mod[i], pinv = invmod(p % q, q);
        for (int x = 0; x < N; x++) {
            i64 rt = centred(u[(size_t)L * N + x], p);
            out[(size_t)i * N + x] = mulmod(submod(u[(size_t)i * N + x], reduce_signed(rt, q), q), pinv, q);
        }
    }
}

/* KeySwitch: d[L][N] in R_Q  ->  (ks0, ks1)[L][N] with ks0 + ks1*s ~ d*s'.
 * digits d_j = [d]_{q_j}, centred lift, reduced into every modulus; (u0,u1) = sum_j d_j*(b_j, a_j)
 * over the L+1 moduli; ModDown of each. */
void orc_keyswitch(const orc_ctx *c, const u64 *d, const u64 *evk, u64 *ks0, u64 *ks1) {
    int N = c->N, L = c->L;
    u64 *u0 = (u64 *)calloc((size_t)(L + 1) * N, 8), *u1 = (u64 *)calloc((size_t)(L + 1) * N, 8);
    u64 *dj = (u64 *)malloc(8 * N), *t = (u64 *)malloc(8 * N);
    for (int j = 0; j < L; j++)
        for (int i = 0; i <= L; i++) {
            u64 q = c->mod[i];
            for (int x = 0; x < N; x++) dj[x] = reduce_signed(centred(d[(size_t)j * N + x], c->mod[j]), q);
            orc_negacyclic_mul(c, i, dj, evk + (((size_t)j * 2 + 0) * (L + 1) + i) * N, t);
            for (int x = 0; x < N; x++) u0[(size_t)i * N + x] = addmod(u0[(size_t)i * N + x], t[x], q);
            orc_negacyclic_mul(c, i, dj, evk + (((size_t)j * 2 + 1) * (L + 1) + i) * N, t);
            for (int x = 0; x < N; x++) u1[(size_t)i * N + x] = addmod(u1[(size_t)i * N + x], t[x], q);
        }
    orc_moddown(c, u0, ks0);
    orc_moddown(c, u1, ks1);
    free(u0); free(u1); free(dj); free(t);
}

/* Rotate(ct, r) = (phi_k(c0) + ks0, ks1), (ks0, ks1) = KeySwitch(phi_k(c1)) under evk_r:
 * automorphism first, then key switch. */
void orc_rotate(const orc_ctx *c, const u64 *ct, int r, const u64 *evk_r, u64 *out) {
    int N = c->N, L = c->L;
    long k = orc_galois(c, r);
    u64 *pc0 = (u64 *)malloc((size_t)L * N * 8), *pc1 = (u64 *)malloc((size_t)L * N * 8);
    u64 *ks0 = (u64 *)malloc((size_t)L * N * 8), *ks1 = (u64 *)malloc((size_t)L * N * 8);
    for (int l = 0; l < L; l++) {
        orc_automorphism(c, l, k, ct + (size_t)(0 * L + l) * N, pc0 + (size_t)l * N);
        orc_automorphism(c, l, k, ct + (size_t)(1 * L + l) * N, pc1 + (size_t)l * N);
    }
    orc_keyswitch(c, pc1, evk_r, ks0, ks1);
    for (int l = 0; l < L; l++)
        for (int x = 0; x < N; x++) {
            out[(size_t)(0 * L + l) * N + x] = addmod(pc0[(size_t)l * N + x], ks0[(size_t)l * N + x], c->mod[l]);
            out[(size_t)(1 * L + l) * N + x] = ks1[(size_t)l * N + x];
        }
    free(pc0); free(pc1); free(ks0); free(ks1);
}

/* Same rotation evaluated the "hoisted" way: decompose c1 into centred digits FIRST, apply the
 * automorphism to each lifted digit, then the inner product and ModDown.  Used only by a test
 * that pins the two orders to identical bits. */
void orc_rotate_hoisted(const orc_ctx *c, const u64 *ct, int r, const u64 *evk_r, u64 *out) {
    int N = c->N, L = c->L;
    long k = orc_galois(c, r);
    u64 *u0 = (u64 *)calloc((size_t)(L + 1) * N, 8), *u1 = (u64 *)calloc((size_t)(L + 1) * N, 8);
    u64 *dj = (u64 *)malloc(8 * N), *pd = (u64 *)malloc(8 * N), *t = (u64 *)malloc(8 * N);
    u64 *ks0 = (u64 *)malloc((size_t)L * N * 8), *ks1 = (u64 *)malloc((size_t)L * N * 8);
    for (int j = 0; j < L; j++)
        for (int i = 0; i <= L; i++) {
            u64 q = c->mod[i];
            for (int x = 0; x < N; x++) dj[x] = reduce_signed(centred(ct[(size_t)(1 * L + j) * N + x], c->mod[j]), q);
            orc_automorphism(c, i, k, dj, pd);
            orc_negacyclic_mul(c, i, pd, evk_r + (((size_t)j * 2 + 0) * (L + 1) + i) * N, t);
            for (int x = 0; x < N; x++) u0[(size_t)i * N + x] = addmod(u0[(size_t)i * N + x], t[x], q);
            orc_negacyclic_mul(c, i, pd, evk_r + (((size_t)j * 2 + 1) * (L + 1) + i) * N, t);
            for (int x = 0; x < N; x++) u1[(size_t)i * N + x] = addmod(u1[(size_t)i * N + x], t[x], q);
        }
    orc_moddown(c, u0, ks0);
    orc_moddown(c, u1, ks1);
    for (int l = 0; l < L; l++) {
        orc_automorphism(c, l, k, ct + (size_t)(0 * L + l) * N, t);
        for (int x = 0; x < N; x++) {
            out[(size_t)(0 * L + l) * N + x] = addmod(t[x], ks0[(size_t)l * N + x], c->mod[l]);
            out[(size_t)(1 * L + l) * N + x] = ks1[(size_t)l * N + x];
        }
    }
    free(u0); free(u1); free(dj); free(pd); free(t); free(ks0); free(ks1);
}

/* Baby set: baby[0] = ct, baby[r] = Rotate(ct, r) taken directly from the original ciphertext,
 * r = 1..B-1.  evk[(r-1)] is the key of rotation r.  baby[B][2][L][N]. */
void orc_baby_set(const orc_ctx *c, const u64 *ct, const u64 *evk, u64 *baby) {
    size_t ctw = (size_t)2 * c->L * c->N, evw = (size_t)c->L * 2 * (c->L + 1) * c->N;
    memcpy(baby, ct, ctw * 8);
#pragma omp parallel for schedule(dynamic)
    for (int r = 1; r < c->B; r++) orc_rotate(c, ct, r, evk + (size_t)(r - 1) * evw, baby + (size_t)r * ctw);
}

/* ------------------------------------------------------------------ candidate block, MAC, rotate-and-sum */

/* Encode one block of candidate rows.  rows[n_rows][R] float32 (n_rows <= n, missing rows are zero);
 * for g < G, b < B the slot vector is  z[i] = M[(i - g*B) mod n][(i + b) mod R]  (diagonal b + g*B of
 * the block, shifted in plaintext by the giant-step amount), encoded at scale Delta and reduced into
 * each ciphertext prime.  pt[G][B][L][N]. */
void orc_encode_block(const orc_ctx *c, const float *rows, int n_rows, u64 *pt) {
    int N = c->N, n = c->n, L = c->L, R = c->R, B = c->B, G = c->G;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int g = 0; g < G; g++)
        for (int b = 0; b < B; b++) {
            double *z = (double *)malloc(sizeof(double) * n);
            i64 *m = (i64 *)malloc(sizeof(i64) * N);
            for (int i = 0; i < n; i++) {
                int row = ((i - g * B) % n + n) % n, col = (i + b) % R;
                z[i] = row < n_rows ? (double)rows[(size_t)row * R + col] : 0.0;
            }
            orc_encode(c, z, c->log_scale, m);
            for (int l = 0; l < L; l++) lift_i64(m, N, c->mod[l], pt + (((size_t)g * B + b) * L + l) * N);
            free(z); free(m);
        }
}

/* inner[g] = ( sum_b pt[g,b]*baby[b].c0 , sum_b pt[g,b]*baby[b].c1 ) in R_Q.  inner[G][2][L][N]. */
void orc_mac(const orc_ctx *c, const u64 *pt, const u64 *baby, u64 *inner) {
    int N = c->N, L = c->L, B = c->B, G = c->G;
    memset(inner, 0, (size_t)G * 2 * L * N * 8);
#pragma omp parallel for collapse(3) schedule(dynamic)
    for (int g = 0; g < G; g++)
        for (int comp = 0; comp < 2; comp++)
            for (int l = 0; l < L; l++) {
                u64 *t = (u64 *)malloc(8 * N);
                u64 *acc = inner + (((size_t)g * 2 + comp) * L + l) * N;
                for (int b = 0; b < B; b++) {
                    orc_negacyclic_mul(c, l, pt + (((size_t)g * B + b) * L + l) * N,
                                       baby + (((size_t)b * 2 + comp) * L + l) * N, t);
                    for (int x = 0; x < N; x++) acc[x] = addmod(acc[x], t[x], c->mod[l]);
                }
                free(t);
            }
}

/* Encrypted database (Sec. 2, deployment setting: the candidate diagonals are ciphertexts too).  Symmetric encryption of
 * the R encoded diagonals of a block: ctdb[g][b] = (-a*s + e + pt[g][b], a).  pt[R][L][N], a[R][L][N], e[R][N]. */
void orc_encrypt_block(const orc_ctx *c, const int8_t *s, const u64 *pt, const u64 *a, const int8_t *e, u64 *ctdb) {
    int N = c->N, L = c->L, R = c->R;
    u64 *sq = (u64 *)malloc(8 * N), *t = (u64 *)malloc(8 * N);
    for (int r = 0; r < R; r++)
        for (int l = 0; l < L; l++) {
            u64 q = c->mod[l];
            const u64 *ar = a + ((size_t)r * L + l) * N;
            u64 *c0 = ctdb + (((size_t)r * 2 + 0) * L + l) * N, *c1 = ctdb + (((size_t)r * 2 + 1) * L + l) * N;
            lift_i8(s, N, q, sq);
            orc_negacyclic_mul(c, l, ar, sq, t);
            for (int x = 0; x < N; x++) {
                u64 v = t[x] ? q - t[x] : 0;
                v = addmod(v, reduce_signed(e[(size_t)r * N + x], q), q);
                c0[x] = addmod(v, pt[((size_t)r * L + l) * N + x], q);
                c1[x] = ar[x];
            }
        }
    free(sq); free(t);
}

/* Ciphertext x ciphertext multiply-accumulate over the baby steps: for every giant step g the degree-2 ciphertext
 * (d0, d1, d2) = sum_b (x0*y0, x0*y1 + x1*y0, x1*y1), x = ctdb[g][b], y = baby[b]; decrypts as d0 + d1*s + d2*s^2.
 * ctdb[R][2][L][N], baby[B][2][L][N] -> inner3[G][3][L][N]. */
void orc_mac_ct(const orc_ctx *c, const u64 *ctdb, const u64 *baby, u64 *inner3) {
    int N = c->N, L = c->L, B = c->B, G = c->G;
    memset(inner3, 0, (size_t)G * 3 * L * N * 8);
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int g = 0; g < G; g++)
        for (int l = 0; l < L; l++) {
            u64 q = c->mod[l];
            u64 *t = (u64 *)malloc(8 * N);
            u64 *d0 = inner3 + (((size_t)g * 3 + 0) * L + l) * N, *d1 = inner3 + (((size_t)g * 3 + 1) * L + l) * N,
                *d2 = inner3 + (((size_t)g * 3 + 2) * L + l) * N;
            for (int b = 0; b < B; b++) {
                const u64 *x0 = ctdb + ((((size_t)g * B + b) * 2 + 0) * L + l) * N, *x1 = ctdb + ((((size_t)g * B + b) * 2 + 1) * L + l) * N;
                const u64 *y0 = baby + (((size_t)b * 2 + 0) * L + l) * N, *y1 = baby + (((size_t)b * 2 + 1) * L + l) * N;
                orc_negacyclic_mul(c, l, x0, y0, t);
                for (int x = 0; x < N; x++) d0[x] = addmod(d0[x], t[x], q);
                orc_negacyclic_mul(c, l, x0, y1, t);
                for (int x = 0; x < N; x++) d1[x] = addmod(d1[x], t[x], q);
                orc_negacyclic_mul(c, l, x1, y0, t);
                for (int x = 0; x < N; x++) d1[x] = addmod(d1[x], t[x], q);
                orc_negacyclic_mul(c, l, x1, y1, t);
                for (int x = 0; x < N; x++) d2[x] = addmod(d2[x], t[x], q);
            }
            free(t);
        }
}

/* Relinearisation of one degree-2 ciphertext: (c0, c1) = (d0 + ks0, d1 + ks1), (ks0, ks1) = KeySwitch(d2) under the
 * relinearisation key.  d[3][L][N] -> ct[2][L][N]. */
void orc_relin(const orc_ctx *c, const u64 *d, const u64 *rlk, u64 *ct) {
    int N = c->N, L = c->L;
    u64 *ks0 = (u64 *)malloc((size_t)L * N * 8), *ks1 = (u64 *)malloc((size_t)L * N * 8);
    orc_keyswitch(c, d + (size_t)2 * L * N, rlk, ks0, ks1);
    for (int l = 0; l < L; l++)
        for (int x = 0; x < N; x++) {
            ct[((size_t)0 * L + l) * N + x] = addmod(d[((size_t)0 * L + l) * N + x], ks0[(size_t)l * N + x], c->mod[l]);
            ct[((size_t)1 * L + l) * N + x] = addmod(d[((size_t)1 * L + l) * N + x], ks1[(size_t)l * N + x], c->mod[l]);
        }
    free(ks0); free(ks1);
}

/* score_ct = sum_g rot_{gB}(inner[g]) by Horner with the single key of rotation B:
 * acc = inner[G-1]; for g = G-2..0: acc = Rotate(acc, B) + inner[g]. */
void orc_rotate_sum(const orc_ctx *c, const u64 *inner, const u64 *evk_B, u64 *score_ct) {
    int N = c->N, L = c->L, G = c->G;
    size_t ctw = (size_t)2 * L * N;
    u64 *acc = (u64 *)malloc(ctw * 8), *rot = (u64 *)malloc(ctw * 8);
    memcpy(acc, inner + (size_t)(G - 1) * ctw, ctw * 8);
    for (int g = G - 2; g >= 0; g--) {
        orc_rotate(c, acc, c->B, evk_B, rot);
        for (int comp = 0; comp < 2; comp++)
            for (int l = 0; l < L; l++)
                for (int x = 0; x < N; x++) {
                    size_t o = ((size_t)comp * L + l) * N + x;
                    acc[o] = addmod(rot[o], inner[(size_t)g * ctw + o], c->mod[l]);
                }
    }
    memcpy(score_ct, acc, ctw * 8);
    free(acc); free(rot);
}

/* ---- second evaluation order of the giant steps: distinct keys, one ModDown ("lazy") --------------------------------
 * The paper fixes only WHAT the giant steps compute, sum_g rot_{gB}(inner[g]) (Sec. 3.1 Detail); Horner with one key
 * (orc_rotate_sum) is one order of evaluation, this is the other one this build supports.  Every term is rotated by its
 * own amount gB with the key of that rotation, the key products are SUMMED in R_{Qp} and brought down once:
 *   (U0, U1) = sum_{g>=1} sum_j digit_j(phi_g(inner[g].c1)) * (b_j, a_j)[key of rotation gB]      over the L+1 moduli,
 *   score = ( inner[0].c0 + sum_{g>=1} phi_g(inner[g].c0) + ModDown(U0),  inner[0].c1 + ModDown(U1) ),  phi_g: X -> X^(5^(gB)).
 * One rounding (ModDown) instead of G-1, and no key-switch result is ever key-switched again. */

/* (u0, u1) += sum_j d_j * (b_j, a_j) over the L+1 moduli: the inner product of orc_keyswitch without its ModDown */
void orc_ks_accumulate(const orc_ctx *c, const u64 *d, const u64 *evk, u64 *u0, u64 *u1) {
    int N = c->N, L = c->L;
    u64 *dj = (u64 *)malloc(8 * N), *t = (u64 *)malloc(8 * N);
    for (int j = 0; j < L; j++)
        for (int i = 0; i <= L; i++) {
            u64 q = c->mod[i];
            for (int x = 0; x < N; x++) dj[x] = reduce_signed(centred(d[(size_t)j * N + x], c->mod[j]), q);
            orc_negacyclic_mul(c, i, dj, evk + (((size_t)j * 2 + 0) * (L + 1) + i) * N, t);
            for (int x = 0; x < N; x++) u0[(size_t)i * N + x] = addmod(u0[(size_t)i * N + x], t[x], q);
            orc_negacyclic_mul(c, i, dj, evk + (((size_t)j * 2 + 1) * (L + 1) + i) * N, t);
            for (int x = 0; x < N; x++) u1[(size_t)i * N + x] = addmod(u1[(size_t)i * N + x], t[x], q);
        }
    free(dj); free(t);
}

/* inner[G][2][L][N]; evk_giant[G-1] keys, entry g-1 the key of rotation g*B; score_ct[2][L][N] */
void orc_rotate_sum_lazy(const orc_ctx *c, const u64 *inner, const u64 *evk_giant, u64 *score_ct) {
    int N = c->N, L = c->L, G = c->G;
    size_t LN = (size_t)L * N, ctw = 2 * LN, evw = (size_t)L * 2 * (L + 1) * N;
    u64 *u0 = (u64 *)calloc((size_t)(L + 1) * N, 8), *u1 = (u64 *)calloc((size_t)(L + 1) * N, 8);
    u64 *pc = (u64 *)malloc(LN * 8), *md = (u64 *)malloc(LN * 8);
    memcpy(score_ct, inner, ctw * 8);                              /* the g = 0 term is not rotated */
    for (int g = 1; g < G; g++) {
        long k = orc_galois(c, g * c->B);
        const u64 *ct = inner + (size_t)g * ctw;
        for (int l = 0; l < L; l++) orc_automorphism(c, l, k, ct + (size_t)l * N, pc + (size_t)l * N);          /* phi_g(c0) */
        for (int l = 0; l < L; l++)
            for (int x = 0; x < N; x++) score_ct[(size_t)l * N + x] = addmod(score_ct[(size_t)l * N + x], pc[(size_t)l * N + x], c->mod[l]);
        for (int l = 0; l < L; l++) orc_automorphism(c, l, k, ct + LN + (size_t)l * N, pc + (size_t)l * N);     /* phi_g(c1) */
        orc_ks_accumulate(c, pc, evk_giant + (size_t)(g - 1) * evw, u0, u1);
    }
    if (G > 1) {
        orc_moddown(c, u0, md);
        for (int l = 0; l < L; l++)
            for (int x = 0; x < N; x++) score_ct[(size_t)l * N + x] = addmod(score_ct[(size_t)l * N + x], md[(size_t)l * N + x], c->mod[l]);
        orc_moddown(c, u1, md);
        for (int l = 0; l < L; l++)
            for (int x = 0; x < N; x++) score_ct[LN + (size_t)l * N + x] = addmod(score_ct[LN + (size_t)l * N + x], md[(size_t)l * N + x], c->mod[l]);
    }
    free(u0); free(u1); free(pc); free(md);
}

/* ---- pieces of the packed projection (Sec. 3.1 Detail: all chunks of W in one object per diagonal, combined with 0/1
 * plaintext masks; see oracle.py PackedProjection for the steps) -------------------------------------------------------- */

/* encode a real slot vector at scale 2^log_scale and reduce it into the L ciphertext primes: pt[L][N] */
void orc_encode_plain(const orc_ctx *c, const double *z, int log_scale, u64 *pt) {
    int N = c->N, L = c->L;
    i64 *m = (i64 *)malloc(sizeof(i64) * N);
    orc_encode(c, z, log_scale, m);
    for (int l = 0; l < L; l++) lift_i64(m, N, c->mod[l], pt + (size_t)l * N);
    free(m);
}

/* acc[2][L][N] += ct[2][L][N] * pt[L][N]: ciphertext x plaintext product of both components, every limb.  A mask
 * multiply is exactly this (the mask is a public constant: no key switch, no relinearisation). */
void orc_mul_plain_acc(const orc_ctx *c, const u64 *ct, const u64 *pt, u64 *acc) {
    int N = c->N, L = c->L;
    u64 *t = (u64 *)malloc(8 * N);
    for (int comp = 0; comp < 2; comp++)
        for (int l = 0; l < L; l++) {
            size_t o = ((size_t)comp * L + l) * N;
            orc_negacyclic_mul(c, l, ct + o, pt + (size_t)l * N, t);
            for (int x = 0; x < N; x++) acc[o + x] = addmod(acc[o + x], t[x], c->mod[l]);
        }
    free(t);
}

/* One block end to end: encode, MAC, rotate-and-sum.  Optional outputs pt_out / inner_out may be NULL. */
void orc_score_block(const orc_ctx *c, const float *rows, int n_rows, const u64 *baby, const u64 *evk_B,
                     u64 *score_ct, u64 *pt_out, u64 *inner_out) {
    size_t ptw = (size_t)c->R * c->L * c->N, inw = (size_t)c->G * 2 * c->L * c->N;
    u64 *pt = pt_out ? pt_out : (u64 *)malloc(ptw * 8);
    u64 *inner = inner_out ? inner_out : (u64 *)malloc(inw * 8);
    orc_encode_block(c, rows, n_rows, pt);
    orc_mac(c, pt, baby, inner);
    orc_rotate_sum(c, inner, evk_B, score_ct);
    if (!pt_out) free(pt);
    if (!inner_out) free(inner);
}

int orc_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
