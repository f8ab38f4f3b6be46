// Element-wise kernels of the scoring path other than the multiply-accumulate (mac.cu): the pieces of hybrid key
// switching (digit lift, inner product with the evaluation key, ModDown), the automorphism gather, the output
// compaction, and the small helpers of the client half.  All polynomials are [.][limb][N] arrays of 64-bit residues in
// [0, q).
#include "internal.h"
#include "debugcheck.cuh"

namespace {

constexpr int kThreads = 256;

inline int grid_for(int64_t work, int per_block = kThreads, int cap = 148 * 16) {
    int64_t g = (work + per_block - 1) / per_block;
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    return (int)g;
}

// ------------------------------------------------------------------------------------------ key switching

// digits[item][j][i][x] = centred lift of src[item][j][x] (a residue mod q_j, coefficient domain) reduced mod
// modulus i, for j < L, i <= L.
__global__ void __launch_bounds__(kThreads) k_lift_digits(const u64* __restrict__ src, long long src_stride,
                                                          u64* __restrict__ digits, int N, int L, long long nitems,
                                                          LimbTable lt) {
    const long long total = nitems * L * N;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const int x = (int)(idx % N);
        const int j = (int)((idx / N) % L);
        const long long item = idx / ((long long)N * L);
        const u64 v = src[item * src_stride + (long long)j * N + x];
        const u64 qj = lt.c[j].q;
        const bool neg = v > lt.c[j].half;
        const u64 mag = neg ? qj - v : v;
        u64* d = digits + ((item * L + j) * (L + 1)) * N + x;
        for (int i = 0; i <= L; i++) {
            u64 r = barrett64(mag, lt.c[i]);
            d[(long long)i * N] = (neg && r) ? lt.c[i].q - r : r;
        }
    }
}

// u[item][comp][i][x] = sum_j digits[item_d][j][i][x] * key[j][comp][i][x] mod modulus i.
// digit_stride = 0 shares one digit set among all items (hoisted rotations of one ciphertext); the key of item
// `it` is keytab[rot0 + it*rot_inc].
__global__ void __launch_bounds__(kThreads) k_ks_inner(const u64* __restrict__ digits, long long digit_stride,
                                                       const u64* const* __restrict__ keytab, int rot0, int rot_inc,
                                                       u64* __restrict__ u, int N, int L, long long nitems,
                                                       LimbTable lt, int f64) {
    const long long L1N = (long long)(L + 1) * N;
    const long long total = nitems * L1N;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const long long item = idx / L1N;
        const long long pos = idx % L1N;  // i*N + x
        const int i = (int)(pos / N);
        const u64* key = keytab[rot0 + (int)item * rot_inc];
        const u64* d = digits + item * digit_stride + pos;
        const LimbConst& lc = lt.c[i];
        u64* o = u + item * 2 * L1N + pos;
        if (f64 && lc.q < (1ULL << 50)) {
            // moduli below 2^50: exact two-word binary64 sums (acc2_fma) of eight digits at a time, their integer words added up
            const double qd = (double)lc.q, halfd = (double)lc.half;
            long long m0 = 0, s0 = 0, m1 = 0, s1 = 0;
            for (int j0 = 0; j0 < L; j0 += 8) {
                double ah0 = kAcc2Start, al0 = 0, ah1 = kAcc2Start, al1 = 0;
                const int j1 = j0 + 8 < L ? j0 + 8 : L;
#pragma unroll 4
                for (int j = j0; j < j1; j++) {
                    const double dv = residue_to_balanced_f64(d[(long long)j * L1N], qd, halfd);
                    acc2_fma(ah0, al0, residue_to_f64(__ldcs(key + ((long long)j * 2 + 0) * L1N + pos)), dv);
                    acc2_fma(ah1, al1, residue_to_f64(__ldcs(key + ((long long)j * 2 + 1) * L1N + pos)), dv);
                }
                m0 += acc2_high(ah0), s0 += acc2_low(al0);
                m1 += acc2_high(ah1), s1 += acc2_low(al1);
            }
            o[0] = acc2_reduce(m0, s0, lc);
            o[L1N] = acc2_reduce(m1, s1, lc);
            continue;
        }
        u64 h0 = 0, l0 = 0, h1 = 0, l1 = 0;
#pragma unroll 4
        for (int j = 0; j < L; j++) {
            u64 dv = d[(long long)j * L1N];
            mac128(h0, l0, dv, __ldcs(key + ((long long)j * 2 + 0) * L1N + pos));
            mac128(h1, l1, dv, __ldcs(key + ((long long)j * 2 + 1) * L1N + pos));
        }
        o[0] = reduce128(h0, l0, lc);
        o[L1N] = reduce128(h1, l1, lc);
    }
}

// Streaming form of the same inner product for L <= 4 digits.  A thread owns one position (modulus i, coefficient x)
// and loops over the items.  When the items share one digit set and differ by key (the hoisted baby rotations:
// KEYS_STREAM), the L digit words stay in registers and the 2L key words of each item stream past them; when the
// items share the key (rotate-and-sum over blocks), the key words stay and the digit words stream.  The streamed
// words of the next item are in flight while the current item is multiplied.  Moduli below 2^50 use the carry-free
// 25-bit Karatsuba products of the multiply-accumulate kernel; the special prime uses 128-bit accumulation.
// MODE 0: moduli below 2^50, 25-bit halves, Karatsuba (3 products); MODE 1: moduli below 2^60 (the special prime),
// 30-bit halves, 4 products (sums of 2 LL <= 8 products of 60 bits fit 64 bits); MODE 2: anything else, 128-bit
// accumulation.
template <int LL, bool KEYS_STREAM, int MODE>
__device__ __forceinline__ void ks_inner_body(const u64* __restrict__ digits, long long digit_stride, const u64* const* __restrict__ keytab,
                                              int rot0, int rot_inc, u64* __restrict__ u, long long L1N, long long pos, long long it0,
                                              long long it1, const LimbConst& lc) {
    constexpr int NS = KEYS_STREAM ? 2 * LL : LL;   // streamed words per item
    constexpr int NST = KEYS_STREAM ? LL : 2 * LL;  // stationary words
    constexpr int SH = MODE == 0 ? 25 : 30;
    constexpr unsigned MASK = (1u << SH) - 1;
    u64 st[NST];
    if (KEYS_STREAM) {
#pragma unroll
        for (int j = 0; j < LL; j++) st[j] = digits[(long long)j * L1N + pos];
    } else {
        const u64* key = keytab[rot0];
#pragma unroll
        for (int k = 0; k < NST; k++) st[k] = key[(long long)k * L1N + pos];  // k = j*2 + comp
    }
    unsigned s0[NST], s1[NST];
    double sd[NST];  // MODE 3: the stationary words as balanced binary64 integers
#pragma unroll
    for (int k = 0; k < NST; k++) {
        if (MODE == 3) {
            sd[k] = residue_to_balanced_f64(st[k], (double)lc.q, (double)lc.half);
        } else {
            s0[k] = (unsigned)st[k] & MASK;
            s1[k] = (unsigned)(st[k] >> SH);
        }
    }
    u64 cur[NS], nxt[NS];
    auto load = [&](long long item, u64(&v)[NS]) {
        if (KEYS_STREAM) {
            const u64* key = keytab[rot0 + (int)item * rot_inc];
#pragma unroll
            for (int k = 0; k < NS; k++) v[k] = __ldcs(key + (long long)k * L1N + pos);  // k = j*2 + comp
        } else {
            const u64* d = digits + item * digit_stride + pos;
#pragma unroll
            for (int k = 0; k < NS; k++) v[k] = __ldcs(d + (long long)k * L1N);
        }
    };
    load(it0, cur);
    for (long long item = it0; item < it1; item++) {
        if (item + 1 < it1) load(item + 1, nxt);
        u64 out[2];
        if (MODE == 3) {
            // moduli below 2^50, at most eight digits: the products summed exactly in two binary64 words per component on the
            // FP64 pipe (acc2_fma), the integer pipe keeps only the final reduction
            static_assert(MODE != 3 || LL <= 8, "the two-word binary64 sum holds eight products");
            double ah[2] = {kAcc2Start, kAcc2Start}, al[2] = {0, 0};
#pragma unroll
            for (int j = 0; j < LL; j++)
#pragma unroll
                for (int c = 0; c < 2; c++)
                    acc2_fma(ah[c], al[c], residue_to_f64(KEYS_STREAM ? cur[2 * j + c] : cur[j]), sd[KEYS_STREAM ? j : 2 * j + c]);
#pragma unroll
            for (int c = 0; c < 2; c++) out[c] = acc2_reduce(acc2_high(ah[c]), acc2_low(al[c]), lc);
        } else if (MODE != 2) {
            u64 p00[2] = {0, 0}, p11[2] = {0, 0}, pm[2] = {0, 0};
#pragma unroll
            for (int j = 0; j < LL; j++)
#pragma unroll
                for (int c = 0; c < 2; c++) {
                    const int ks = KEYS_STREAM ? j : 2 * j + c;            // stationary word
                    const u64 sv = KEYS_STREAM ? cur[2 * j + c] : cur[j];  // streamed word
                    const unsigned b0 = (unsigned)sv & MASK, b1 = (unsigned)(sv >> SH);
                    p00[c] += (u64)s0[ks] * b0;
                    p11[c] += (u64)s1[ks] * b1;
                    if (MODE == 0) {
                        pm[c] += (u64)(s0[ks] + s1[ks]) * (b0 + b1);
                    } else {
                        pm[c] += (u64)s0[ks] * b1;
                        pm[c] += (u64)s1[ks] * b0;
                    }
                }
#pragma unroll
            for (int c = 0; c < 2; c++) {
                // value = p00 + cross * 2^SH + p11 * 2^(2 SH)
                const u64 cross = MODE == 0 ? pm[c] - p00[c] - p11[c] : pm[c];
                u64 lo = p00[c], hi = 0;
                const u64 c_lo = cross << SH, c_hi = cross >> (64 - SH);
                lo += c_lo;
                hi += c_hi + (lo < c_lo ? 1 : 0);
                const u64 d_lo = p11[c] << (2 * SH), d_hi = p11[c] >> (64 - 2 * SH);
                lo += d_lo;
                hi += d_hi + (lo < d_lo ? 1 : 0);
                out[c] = reduce128(hi, lo, lc);
            }
        } else {
            u64 h[2] = {0, 0}, l[2] = {0, 0};
#pragma unroll
            for (int j = 0; j < LL; j++)
#pragma unroll
                for (int c = 0; c < 2; c++) mac128(h[c], l[c], KEYS_STREAM ? st[j] : cur[j], KEYS_STREAM ? cur[2 * j + c] : st[2 * j + c]);
            out[0] = reduce128(h[0], l[0], lc);
            out[1] = reduce128(h[1], l[1], lc);
        }
        u64* o = u + item * 2 * L1N + pos;
        o[0] = out[0];
        o[L1N] = out[1];
#pragma unroll
        for (int k = 0; k < NS; k++) cur[k] = nxt[k];
    }
}

// blockIdx.z selects one of several independent batches of `nitems` items laid out one after the other (digits and u), batch
// z using rotation rot0 + z * rot_zinc: the giant steps of the lazy rotate-and-sum, each under its own key
template <int LL, bool KEYS_STREAM>
__global__ void __launch_bounds__(128) k_ks_inner_stream(const u64* __restrict__ digits, long long digit_stride,
                                                         const u64* const* __restrict__ keytab, int rot0, int rot_inc,
                                                         u64* __restrict__ u, int N, long long nitems, int items_per_cta,
                                                         const LimbConst* __restrict__ lt, int rot_zinc, int f64) {
    const long long L1N = (long long)(LL + 1) * N;
    const long long pos = (long long)blockIdx.x * 128 + threadIdx.x;  // i*N + x
    const LimbConst lc = lt[pos / N];
    rot0 += (int)blockIdx.z * rot_zinc;
    digits += (long long)blockIdx.z * nitems * digit_stride;
    u += (long long)blockIdx.z * nitems * 2 * L1N;
    const long long it0 = (long long)blockIdx.y * items_per_cta;
    const long long it1 = it0 + items_per_cta < nitems ? it0 + items_per_cta : nitems;
    if (it0 >= it1) return;
    // a CTA lies inside one limb, so the choice is uniform
    if (lc.q < (1ULL << 50) && f64) ks_inner_body<LL, KEYS_STREAM, 3>(digits, digit_stride, keytab, rot0, rot_inc, u, L1N, pos, it0, it1, lc);
    else if (lc.q < (1ULL << 50)) ks_inner_body<LL, KEYS_STREAM, 0>(digits, digit_stride, keytab, rot0, rot_inc, u, L1N, pos, it0, it1, lc);
    else if (lc.q < (1ULL << 60)) ks_inner_body<LL, KEYS_STREAM, 1>(digits, digit_stride, keytab, rot0, rot_inc, u, L1N, pos, it0, it1, lc);
    else ks_inner_body<LL, KEYS_STREAM, 2>(digits, digit_stride, keytab, rot0, rot_inc, u, L1N, pos, it0, it1, lc);
}

// lifted[poly][i][x] = centred lift of up[poly][x] (residue mod p, coefficient domain) reduced mod q_i.
// up is the special-prime limb inside u: poly = item*2 + comp lives at u + poly*(L+1)*N + L*N.
__global__ void __launch_bounds__(kThreads) k_moddown_lift(const u64* __restrict__ u, u64* __restrict__ lifted, int N,
                                                           int L, long long npoly, LimbTable lt) {
    const long long total = npoly * N;
    const u64 p = lt.c[L].q, half = lt.c[L].half;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const long long poly = idx / N;
        const int x = (int)(idx % N);
        const u64 v = u[poly * (L + 1) * N + (long long)L * N + x];
        const bool neg = v > half;
        const u64 mag = neg ? p - v : v;
        for (int i = 0; i < L; i++) {
            u64 r = barrett64(mag, lt.c[i]);
            lifted[(poly * L + i) * N + x] = (neg && r) ? lt.c[i].q - r : r;
        }
    }
}

// out[item][comp][i][t] = (u[item][comp][i][s] - lifted[item][comp][i][s]) * p^{-1}
//                         + (comp == 0 ? c0[item][i][s] : 0) + addend[item][comp][i][t],   s = galois source of t
// for the Galois element of rotation rot0 + item*rot_inc (rotation 0 = identity).  All arrays in the transform domain.
__global__ void __launch_bounds__(kThreads) k_moddown_combine(
    const u64* __restrict__ u, const u64* __restrict__ lifted, long long nitems, const unsigned* __restrict__ galois,
    int rot0, int rot_inc, const u64* __restrict__ c0, long long c0_stride, const u64* __restrict__ addend,
    long long addend_stride, u64* __restrict__ out0, u64* __restrict__ out1, long long out_stride, int N, int logN, int L,
    int tau, LimbTable lt) {
    const long long LN = (long long)L * N, L1N = (long long)(L + 1) * N;
    const long long total = nitems * 2 * LN;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const int t = (int)(idx % N);
        const int i = (int)((idx / N) % L);
        const int comp = (int)((idx / LN) % 2);
        const long long item = idx / (2 * LN);
        const unsigned k = galois[rot0 + (int)item * rot_inc];
        const int s = (k == 1u) ? t : galois_src(t, k, logN, tau);
        if (!HANN_CHECK_INDEX(s, N)) continue;
        const LimbConst& lc = lt.c[i];
        u64 a = u[(item * 2 + comp) * L1N + (long long)i * N + s];
        u64 b = lifted[((item * 2 + comp) * L + i) * N + s];
        u64 v = csub(shoup_mul(submod(a, b, lc.q), lc.pinv, lc.pinv_s, lc.q), lc.q);
        if (comp == 0 && c0) v = addmod(v, c0[item * c0_stride + (long long)i * N + s], lc.q);
        if (addend) v = addmod(v, addend[item * addend_stride + (long long)comp * LN + (long long)i * N + t], lc.q);
        u64* o = (comp == 0 ? out0 : out1) + item * out_stride + (long long)i * N + t;
        *o = v;
    }
}

// The same combine for rings of at least 256 points, without scattered global reads.  In bit-reversed order the
// automorphism maps every aligned chunk of 256 positions onto another aligned chunk (the top 8 bits of a position are
// the low 8 bits of its evaluation index, which an affine map modulo 2^logN keeps together), so a CTA loads the source
// chunk of u, lifted and c0 contiguously into shared memory and permutes there.
__global__ void __launch_bounds__(256) k_moddown_combine_chunk(
    const u64* __restrict__ u, const u64* __restrict__ lifted, const unsigned* __restrict__ galois, int rot0, int rot_inc,
    const u64* __restrict__ c0, long long c0_stride, const u64* __restrict__ addend, long long addend_stride,
    u64* __restrict__ out0, u64* __restrict__ out1, long long out_stride, int N, int logN, int L, int tau,
    const LimbConst* __restrict__ lt) {
    __shared__ u64 su[2][256], sl[2][256], sc[256];
    const long long LN = (long long)L * N, L1N = (long long)(L + 1) * N;
    const int chunks = N >> 8;
    const int chunk = blockIdx.x % chunks;
    const int i = (blockIdx.x / chunks) % L;
    const long long item = blockIdx.x / ((long long)chunks * L);
    const unsigned k = galois[rot0 + (int)item * rot_inc];
    const int t = (chunk << 8) + threadIdx.x;
    const int s = (k == 1u) ? t : galois_src(t, k, logN, tau);
    const int src_chunk = ((k == 1u) ? (chunk << 8) : galois_src(chunk << 8, k, logN, tau)) & ~255;
    // the source chunk must lie inside the polynomial (uniform over the CTA, so leaving here cannot split it at the
    // barrier); that the source of every t lies in that chunk is checked per thread below, where only the store is skipped
    if (!HANN_CHECK_INDEX(src_chunk + 255, N)) return;
    const bool in_chunk = HANN_CHECK_INDEX((s & ~255) - src_chunk, 1);
    const LimbConst lc = lt[i];
#pragma unroll
    for (int comp = 0; comp < 2; comp++) {
        su[comp][threadIdx.x] = u[(item * 2 + comp) * L1N + (long long)i * N + src_chunk + threadIdx.x];
        sl[comp][threadIdx.x] = lifted[((item * 2 + comp) * L + i) * N + src_chunk + threadIdx.x];
    }
    if (c0) sc[threadIdx.x] = c0[item * c0_stride + (long long)i * N + src_chunk + threadIdx.x];
    __syncthreads();
    const int ls = s & 255;
#pragma unroll
    for (int comp = 0; comp < 2; comp++) {
        u64 v = csub(shoup_mul(submod(su[comp][ls], sl[comp][ls], lc.q), lc.pinv, lc.pinv_s, lc.q), lc.q);
        if (comp == 0 && c0) v = addmod(v, sc[ls], lc.q);
        if (addend) v = addmod(v, addend[item * addend_stride + (long long)comp * LN + (long long)i * N + t], lc.q);
        u64* o = (comp == 0 ? out0 : out1) + item * out_stride + (long long)i * N + t;
        if (in_chunk) *o = v;
    }
}

// ---- lazy giant steps: the key products of G-1 differently rotated terms are summed before ONE ModDown -------------------
// Items are laid out giant step after giant step: item (g, blk) = (g - 1) * nblk + blk, g = 1 .. G-1; the keys are stored
// pre-permuted, so the product u of item (g, blk) still awaits the automorphism of rotation g * B.

// up[blk][comp][t] = sum_g u[(g, blk)][comp][limb L][source_g(t)] mod p      (special-prime limb of the summed products)
__global__ void __launch_bounds__(kThreads) k_giant_sum_p(const u64* __restrict__ u, u64* __restrict__ up, long long nblk, int G, int B,
                                                          const unsigned* __restrict__ galois, int N, int logN, int L, int tau,
                                                          LimbTable lt) {
    const long long L1N = (long long)(L + 1) * N, total = nblk * 2 * N;
    const u64 p = lt.c[L].q;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const int t = (int)(idx % N);
        const int comp = (int)((idx / N) % 2);
        const long long blk = idx / (2 * (long long)N);
        u64 acc = 0;
        for (int g = 1; g < G; g++) {
            const int s = galois_src(t, galois[g * B], logN, tau);
            if (!HANN_CHECK_INDEX(s, N)) continue;
            acc = addmod(acc, u[((((long long)(g - 1) * nblk + blk) * 2 + comp) * L1N) + (long long)L * N + s], p);
        }
        up[idx] = acc;
    }
}

// lifted[poly][i][x] = centred lift of up[poly][x] (residue mod p, coefficient domain, polynomials N words apart) mod q_i
__global__ void __launch_bounds__(kThreads) k_lift_p(const u64* __restrict__ up, u64* __restrict__ lifted, int N, int L, long long npoly,
                                                     LimbTable lt) {
    const long long total = npoly * N;
    const u64 p = lt.c[L].q, half = lt.c[L].half;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const long long poly = idx / N;
        const int x = (int)(idx % N);
        const u64 v = up[idx];
        const bool neg = v > half;
        const u64 mag = neg ? p - v : v;
        for (int i = 0; i < L; i++) {
            u64 r = barrett64(mag, lt.c[i]);
            lifted[(poly * L + i) * N + x] = (neg && r) ? lt.c[i].q - r : r;
        }
    }
}

// score[blk][comp][i][t] = (sum_g u[(g, blk)][comp][i][source_g(t)] - lifted[blk][comp][i][t]) * p^{-1}
//                          + inner[blk][0][comp][i][t] + (comp == 0 ? sum_g inner[blk][g][0][i][source_g(t)] : 0)
// (every aligned chunk of 256 positions maps onto one chunk under an automorphism, so the gathered reads of a CTA stay inside
// a few cache lines)
__global__ void __launch_bounds__(kThreads) k_giant_combine(const u64* __restrict__ u, const u64* __restrict__ lifted,
                                                            const u64* __restrict__ inner, u64* __restrict__ score, long long nblk, int G,
                                                            int B, const unsigned* __restrict__ galois, int N, int logN, int L, int tau,
                                                            LimbTable lt) {
    const long long LN = (long long)L * N, L1N = (long long)(L + 1) * N, ctw = 2 * LN;
    const long long total = nblk * LN;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const int t = (int)(idx % N);
        const int i = (int)((idx / N) % L);
        const long long blk = idx / LN;
        const LimbConst& lc = lt.c[i];
        u64 a0 = 0, a1 = 0, c0 = inner[(blk * G) * ctw + (long long)i * N + t];
        for (int g = 1; g < G; g++) {
            const int s = galois_src(t, galois[g * B], logN, tau);
            if (!HANN_CHECK_INDEX(s, N)) continue;
            const u64* ug = u + (((long long)(g - 1) * nblk + blk) * 2) * L1N + (long long)i * N + s;
            a0 = addmod(a0, ug[0], lc.q);
            a1 = addmod(a1, ug[L1N], lc.q);
            c0 = addmod(c0, inner[(blk * G + g) * ctw + (long long)i * N + s], lc.q);
        }
        const u64* lf = lifted + (blk * 2 * L + i) * N + t;
        const u64 v0 = csub(shoup_mul(submod(a0, lf[0], lc.q), lc.pinv, lc.pinv_s, lc.q), lc.q);
        const u64 v1 = csub(shoup_mul(submod(a1, lf[LN], lc.q), lc.pinv, lc.pinv_s, lc.q), lc.q);
        score[blk * ctw + (long long)i * N + t] = addmod(v0, c0, lc.q);
        score[blk * ctw + LN + (long long)i * N + t] = addmod(v1, inner[(blk * G) * ctw + LN + (long long)i * N + t], lc.q);
    }
}

// dst[poly][t] = src[poly][galois source of t]   (transform domain automorphism X -> X^k)
__global__ void __launch_bounds__(kThreads) k_permute(const u64* __restrict__ src, u64* __restrict__ dst, long long npoly,
                                                      unsigned k, int N, int logN, int tau) {
    const long long total = npoly * N;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const long long poly = idx / N;
        const int t = (int)(idx % N);
        const int sidx = galois_src(t, k, logN, tau);
        if (!HANN_CHECK_INDEX(sidx, N)) continue;
        dst[idx] = src[poly * N + sidx];
    }
}

// ------------------------------------------------------------------------------------------ client-side helpers

// out[l][x] = residue of the small signed coefficient v[x] modulo limb first + l
__global__ void __launch_bounds__(kThreads) k_lift_i8(const int8_t* __restrict__ v, u64* __restrict__ out, int N,
                                                      int nlimbs, LimbTable lt) {
    const long long total = (long long)nlimbs * N;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const int l = (int)(idx / N), x = (int)(idx % N);
        int s = v[x];
        out[idx] = s >= 0 ? (u64)s : lt.c[l].q - (u64)(-s);
    }
}

// out[p][x] = a[p][x] * b[(p % bperiod)][x] mod limb(p)
__global__ void __launch_bounds__(kThreads) k_mul(const u64* __restrict__ a, const u64* __restrict__ b, int bperiod,
                                                  u64* __restrict__ out, long long npoly, int N, LimbMap lm, LimbTable lt) {
    const long long total = npoly * N;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const long long p = idx / N;
        const int x = (int)(idx % N);
        const LimbConst& lc = lt.c[lm.limb[p % lm.period]];
        out[idx] = mulmod(a[idx], b[(p % bperiod) * N + x], lc);
    }
}

// out[p][x] = a[p][x] + b[p][x] mod limb(p)
__global__ void __launch_bounds__(kThreads) k_add(const u64* __restrict__ a, const u64* __restrict__ b,
                                                  u64* __restrict__ out, long long npoly, int N, LimbMap lm, LimbTable lt) {
    const long long total = npoly * N;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const long long p = idx / N;
        out[idx] = addmod(a[idx], b[idx], lt.c[lm.limb[p % lm.period]].q);
    }
}

// evaluation key finish, coefficient domain: b[j][i][x] = -as[j][i][x] + e[j][x] + (i == j ? (p mod q_j) * s'[x] : 0)
__global__ void __launch_bounds__(kThreads) k_evk_finish(const u64* __restrict__ as, const int8_t* __restrict__ e,
                                                         const int8_t* __restrict__ sprime, u64* __restrict__ b_out,
                                                         int N, int L, LimbTable lt) {
    const long long total = (long long)L * (L + 1) * N;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const int x = (int)(idx % N);
        const int i = (int)((idx / N) % (L + 1));
        const int j = (int)(idx / ((long long)N * (L + 1)));
        const LimbConst& lc = lt.c[i];
        u64 v = as[idx] ? lc.q - as[idx] : 0;
        v = addmod(v, reduce_signed((i64)e[(long long)j * N + x], lc), lc.q);
        if (i == j) {
            int sp = sprime[x];
            u64 f = lc.pmod;  // p mod q_j
            if (sp > 0) v = addmod(v, f, lc.q);
            else if (sp < 0) v = submod(v, f, lc.q);
        }
        b_out[idx] = v;
    }
}

// relinearisation key finish, coefficient domain: b[j][i][x] = -as[j][i][x] + e[j][x] + (i == j ? (p mod q_j) * s2[j][x] : 0),
// s2[i][x] the residues of s^2 modulo limb i
__global__ void __launch_bounds__(kThreads) k_rlk_finish(const u64* __restrict__ as, const int8_t* __restrict__ e,
                                                         const u64* __restrict__ s2, u64* __restrict__ b_out, int N, int L,
                                                         LimbTable lt) {
    const long long total = (long long)L * (L + 1) * N;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const int x = (int)(idx % N);
        const int i = (int)((idx / N) % (L + 1));
        const int j = (int)(idx / ((long long)N * (L + 1)));
        const LimbConst& lc = lt.c[i];
        u64 v = as[idx] ? lc.q - as[idx] : 0;
        v = addmod(v, reduce_signed((i64)e[(long long)j * N + x], lc), lc.q);
        if (i == j) v = addmod(v, mulmod(lc.pmod, s2[(long long)i * N + x], lc), lc.q);
        b_out[idx] = v;
    }
}

// block encryption finish, transform domain: c0[r][l][t] = pt[r][l][t] - as[r][l][t] + ehat[r][l][t]; pt in its stored
// form [r][l][N/2] (position t >= N/2 is the mirror image of position N - 1 - t)
__global__ void __launch_bounds__(kThreads) k_encrypt_block_finish(const u64* __restrict__ pt, const u64* __restrict__ as,
                                                                   const u64* __restrict__ ehat, u64* __restrict__ ct, int N, int L,
                                                                   long long npt, LimbTable lt) {
    const long long LN = (long long)L * N, total = npt * LN;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const long long r = idx / LN, rem = idx % LN;
        const u64 q = lt.c[(int)(rem / N)].q;
        const int l = (int)(rem / N), t = (int)(rem % N), n = N >> 1;
        const u64 m = pt[(r * L + l) * n + (t < n ? t : N - 1 - t)];
        ct[r * 2 * LN + rem] = addmod(submod(m, as[idx], q), ehat[idx], q);
    }
}

// the uniform half of a seed-compressed ciphertext: a[l][x] = h(seed, stream, l*N + x) mod q_l, h the 64-bit counter hash
// mix(mix(mix(seed + M1) ^ (stream * M2)) + ctr * M1), mix(x): x ^= x >> 32; x *= M1; x ^= x >> 29; x *= M2; x ^= x >> 32
__device__ __forceinline__ u64 mix64(u64 x) {
    x ^= x >> 32;
    x *= 0x9E3779B97F4A7C15ULL;
    x ^= x >> 29;
    x *= 0xBB67AE8584CAA73BULL;
    x ^= x >> 32;
    return x;
}
__global__ void __launch_bounds__(kThreads) k_expand_uniform(u64* __restrict__ a, u64 seed, u64 stream, int N, int L, LimbTable lt) {
    const long long total = (long long)L * N;
    const u64 b = mix64(mix64(seed + 0x9E3779B97F4A7C15ULL) ^ (stream * 0xBB67AE8584CAA73BULL));
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads)
        a[idx] = barrett64(mix64(b + (u64)idx * 0x9E3779B97F4A7C15ULL), lt.c[(int)(idx / N)]);
}

// the same generator over the L+1 moduli of an evaluation key: a[j][i][x] = h(seed, stream, ctr0 + (j (L+1) + i) N + x) mod m_i
__global__ void __launch_bounds__(kThreads) k_expand_uniform_qp(u64* __restrict__ a, u64 seed, u64 stream, u64 ctr0, int N, int L, LimbTable lt) {
    const long long total = (long long)L * (L + 1) * N;
    const u64 b = mix64(mix64(seed + 0x9E3779B97F4A7C15ULL) ^ (stream * 0xBB67AE8584CAA73BULL));
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads)
        a[idx] = barrett64(mix64(b + (ctr0 + (u64)idx) * 0x9E3779B97F4A7C15ULL), lt.c[(int)((idx / N) % (L + 1))]);
}

// symmetric encryption finish, coefficient domain: c0[l][x] = -as[l][x] + e[x] + m[l][x]
__global__ void __launch_bounds__(kThreads) k_encrypt_finish(const u64* __restrict__ as, const int8_t* __restrict__ e,
                                                             const u64* __restrict__ m, u64* __restrict__ c0, int N, int L,
                                                             LimbTable lt) {
    const long long total = (long long)L * N;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const int x = (int)(idx % N);
        const int l = (int)(idx / N);
        const LimbConst& lc = lt.c[l];
        u64 v = as[idx] ? lc.q - as[idx] : 0;
        v = addmod(v, reduce_signed((i64)e[x], lc), lc.q);
        c0[idx] = addmod(v, m[idx], lc.q);
    }
}

}  // namespace

// out[poly][l][t] = a[poly][l][t] * ma_l (+ b[poly][l][t] * mb_l) (+ k_l on the first polynomial of every ciphertext), mod q_l:
// the additions, negations, integer multiples and added constants of a leveled circuit, in the transform domain (a constant
// polynomial transforms to its constant in every position).  Ciphertexts of `limbs` limbs: polynomial pairs.
struct LinearArgs {
    u64 ma[HANN_MAXL1], mb[HANN_MAXL1], k[HANN_MAXL1];
};
// b_period > 0: b has only b_period words (one ciphertext) and is used for every ciphertext of a.
__global__ void __launch_bounds__(kThreads) k_linear(const u64* __restrict__ a, const u64* __restrict__ b, u64* __restrict__ out,
                                                     long long npoly, int limbs, int N, long long b_period, LinearArgs la, LimbTable lt) {
    const long long total = npoly * limbs * N;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const int l = (int)((idx / N) % limbs);
        const long long poly = idx / ((long long)limbs * N);
        const LimbConst& lc = lt.c[l];
        u64 v = la.ma[l] == 1 ? a[idx] : mulmod(a[idx], la.ma[l], lc);
        if (b) {
            const u64 bv = b[b_period > 0 ? idx % b_period : idx];
            v = addmod(v, la.mb[l] == 1 ? bv : mulmod(bv, la.mb[l], lc), lc.q);
        }
        if ((poly & 1) == 0 && la.k[l]) v = addmod(v, la.k[l], lc.q);
        out[idx] = v;
    }
}

// degree-2 product of `count` independent ciphertext pairs: d[i] = (a0 b0, a0 b1 + a1 b0, a1 b1), all [.][limbs][N], elementwise
// in the transform domain
__global__ void __launch_bounds__(kThreads) k_mul_ct(const u64* __restrict__ a, const u64* __restrict__ b, u64* __restrict__ d,
                                                     long long count, int limbs, int N, LimbTable lt) {
    const long long LN = (long long)limbs * N, total = count * LN;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const long long i = idx / LN, pos = idx % LN;
        const LimbConst& lc = lt.c[(int)(pos / N)];
        const u64 a0 = a[i * 2 * LN + pos], a1 = a[i * 2 * LN + LN + pos], b0 = b[i * 2 * LN + pos], b1 = b[i * 2 * LN + LN + pos];
        u64* o = d + i * 3 * LN + pos;
        o[0] = mulmod(a0, b0, lc);
        o[LN] = addmod(mulmod(a0, b1, lc), mulmod(a1, b0, lc), lc.q);
        o[2 * LN] = mulmod(a1, b1, lc);
    }
}

// ---- workspace guards (debugging aid): 32 words behind a sub-buffer hold a pattern derived from their own address
__global__ void k_guard_fill(u64* guard) { guard[threadIdx.x] = 0xC0DEC0DEC0DEC0DEULL ^ (u64)(uintptr_t)(guard + threadIdx.x); }
__global__ void k_guard_verify(u64* const* guards, long long count, unsigned long long* damaged) {
    const long long gi = blockIdx.x;
    if (gi >= count) return;
    const u64* g = guards[gi];
    const bool bad = g[threadIdx.x] != (0xC0DEC0DEC0DEC0DEULL ^ (u64)(uintptr_t)(g + threadIdx.x));
    if (__any_sync(0xffffffffu, bad) && threadIdx.x == 0) {
        atomicAdd(damaged, 1ULL);
        atomicMin(damaged + 1, (unsigned long long)gi);   // the first damaged guard, in the order they were carved
    }
}

HANN_DEBUG_DEFINE_BIND(debug_bind_keyswitch)

int check_launch(hann_ctx* c, const char* what) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        c->err = std::string(what) + ": " + cudaGetErrorString(e);
        return HANN_ECUDA;
    }
    return HANN_OK;
}

// out = ma * a + mb * b + k (k on the c0 of every ciphertext); ma, mb, k signed integers below 2^62 in magnitude, reduced per limb
// here; b may be null.  npoly polynomials of c->L limbs; b_period > 0: b is ONE ciphertext (b_period words) added to every one of a.
int launch_mul_ct(hann_ctx* c, const u64* a, const u64* b, int64_t count, u64* d) {
    {
        KProf kp(c, KC_MAC);
        k_mul_ct<<<grid_for(count * c->L * c->N), kThreads, 0, c->stream>>>(a, b, d, count, c->L, c->N, c->lt);
    }
    return check_launch(c, "mul_ct");
}

int launch_linear(hann_ctx* c, const u64* a, long long ma, const u64* b, long long mb, long long k, int64_t npoly, u64* out,
                  int64_t b_period) {
    LinearArgs la = {};
    auto residue = [](long long v, u64 q) { return v >= 0 ? (u64)v % q : (q - ((u64)(-v) % q)) % q; };
    for (int l = 0; l < c->L; l++) {
        la.ma[l] = residue(ma, c->mod[l]);
        la.mb[l] = residue(mb, c->mod[l]);
        la.k[l] = residue(k, c->mod[l]);
    }
    {
        KProf kp(c, KC_OTHER);
        k_linear<<<grid_for(npoly * c->L * c->N), kThreads, 0, c->stream>>>(a, b, out, npoly, c->L, c->N, b_period, la, c->lt);
    }
    return check_launch(c, "linear");
}

int launch_guard_fill(hann_ctx* c, u64* guard) {
    k_guard_fill<<<1, 32, 0, c->stream>>>(guard);
    return check_launch(c, "guard_fill");
}

int launch_guard_verify(hann_ctx* c, u64* const* guards, int64_t count, unsigned long long* damaged) {
    k_guard_verify<<<(unsigned)count, 32, 0, c->stream>>>(guards, count, damaged);
    return check_launch(c, "guard_verify");
}

int launch_lift_digits(hann_ctx* c, const u64* src, int64_t src_stride, int64_t nitems, u64* digits) {
    {
        KProf kp(c, KC_LIFT_DIGITS);
        k_lift_digits<<<grid_for(nitems * c->L * c->N), kThreads, 0, c->stream>>>(src, src_stride, digits, c->N, c->L, nitems, c->lt);
    }
    return check_launch(c, "lift_digits");
}

template <int LL>
void launch_ks_inner_stream(hann_ctx* c, const u64* digits, int64_t digit_stride, int rot0, int rot_inc, int64_t nitems, u64* u,
                            int nz = 1, int rot_zinc = 0) {
    const long long L1N = (long long)(LL + 1) * c->N;
    const int tiles = (int)(L1N / 128);
    int split = 1;
    while ((long long)tiles * split * nz < 148 * 8 && split < nitems) split *= 2;
    const int per = (int)((nitems + split - 1) / split);
    split = (int)((nitems + per - 1) / per);
    KProf kp(c, digit_stride == 0 && nitems > 1 ? KC_KS_INNER_KEYS : KC_KS_INNER);  // streamed keys timed on their own
    if (digit_stride == 0)
        k_ks_inner_stream<LL, true><<<dim3(tiles, split, nz), 128, 0, c->stream>>>(digits, 0, c->keytab_dev, rot0, rot_inc, u, c->N, nitems,
                                                                                per, c->lt_dev, rot_zinc, c->mac_f64);
    else
        k_ks_inner_stream<LL, false><<<dim3(tiles, split, nz), 128, 0, c->stream>>>(digits, digit_stride, c->keytab_dev, rot0, rot_inc, u,
                                                                                 c->N, nitems, per, c->lt_dev, rot_zinc, c->mac_f64);
}

int launch_ks_inner(hann_ctx* c, const u64* digits, int64_t digit_stride, int rot0, int rot_inc, int64_t nitems, u64* u) {
    // the streaming kernel covers the two shapes the path produces: one digit set under many keys (digit_stride == 0)
    // and many digit sets under one key (rot_inc == 0)
    if (c->L <= 4 && c->N >= 128 && (digit_stride == 0 || rot_inc == 0)) {
        switch (c->L) {
            case 1: launch_ks_inner_stream<1>(c, digits, digit_stride, rot0, rot_inc, nitems, u); break;
            case 2: launch_ks_inner_stream<2>(c, digits, digit_stride, rot0, rot_inc, nitems, u); break;
            case 3: launch_ks_inner_stream<3>(c, digits, digit_stride, rot0, rot_inc, nitems, u); break;
            default: launch_ks_inner_stream<4>(c, digits, digit_stride, rot0, rot_inc, nitems, u); break;
        }
        return check_launch(c, "ks_inner_stream");
    }
    {
        KProf kp(c, KC_KS_INNER);
        k_ks_inner<<<grid_for(nitems * (c->L + 1) * c->N), kThreads, 0, c->stream>>>(digits, digit_stride, c->keytab_dev, rot0, rot_inc, u,
                                                                                   c->N, c->L, nitems, c->lt, c->mac_f64);
    }
    return check_launch(c, "ks_inner");
}

// nz batches of `per_z` digit sets each (digits and u laid out batch after batch); every item of batch z is multiplied with
// the key of rotation rot0 + z * rot_zinc
int launch_ks_inner_batches(hann_ctx* c, const u64* digits, int64_t digit_stride, int rot0, int rot_zinc, int nz, int64_t per_z, u64* u) {
    if (nz <= 0 || per_z <= 0) return HANN_OK;
    if (c->L <= 4 && c->N >= 128 && digit_stride != 0) {
        switch (c->L) {
            case 1: launch_ks_inner_stream<1>(c, digits, digit_stride, rot0, 0, per_z, u, nz, rot_zinc); break;
            case 2: launch_ks_inner_stream<2>(c, digits, digit_stride, rot0, 0, per_z, u, nz, rot_zinc); break;
            case 3: launch_ks_inner_stream<3>(c, digits, digit_stride, rot0, 0, per_z, u, nz, rot_zinc); break;
            default: launch_ks_inner_stream<4>(c, digits, digit_stride, rot0, 0, per_z, u, nz, rot_zinc); break;
        }
        return check_launch(c, "ks_inner_stream");
    }
    for (int z = 0; z < nz; z++) {
        const int r = launch_ks_inner(c, digits + z * per_z * digit_stride, digit_stride, rot0 + z * rot_zinc, 0, per_z,
                                      u + z * per_z * 2 * (int64_t)(c->L + 1) * c->N);
        if (r != HANN_OK) return r;
    }
    return HANN_OK;
}

int launch_giant_sum_p(hann_ctx* c, const u64* u, int64_t nblk, u64* up) {
    {
        KProf kp(c, KC_PERMUTE);
        k_giant_sum_p<<<grid_for(nblk * 2 * c->N), kThreads, 0, c->stream>>>(u, up, nblk, c->G, c->B, c->galois_dev, c->N, c->logN, c->L,
                                                                           c->ntt_tau, c->lt);
    }
    return check_launch(c, "giant_sum_p");
}

int launch_lift_p(hann_ctx* c, const u64* up, int64_t npoly, u64* lifted) {
    {
        KProf kp(c, KC_MODDOWN_LIFT);
        k_lift_p<<<grid_for(npoly * c->N), kThreads, 0, c->stream>>>(up, lifted, c->N, c->L, npoly, c->lt);
    }
    return check_launch(c, "lift_p");
}

int launch_giant_combine(hann_ctx* c, const u64* u, const u64* lifted, const u64* inner, int64_t nblk, u64* score) {
    {
        KProf kp(c, KC_MODDOWN_COMBINE);
        k_giant_combine<<<grid_for(nblk * c->L * c->N, kThreads, 148 * 32), kThreads, 0, c->stream>>>(
            u, lifted, inner, score, nblk, c->G, c->B, c->galois_dev, c->N, c->logN, c->L, c->ntt_tau, c->lt);
    }
    return check_launch(c, "giant_combine");
}

int launch_moddown_lift(hann_ctx* c, const u64* u, int64_t npoly, u64* lifted) {
    {
        KProf kp(c, KC_MODDOWN_LIFT);
        k_moddown_lift<<<grid_for(npoly * c->N), kThreads, 0, c->stream>>>(u, lifted, c->N, c->L, npoly, c->lt);
    }
    return check_launch(c, "moddown_lift");
}

int launch_moddown_combine(hann_ctx* c, const u64* u, const u64* lifted, int64_t nitems, int rot0, int rot_inc, const u64* c0,
                           int64_t c0_stride, const u64* addend, int64_t addend_stride, u64* out0, u64* out1,
                           int64_t out_stride) {
    if (c->N >= 256) {
        const long long ctas = nitems * c->L * (c->N >> 8);
        KProf kp(c, KC_MODDOWN_COMBINE);
        k_moddown_combine_chunk<<<(unsigned)ctas, 256, 0, c->stream>>>(u, lifted, c->galois_dev, rot0, rot_inc, c0, c0_stride, addend,
                                                                     addend_stride, out0, out1, out_stride, c->N, c->logN, c->L,
                                                                     c->ntt_tau, c->lt_dev);
        return check_launch(c, "moddown_combine_chunk");
    }
    {
        KProf kp(c, KC_MODDOWN_COMBINE);
        k_moddown_combine<<<grid_for(nitems * 2 * c->L * c->N), kThreads, 0, c->stream>>>(
            u, lifted, nitems, c->galois_dev, rot0, rot_inc, c0, c0_stride, addend, addend_stride, out0, out1, out_stride, c->N,
            c->logN, c->L, c->ntt_tau, c->lt);
    }
    return check_launch(c, "moddown_combine");
}

// ---- output compaction: rescale by the last ciphertext prime ---------------------------------------------------------
// lifted[poly][i][x] = centred lift of t[poly][x] (residue mod q_{L-1}, coefficient domain) reduced mod q_i, i < keep
__global__ void __launch_bounds__(kThreads) k_rescale_lift(const u64* __restrict__ t, u64* __restrict__ lifted, int N, int L,
                                                           int keep, long long npoly, LimbTable lt) {
    const long long total = npoly * N;
    const u64 ql = lt.c[L - 1].q, half = lt.c[L - 1].half;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const long long poly = idx / N;
        const int x = (int)(idx % N);
        const u64 v = t[idx];
        const bool neg = v > half;
        const u64 mag = neg ? ql - v : v;
        for (int i = 0; i < keep; i++) {
            u64 r = barrett64(mag, lt.c[i]);
            lifted[(poly * keep + i) * N + x] = (neg && r) ? lt.c[i].q - r : r;
        }
    }
}

struct RescaleConst {
    u64 w[HANN_MAXL1], ws[HANN_MAXL1];  // q_{L-1}^{-1} mod q_i and its Shoup companion
};

// out[poly][i][x] = (src[poly][i][x] - lifted[poly][i][x]) * q_{L-1}^{-1} mod q_i; src polynomials have L limbs, out keep
__global__ void __launch_bounds__(kThreads) k_rescale_combine(const u64* __restrict__ src, const u64* __restrict__ lifted,
                                                              u64* __restrict__ out, int N, int L, int keep, long long npoly,
                                                              LimbTable lt, RescaleConst rc) {
    const long long total = npoly * keep * N;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const int x = (int)(idx % N);
        const int i = (int)((idx / N) % keep);
        const long long poly = idx / ((long long)keep * N);
        const u64 q = lt.c[i].q;
        const u64 d = submod(src[(poly * L + i) * N + x], lifted[idx], q);
        out[idx] = csub(shoup_mul(d, rc.w[i], rc.ws[i], q), q);
    }
}

int launch_rescale_lift(hann_ctx* c, const u64* t, int64_t npoly, int keep, u64* lifted) {
    {
        KProf kp(c, KC_OTHER);
        k_rescale_lift<<<grid_for(npoly * c->N), kThreads, 0, c->stream>>>(t, lifted, c->N, c->L, keep, npoly, c->lt);
    }
    return check_launch(c, "rescale_lift");
}

int launch_rescale_combine(hann_ctx* c, const u64* src, const u64* lifted, int64_t npoly, int keep, u64* out) {
    RescaleConst rc = {};
    const u64 ql = c->mod[c->L - 1];
    for (int i = 0; i < keep; i++) {
        rc.w[i] = hm::invmod(ql % c->mod[i], c->mod[i]);
        rc.ws[i] = hm::shoup(rc.w[i], c->mod[i]);
    }
    {
        KProf kp(c, KC_OTHER);
        k_rescale_combine<<<grid_for(npoly * keep * c->N), kThreads, 0, c->stream>>>(src, lifted, out, c->N, c->L, keep, npoly, c->lt, rc);
    }
    return check_launch(c, "rescale_combine");
}

int launch_permute(hann_ctx* c, const u64* src, u64* dst, int64_t npoly, unsigned k) {
    {
        KProf kp(c, KC_PERMUTE);
        k_permute<<<grid_for(npoly * c->N), kThreads, 0, c->stream>>>(src, dst, npoly, k, c->N, c->logN, c->ntt_tau);
    }
    return check_launch(c, "permute");
}

int launch_lift_i8(hann_ctx* c, const int8_t* v, int nlimbs, u64* out) {
    {
        KProf kp(c, KC_OTHER);
        k_lift_i8<<<grid_for((int64_t)nlimbs * c->N), kThreads, 0, c->stream>>>(v, out, c->N, nlimbs, c->lt);
    }
    return check_launch(c, "lift_i8");
}

int launch_mul(hann_ctx* c, const u64* a, const u64* b, int bperiod, u64* out, int64_t npoly, const LimbMap& lm) {
    {
        KProf kp(c, KC_OTHER);
        k_mul<<<grid_for(npoly * c->N), kThreads, 0, c->stream>>>(a, b, bperiod, out, npoly, c->N, lm, c->lt);
    }
    return check_launch(c, "mul");
}

int launch_add(hann_ctx* c, const u64* a, const u64* b, u64* out, int64_t npoly, const LimbMap& lm) {
    {
        KProf kp(c, KC_OTHER);
        k_add<<<grid_for(npoly * c->N), kThreads, 0, c->stream>>>(a, b, out, npoly, c->N, lm, c->lt);
    }
    return check_launch(c, "add");
}

int launch_evk_finish(hann_ctx* c, const u64* as_coeff, const int8_t* e, const int8_t* sprime, u64* b_out) {
    {
        KProf kp(c, KC_OTHER);
        k_evk_finish<<<grid_for((int64_t)c->L * (c->L + 1) * c->N), kThreads, 0, c->stream>>>(as_coeff, e, sprime, b_out, c->N, c->L, c->lt);
    }
    return check_launch(c, "evk_finish");
}

int launch_rlk_finish(hann_ctx* c, const u64* as_coeff, const int8_t* e, const u64* s2, u64* b_out) {
    {
        KProf kp(c, KC_OTHER);
        k_rlk_finish<<<grid_for((int64_t)c->L * (c->L + 1) * c->N), kThreads, 0, c->stream>>>(as_coeff, e, s2, b_out, c->N, c->L, c->lt);
    }
    return check_launch(c, "rlk_finish");
}

// rows x width words, source and destination rows pitch words apart, copied by the SMs: a cudaMemcpy between device
// buffers may be scheduled on a copy engine behind queued host transfers, which would stall the compute stream of
// hann_score_level_host until all of a level's rows have arrived
namespace {
__global__ void __launch_bounds__(kThreads) k_copy2d(u64* __restrict__ dst, long long dst_pitch, const u64* __restrict__ src,
                                                     long long src_pitch, long long width, long long rows) {
    const long long total = rows * width;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const long long r = idx / width, x = idx % width;
        dst[r * dst_pitch + x] = src[r * src_pitch + x];
    }
}
}  // namespace
int launch_copy2d(hann_ctx* c, u64* dst, int64_t dst_pitch, const u64* src, int64_t src_pitch, int64_t width, int64_t rows) {
    if (width <= 0 || rows <= 0) return HANN_OK;
    k_copy2d<<<grid_for(width * rows), kThreads, 0, c->stream>>>(dst, dst_pitch, src, src_pitch, width, rows);
    return check_launch(c, "copy2d");
}

int launch_encrypt_block_finish(hann_ctx* c, const u64* pt, const u64* as, const u64* ehat, u64* ct, int64_t npt) {
    {
        KProf kp(c, KC_OTHER);
        k_encrypt_block_finish<<<grid_for(npt * c->L * c->N), kThreads, 0, c->stream>>>(pt, as, ehat, ct, c->N, c->L, npt, c->lt);
    }
    return check_launch(c, "encrypt_block_finish");
}

int launch_expand_uniform(hann_ctx* c, u64 seed, u64 stream, u64* a) {
    {
        KProf kp(c, KC_OTHER);
        k_expand_uniform<<<grid_for((int64_t)c->L * c->N), kThreads, 0, c->stream>>>(a, seed, stream, c->N, c->L, c->lt);
    }
    return check_launch(c, "expand_uniform");
}

int launch_expand_uniform_qp(hann_ctx* c, u64 seed, u64 stream, u64 ctr0, u64* a) {
    {
        KProf kp(c, KC_OTHER);
        k_expand_uniform_qp<<<grid_for((int64_t)c->L * (c->L + 1) * c->N), kThreads, 0, c->stream>>>(a, seed, stream, ctr0, c->N, c->L, c->lt);
    }
    return check_launch(c, "expand_uniform_qp");
}

int launch_encrypt_finish(hann_ctx* c, const u64* as_coeff, const int8_t* e, const u64* m, u64* c0_out) {
    {
        KProf kp(c, KC_OTHER);
        k_encrypt_finish<<<grid_for((int64_t)c->L * c->N), kThreads, 0, c->stream>>>(as_coeff, e, m, c0_out, c->N, c->L, c->lt);
    }
    return check_launch(c, "encrypt_finish");
}
