// Multiply-accumulate kernels: ciphertext x plaintext (the hot path's inner loop, Sec. 3.4), its paired form for two
// queries, and ciphertext x ciphertext for an encrypted database.  Ciphertext polynomials are [.][limb][N] arrays of 64-bit
// residues in [0, q), in the transform domain.  A PLAINTEXT is stored as [limb][N/2]: the encoding of a real slot vector
// is fixed by X -> 1/X, so position t and position N - 1 - t of its transform hold the same value, and every stored word
// serves both positions (a thread multiplies it with the baby-step words of both and produces both outputs).
#include <cuda.h>

#include "internal.h"
#include "bulkcopy.cuh"

namespace {

constexpr int kThreads = 256;

// ------------------------------------------------------------------------------------------ multiply-accumulate

// inner[blk][g][comp][l][x] = sum_b pt[blk][g][b][l][x] * baby[b][comp][l][x] mod q_l.
//
// Generic kernel (any modulus): one thread owns one (l, x) position for a range of (blk, g) pairs; products are
// accumulated in 128 bits and reduced once per output.
__global__ void __launch_bounds__(kThreads) k_mac(const u64* __restrict__ baby, const u64* __restrict__ pt,
                                                  u64* __restrict__ inner, int N, int L, int B, int G,
                                                  long long n_bg, LimbTable lt) {
    const long long LN = (long long)L * N;
    const int n = N >> 1;
    const long long Ln = (long long)L * n;
    for (long long pos = (long long)blockIdx.x * kThreads + threadIdx.x; pos < LN; pos += (long long)gridDim.x * kThreads) {
        const int l = (int)(pos / N), t = (int)(pos % N);
        const LimbConst& lc = lt.c[l];
        for (long long bg = blockIdx.y; bg < n_bg; bg += gridDim.y) {
            const u64* p = pt + bg * B * Ln + (long long)l * n + (t < n ? t : N - 1 - t);
            u64 h0 = 0, l0 = 0, h1 = 0, l1 = 0;
            for (int b = 0; b < B; b++) {
                u64 v = p[(long long)b * Ln];
                mac128(h0, l0, v, baby[((long long)b * 2 + 0) * LN + pos]);
                mac128(h1, l1, v, baby[((long long)b * 2 + 1) * LN + pos]);
            }
            u64* o = inner + bg * 2 * LN + pos;
            o[0] = reduce128(h0, l0, lc);
            o[LN] = reduce128(h1, l1, lc);
        }
    }
}

// Streaming kernel for moduli below 2^50 (the HBM-bound case the path is sized for).  A CTA owns 32 consecutive
// positions of one limb.  Its NG warps split the B baby steps among them: warp w keeps the baby-step words of steps
// w*BB .. w*BB+BB-1 (both ciphertext components) for its lane's position in REGISTERS for the CTA's whole life, and
// streams the matching plaintext rows of every (blk, g) pair past them, so every plaintext word is read from HBM
// exactly once, 256 contiguous bytes per warp load, with the next pair's loads in flight while the current pair is
// multiplied.  The warps' partial sums meet in shared memory once per (blk, g) pair.
// The GPU has no native 64-bit multiplier, so each residue is split into two 25-bit halves and a product costs three
// 32x32->64 multiply-adds (Karatsuba) accumulated carry-free in 64-bit registers: a sum of B <= 128 products of
// 25-bit halves stays below 2^57, of the 26-bit half sums below 2^59.
constexpr unsigned kM25 = (1u << 25) - 1;

// NQ queries at once (cross-query batching against the same encoded candidates): the warp keeps the baby-step words of NQ
// baby sets (query q at baby + q * baby_stride) and every plaintext word, still read once, feeds NQ times the products;
// partial sums of query q go to inner + q * inner_stride.
template <int NG, int BB, int NQ, int F64>
__global__ void __launch_bounds__(32 * NG) k_mac_stream(const u64* __restrict__ baby, long long baby_stride,
                                                        const u64* __restrict__ pt, u64* __restrict__ inner,
                                                        long long inner_stride, int N, int L, long long n_bg, int bg_per_cta,
                                                        const LimbConst* __restrict__ lt) {
    constexpr int B = NG * BB;
    constexpr int NV = 2 * NQ;  // (query, side): side 0 is position t, side 1 its mirror image N - 1 - t
    constexpr int PS = F64 ? 2 : 3;  // words per partial sum: (high, low) of the binary64 sums, or the three Karatsuba sums
    static_assert(F64 == 0 || BB <= 8, "the two-word binary64 sum holds eight products");
    // two buffers (a warp may write the next pair's partial sums while others still add up this pair's) where they fit the
    // static shared memory, one and a second barrier per pair otherwise
    constexpr int NBUF = (size_t)2 * NG * PS * 2 * NV * 32 * 8 > 48 * 1024 ? 1 : 2;
    __shared__ u64 part[NBUF][NG][PS * 2 * NV][32];
    const int n = N >> 1;
    const long long LN = (long long)L * N, Ln = (long long)L * n;
    const long long hpos0 = (long long)blockIdx.x * 32;  // in the stored plaintext layout [L][N/2]
    const int lane = threadIdx.x & 31, wg = threadIdx.x >> 5;
    const int limb = (int)(hpos0 / n), t0 = (int)(hpos0 % n);
    const LimbConst* lc = lt + limb;
    const long long posv[2] = {(long long)limb * N + t0 + lane, (long long)limb * N + (N - 1 - t0 - lane)};
    // this warp's baby-step words, split into 25-bit halves or (F64) as balanced binary64 integers
    unsigned w0[NV][BB][2], w1[NV][BB][2];
    double wd[NV][BB][2];
    const double qd = (double)lc->q, halfd = (double)lc->half;
    const bool big = F64 == 2 && lc->q >= (1ULL << 50);  // see k_mac_bulk
#pragma unroll
    for (int v = 0; v < NV; v++)
#pragma unroll
        for (int k = 0; k < BB; k++)
#pragma unroll
            for (int c = 0; c < 2; c++) {
                const u64 x = baby[(v >> 1) * baby_stride + ((long long)(wg * BB + k) * 2 + c) * LN + posv[v & 1]];
                if (F64) {
                    wd[v][k][c] = big ? __longlong_as_double((long long)x) : residue_to_balanced_f64(x, qd, halfd);
                } else {
                    w0[v][k][c] = (unsigned)x & kM25;
                    w1[v][k][c] = (unsigned)(x >> 25);
                }
            }
    const long long bg0 = (long long)blockIdx.y * bg_per_cta;
    const long long bg1 = bg0 + bg_per_cta < n_bg ? bg0 + bg_per_cta : n_bg;
    if (bg0 >= bg1) return;
    const u64* p = pt + (bg0 * B + wg * BB) * Ln + hpos0 + lane;
    u64 cur[BB], nxt[BB];
#pragma unroll
    for (int k = 0; k < BB; k++) cur[k] = __ldcs(p + (long long)k * Ln);
    for (long long bg = bg0; bg < bg1; bg++) {
        if (bg + 1 < bg1) {
            const u64* pn = p + (long long)B * Ln;
#pragma unroll
            for (int k = 0; k < BB; k++) nxt[k] = __ldcs(pn + (long long)k * Ln);
        }
        u64(*buf)[PS * 2 * NV][32] = part[NBUF == 2 ? (bg & 1) : 0];
        if (F64 == 2 && big) {
            u64 hi[NV][2], lo[NV][2];
#pragma unroll
            for (int v = 0; v < NV; v++)
#pragma unroll
                for (int c = 0; c < 2; c++) hi[v][c] = lo[v][c] = 0;
#pragma unroll
            for (int k = 0; k < BB; k++)
#pragma unroll
                for (int v = 0; v < NV; v++)
#pragma unroll
                    for (int c = 0; c < 2; c++) mac128(hi[v][c], lo[v][c], cur[k], (u64)__double_as_longlong(wd[v][k][c]));
#pragma unroll
            for (int v = 0; v < NV; v++)
#pragma unroll
                for (int c = 0; c < 2; c++) {
                    buf[wg][(v * 2 + c) * PS + 0][lane] = hi[v][c];
                    buf[wg][(v * 2 + c) * PS + 1][lane] = lo[v][c];
                }
        } else if (F64) {
            double ah[NV][2], al[NV][2];
#pragma unroll
            for (int v = 0; v < NV; v++)
#pragma unroll
                for (int c = 0; c < 2; c++) ah[v][c] = kAcc2Start, al[v][c] = 0;
#pragma unroll
            for (int k = 0; k < BB; k++) {
                const double pd = residue_to_f64(cur[k]);
#pragma unroll
                for (int v = 0; v < NV; v++)
#pragma unroll
                    for (int c = 0; c < 2; c++) acc2_fma(ah[v][c], al[v][c], pd, wd[v][k][c]);
            }
#pragma unroll
            for (int v = 0; v < NV; v++)
#pragma unroll
                for (int c = 0; c < 2; c++) {
                    buf[wg][(v * 2 + c) * PS + 0][lane] = (u64)acc2_high(ah[v][c]);
                    buf[wg][(v * 2 + c) * PS + 1][lane] = (u64)acc2_low(al[v][c]);
                }
        } else {
            u64 p00[NV][2], p11[NV][2], pm[NV][2];
#pragma unroll
            for (int v = 0; v < NV; v++)
#pragma unroll
                for (int c = 0; c < 2; c++) p00[v][c] = p11[v][c] = pm[v][c] = 0;
#pragma unroll
            for (int k = 0; k < BB; k++) {
                const unsigned a0 = (unsigned)cur[k] & kM25, a1 = (unsigned)(cur[k] >> 25), as = a0 + a1;
#pragma unroll
                for (int v = 0; v < NV; v++)
#pragma unroll
                    for (int c = 0; c < 2; c++) {
                        p00[v][c] += (u64)a0 * w0[v][k][c];
                        p11[v][c] += (u64)a1 * w1[v][k][c];
                        pm[v][c] += (u64)as * (w0[v][k][c] + w1[v][k][c]);
                    }
            }
#pragma unroll
            for (int v = 0; v < NV; v++)
#pragma unroll
                for (int c = 0; c < 2; c++) {
                    buf[wg][(v * 2 + c) * PS + 0][lane] = p00[v][c];
                    buf[wg][(v * 2 + c) * PS + 1][lane] = pm[v][c];
                    buf[wg][(v * 2 + c) * PS + 2][lane] = p11[v][c];
                }
        }
        __syncthreads();
        // the warps share out the 2 * NV (query, side, component) sums
        for (int vc = wg; vc < 2 * NV; vc += NG) {
            u64 r;
            if (F64 == 2 && big) {
                u64 hi = 0, lo = 0;  // at most 64 products below 2^120 each
#pragma unroll
                for (int g = 0; g < NG; g++) {
                    const u64 l = buf[g][vc * PS + 1][lane];
                    lo += l;
                    hi += buf[g][vc * PS + 0][lane] + (lo < l ? 1 : 0);
                }
                r = reduce128(hi, lo, *lc);
            } else if (F64) {
                long long m = 0, sl = 0;
#pragma unroll
                for (int g = 0; g < NG; g++) {
                    m += (long long)buf[g][vc * PS + 0][lane];
                    sl += (long long)buf[g][vc * PS + 1][lane];
                }
                r = acc2_reduce(m, sl, *lc);
            } else {
                u64 s00 = 0, sm = 0, s11 = 0;
#pragma unroll
                for (int g = 0; g < NG; g++) {
                    s00 += buf[g][vc * PS + 0][lane];
                    sm += buf[g][vc * PS + 1][lane];
                    s11 += buf[g][vc * PS + 2][lane];
                }
                // value = s00 + cross * 2^25 + s11 * 2^50 with cross = sm - s00 - s11 < 2^59
                const u64 cross = sm - s00 - s11;
                u64 lo = s00, hi = 0;
                const u64 c_lo = cross << 25, c_hi = cross >> 39;
                lo += c_lo;
                hi += c_hi + (lo < c_lo ? 1 : 0);
                const u64 d_lo = s11 << 50, d_hi = s11 >> 14;
                lo += d_lo;
                hi += d_hi + (lo < d_lo ? 1 : 0);
                r = reduce128(hi, lo, *lc);
            }
            const int v = vc >> 1;
            inner[(v >> 1) * inner_stride + (bg * 2 + (vc & 1)) * LN + posv[v & 1]] = r;
        }
        if (NBUF == 1 || NG < 2 * NV) __syncthreads();  // a warp that finishes several sums may still be reading while the next pair is written
#pragma unroll
        for (int k = 0; k < BB; k++) cur[k] = nxt[k];
        p += (long long)B * Ln;
    }
}

// Streaming form of the ct x ct multiply-accumulate for moduli below 2^50: the structure of k_mac_stream (a warp keeps
// the 25-bit halves of its BB baby-step words, both components, in registers), with the two polynomials x0, x1 of every
// database ciphertext streamed past them one after the other: x_h * y_c adds to d_{h+c}, so the three degree-2 sums share
// one set of Karatsuba accumulators and every database word is read once.
template <int NG, int BB, bool F64>
__global__ void __launch_bounds__(32 * NG) k_mac_ct_stream(const u64* __restrict__ baby, const u64* __restrict__ ctdb,
                                                           u64* __restrict__ inner3, int N, int L, long long n_bg, int bg_per_cta,
                                                           const LimbConst* __restrict__ lt) {
    constexpr int B = NG * BB;
    // partial sums per thread: three Karatsuba triples, or (F64) the two-word binary64 sums of the four products x_h y_c
    constexpr int PW = F64 ? 8 : 9;
    static_assert(!F64 || BB <= 8, "the two-word binary64 sum holds eight products");
    __shared__ u64 part[2][NG][PW][32];
    const long long LN = (long long)L * N;
    const long long pos0 = (long long)blockIdx.x * 32;
    const int lane = threadIdx.x & 31, wg = threadIdx.x >> 5;
    const LimbConst* lc = lt + pos0 / N;
    unsigned w0[BB][2], w1[BB][2];
    double wd[BB][2];
    const double qd = (double)lc->q, halfd = (double)lc->half;
#pragma unroll
    for (int k = 0; k < BB; k++)
#pragma unroll
        for (int c = 0; c < 2; c++) {
            const u64 v = baby[((long long)(wg * BB + k) * 2 + c) * LN + pos0 + lane];
            if (F64) {
                wd[k][c] = residue_to_balanced_f64(v, qd, halfd);
            } else {
                w0[k][c] = (unsigned)v & kM25;
                w1[k][c] = (unsigned)(v >> 25);
            }
        }
    const long long bg0 = (long long)blockIdx.y * bg_per_cta;
    const long long bg1 = bg0 + bg_per_cta < n_bg ? bg0 + bg_per_cta : n_bg;
    if (bg0 >= bg1) return;
    // polynomial h of the ciphertext of (pair bg, step b): ctdb + ((bg * B + b) * 2 + h) * LN
    const u64* p = ctdb + ((bg0 * B + wg * BB) * 2) * LN + pos0 + lane;
    u64 cur[BB], nxt[BB];
#pragma unroll
    for (int k = 0; k < BB; k++) cur[k] = __ldcs(p + (long long)k * 2 * LN);
    for (long long bg = bg0; bg < bg1; bg++) {
        u64 p00[3] = {0, 0, 0}, p11[3] = {0, 0, 0}, pm[3] = {0, 0, 0};
        double ah[2][2] = {{kAcc2Start, kAcc2Start}, {kAcc2Start, kAcc2Start}}, al[2][2] = {{0, 0}, {0, 0}};
#pragma unroll
        for (int h = 0; h < 2; h++) {
            // next stream element: the other polynomial of this pair, or x0 of the next pair
            const bool more = h == 0 || bg + 1 < bg1;
            if (more) {
                const u64* pn = h == 0 ? p + LN : p + (long long)B * 2 * LN;
#pragma unroll
                for (int k = 0; k < BB; k++) nxt[k] = __ldcs(pn + (long long)k * 2 * LN);
            }
#pragma unroll
            for (int k = 0; k < BB; k++) {
                if (F64) {
                    const double x = residue_to_f64(cur[k]);
#pragma unroll
                    for (int c = 0; c < 2; c++) acc2_fma(ah[h][c], al[h][c], x, wd[k][c]);
                } else {
                    const unsigned a0 = (unsigned)cur[k] & kM25, a1 = (unsigned)(cur[k] >> 25), as = a0 + a1;
#pragma unroll
                    for (int c = 0; c < 2; c++) {
                        p00[h + c] += (u64)a0 * w0[k][c];
                        p11[h + c] += (u64)a1 * w1[k][c];
                        pm[h + c] += (u64)as * (w0[k][c] + w1[k][c]);
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < BB; k++) cur[k] = nxt[k];
        }
        p += (long long)B * 2 * LN;
        u64(*buf)[PW][32] = part[bg & 1];
        if (F64) {
#pragma unroll
            for (int h = 0; h < 2; h++)
#pragma unroll
                for (int c = 0; c < 2; c++) {
                    buf[wg][(h * 2 + c) * 2 + 0][lane] = (u64)acc2_high(ah[h][c]);
                    buf[wg][(h * 2 + c) * 2 + 1][lane] = (u64)acc2_low(al[h][c]);
                }
        } else {
#pragma unroll
            for (int c = 0; c < 3; c++) {
                buf[wg][c * 3 + 0][lane] = p00[c];
                buf[wg][c * 3 + 1][lane] = pm[c];
                buf[wg][c * 3 + 2][lane] = p11[c];
            }
        }
        __syncthreads();
        for (int c = wg; c < 3; c += NG) {
            u64 r;
            if (F64) {
                // d_c = sum over the warps of the products x_h y_(c-h): (0,0) | (0,1) + (1,0) | (1,1)
                long long m = 0, sl = 0;
#pragma unroll
                for (int g = 0; g < NG; g++) {
                    if (c != 2) {
                        m += (long long)buf[g][c * 2 + 0][lane];
                        sl += (long long)buf[g][c * 2 + 1][lane];
                    }
                    if (c != 0) {
                        m += (long long)buf[g][(c + 1) * 2 + 0][lane];
                        sl += (long long)buf[g][(c + 1) * 2 + 1][lane];
                    }
                }
                r = acc2_reduce(m, sl, *lc);
            } else {
                u64 s00 = 0, sm = 0, s11 = 0;
#pragma unroll
                for (int g = 0; g < NG; g++) {
                    s00 += buf[g][c * 3 + 0][lane];
                    sm += buf[g][c * 3 + 1][lane];
                    s11 += buf[g][c * 3 + 2][lane];
                }
                // d1 sums 2 B products: B <= 64 keeps the 25-bit-half sums below 2^57 and the half-sum products below 2^59
                const u64 cross = sm - s00 - s11;
                u64 lo = s00, hi = 0;
                const u64 c_lo = cross << 25, c_hi = cross >> 39;
                lo += c_lo;
                hi += c_hi + (lo < c_lo ? 1 : 0);
                const u64 d_lo = s11 << 50, d_hi = s11 >> 14;
                lo += d_lo;
                hi += d_hi + (lo < d_lo ? 1 : 0);
                r = reduce128(hi, lo, *lc);
            }
            inner3[(bg * 3 + c) * LN + pos0 + lane] = r;
        }
        if (NG < 3) __syncthreads();
    }
}

// The single-query kernel with the plaintext rows brought in by bulk asynchronous copies.  With register prefetch a warp
// has 2 KiB in flight and an SM 32 KiB, short of what the memory latency needs at full bandwidth; here every warp runs its
// own ring of kMacStages buffers (one (blk, g) pair of its BB rows each, 256 B per row: ONE box of a 2-D tensor map over
// the plaintexts, rows = (blk, g, b), columns = limb positions), refilled by lane 0 as soon as the warp has taken a pair
// into registers, so an SM keeps about four times as much in flight and the registers of the prefetch
// are free.  Completion is signalled on per-buffer mbarriers; waits are bounded, and a warp whose wait runs out raises the
// context's kernel flag and lets the whole CTA leave at its next barrier.
constexpr int kMacStages = 4;

// partial sums per thread that cross the warps: four sums of three words (integer multiplier) or of two (FP64 pipe)
template <int NG, int BB, int F64>
constexpr size_t mac_bulk_smem() {
    return (size_t)NG * kMacStages * BB * 256 + (size_t)2 * NG * (F64 ? 8 : 12) * 256 + (size_t)NG * kMacStages * 8 + 16;
}

// F64 != 0: the products are summed exactly in pairs of binary64 words on the FP64 pipe (acc2_fma: four operations per
// product on a pipe of more than twice the multiplier's throughput, and two words of partial sum per thread instead of
// three); 0: on the integer multiplier as in k_mac_stream.  Same integers either way, hence the same residues.
template <int NG, int BB, int F64>
__global__ void __launch_bounds__(32 * NG) k_mac_bulk(const u64* __restrict__ baby, const __grid_constant__ CUtensorMap pt_map,
                                                      u64* __restrict__ inner, int N, int L, long long n_bg, int bg_per_cta,
                                                      const LimbConst* __restrict__ lt, int* kflag) {
    constexpr int B = NG * BB;
    extern __shared__ __align__(128) u64 smem_mac[];
    u64(*ring)[kMacStages][BB][32] = (u64(*)[kMacStages][BB][32])smem_mac;                        // [NG]
    constexpr int PS = F64 ? 2 : 3, PW = 4 * PS;  // words per partial sum, per thread
    u64(*part)[NG][PW][32] = (u64(*)[NG][PW][32])(smem_mac + (size_t)NG * kMacStages * BB * 32);  // [2]
    u64(*bars)[kMacStages] = (u64(*)[kMacStages])(smem_mac + (size_t)NG * kMacStages * BB * 32 + (size_t)2 * NG * PW * 32);  // [NG]
    int& s_abort = *(int*)(&bars[NG][0]);
    const int n = N >> 1;
    const long long LN = (long long)L * N;
    const long long hpos0 = (long long)blockIdx.x * 32;  // in the stored plaintext layout [L][N/2]
    const int lane = threadIdx.x & 31, wg = threadIdx.x >> 5;
    const int limb = (int)(hpos0 / n), t0 = (int)(hpos0 % n);
    const LimbConst* lc = lt + limb;
    // side 0: position t of the limb, side 1: its mirror image N - 1 - t (same plaintext word)
    const long long posv[2] = {(long long)limb * N + t0 + lane, (long long)limb * N + (N - 1 - t0 - lane)};
    const long long bg0 = (long long)blockIdx.y * bg_per_cta;
    const long long bg1 = bg0 + bg_per_cta < n_bg ? bg0 + bg_per_cta : n_bg;
    if (bg0 >= bg1) return;
    const int npairs = (int)(bg1 - bg0);
    const unsigned bar0 = smem_addr(&bars[wg][0]), ring0 = smem_addr(&ring[wg][0][0][0]);
    const int row0 = (int)(bg0 * B + wg * BB);  // first plaintext row of this warp's pair 0; pair i starts B rows further
    if (threadIdx.x == 0) s_abort = 0;
    if (lane == 0) {
        for (int st = 0; st < kMacStages; st++) mbar_init(bar0 + 8 * st, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int i = 0; i < kMacStages && i < npairs; i++) {
            mbar_expect_tx(bar0 + 8 * i, BB * 256);
            tensor_load_2d(ring0 + i * BB * 256, &pt_map, (int)hpos0, row0 + i * B, bar0 + 8 * i);
        }
    }
    // this warp's baby-step words of both sides: split into 25-bit halves, or (F64) as balanced binary64 integers
    static_assert(F64 == 0 || BB <= 8, "the two-word binary64 sum holds eight products");
    unsigned w0[2][BB][2], w1[2][BB][2];
    double wd[2][BB][2];
    const double qd = (double)lc->q, halfd = (double)lc->half;
    // F64 == 2: the chain has primes in [2^50, 2^60); their limbs (uniform over a CTA) take 128-bit integer sums, the words
    // kept as they are
    const bool big = F64 == 2 && lc->q >= (1ULL << 50);
#pragma unroll
    for (int v = 0; v < 2; v++)
#pragma unroll
        for (int k = 0; k < BB; k++)
#pragma unroll
            for (int c = 0; c < 2; c++) {
                const u64 x = baby[((long long)(wg * BB + k) * 2 + c) * LN + posv[v]];
                if (F64) {
                    wd[v][k][c] = big ? __longlong_as_double((long long)x) : residue_to_balanced_f64(x, qd, halfd);
                } else {
                    w0[v][k][c] = (unsigned)x & kM25;
                    w1[v][k][c] = (unsigned)(x >> 25);
                }
            }
    __syncthreads();  // s_abort and the barriers are initialised
    for (int i = 0; i < npairs; i++) {
        const int st = i % kMacStages;
        const bool arrived = mbar_wait(bar0 + 8 * st, (unsigned)(i / kMacStages) & 1u);
        if (!arrived && lane == 0) {
            raise_flag(kflag);
            s_abort = 1;
        }
        u64 cur[BB];
#pragma unroll
        for (int k = 0; k < BB; k++) cur[k] = ring[wg][st][k][lane];
        // every lane holds its words: order the reads before the asynchronous refill of the buffer
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0 && arrived && i + kMacStages < npairs) {
            mbar_expect_tx(bar0 + 8 * st, BB * 256);
            tensor_load_2d(ring0 + st * BB * 256, &pt_map, (int)hpos0, row0 + (i + kMacStages) * B, bar0 + 8 * st);
        }
        u64(*buf)[PW][32] = part[i & 1];
        if (F64 == 2 && big) {
            u64 hi[2][2] = {{0, 0}, {0, 0}}, lo[2][2] = {{0, 0}, {0, 0}};
#pragma unroll
            for (int k = 0; k < BB; k++)
#pragma unroll
                for (int v = 0; v < 2; v++)
#pragma unroll
                    for (int c = 0; c < 2; c++) mac128(hi[v][c], lo[v][c], cur[k], (u64)__double_as_longlong(wd[v][k][c]));
#pragma unroll
            for (int v = 0; v < 2; v++)
#pragma unroll
                for (int c = 0; c < 2; c++) {
                    buf[wg][(v * 2 + c) * PS + 0][lane] = hi[v][c];
                    buf[wg][(v * 2 + c) * PS + 1][lane] = lo[v][c];
                }
        } else if (F64) {
            double ah[2][2] = {{kAcc2Start, kAcc2Start}, {kAcc2Start, kAcc2Start}}, al[2][2] = {{0, 0}, {0, 0}};
#pragma unroll
            for (int k = 0; k < BB; k++) {
                const double p = residue_to_f64(cur[k]);
#pragma unroll
                for (int v = 0; v < 2; v++)
#pragma unroll
                    for (int c = 0; c < 2; c++) acc2_fma(ah[v][c], al[v][c], p, wd[v][k][c]);
            }
#pragma unroll
            for (int v = 0; v < 2; v++)
#pragma unroll
                for (int c = 0; c < 2; c++) {
                    buf[wg][(v * 2 + c) * PS + 0][lane] = (u64)acc2_high(ah[v][c]);
                    buf[wg][(v * 2 + c) * PS + 1][lane] = (u64)acc2_low(al[v][c]);
                }
        } else {
            u64 p00[2][2] = {{0, 0}, {0, 0}}, p11[2][2] = {{0, 0}, {0, 0}}, pm[2][2] = {{0, 0}, {0, 0}};
#pragma unroll
            for (int k = 0; k < BB; k++) {
                const unsigned a0 = (unsigned)cur[k] & kM25, a1 = (unsigned)(cur[k] >> 25), as = a0 + a1;
#pragma unroll
                for (int v = 0; v < 2; v++)
#pragma unroll
                    for (int c = 0; c < 2; c++) {
                        p00[v][c] += (u64)a0 * w0[v][k][c];
                        p11[v][c] += (u64)a1 * w1[v][k][c];
                        pm[v][c] += (u64)as * (w0[v][k][c] + w1[v][k][c]);
                    }
            }
#pragma unroll
            for (int v = 0; v < 2; v++)
#pragma unroll
                for (int c = 0; c < 2; c++) {
                    buf[wg][(v * 2 + c) * PS + 0][lane] = p00[v][c];
                    buf[wg][(v * 2 + c) * PS + 1][lane] = pm[v][c];
                    buf[wg][(v * 2 + c) * PS + 2][lane] = p11[v][c];
                }
        }
        __syncthreads();
        if (s_abort) {
            // leave together; first give this warp's copies still in flight the same bounded time
            for (int j = i + 1; j < npairs && j < i + kMacStages; j++) mbar_wait(bar0 + 8 * (j % kMacStages), (unsigned)(j / kMacStages) & 1u);
            return;
        }
        for (int vc = wg; vc < 4; vc += NG) {
            u64 r;
            if (F64 == 2 && big) {
                u64 hi = 0, lo = 0;  // at most 64 products below 2^120 each
#pragma unroll
                for (int g = 0; g < NG; g++) {
                    const u64 l = buf[g][vc * PS + 1][lane];
                    lo += l;
                    hi += buf[g][vc * PS + 0][lane] + (lo < l ? 1 : 0);
                }
                r = reduce128(hi, lo, *lc);
            } else if (F64) {
                long long m = 0, sl = 0;
#pragma unroll
                for (int g = 0; g < NG; g++) {
                    m += (long long)buf[g][vc * PS + 0][lane];
                    sl += (long long)buf[g][vc * PS + 1][lane];
                }
                r = acc2_reduce(m, sl, *lc);
            } else {
                u64 s00 = 0, sm = 0, s11 = 0;
#pragma unroll
                for (int g = 0; g < NG; g++) {
                    s00 += buf[g][vc * PS + 0][lane];
                    sm += buf[g][vc * PS + 1][lane];
                    s11 += buf[g][vc * PS + 2][lane];
                }
                const u64 cross = sm - s00 - s11;
                u64 lo = s00, hi = 0;
                const u64 c_lo = cross << 25, c_hi = cross >> 39;
                lo += c_lo;
                hi += c_hi + (lo < c_lo ? 1 : 0);
                const u64 d_lo = s11 << 50, d_hi = s11 >> 14;
                lo += d_lo;
                hi += d_hi + (lo < d_lo ? 1 : 0);
                r = reduce128(hi, lo, *lc);
            }
            inner[((bg0 + i) * 2 + (vc & 1)) * LN + posv[vc >> 1]] = r;
        }
        if (NG < 4) __syncthreads();
    }
}

// ct x ct multiply-accumulate (generic, any modulus): inner3[bg][0..2][l][t] = sum_b (x0 y0, x0 y1 + x1 y0, x1 y1),
// x = ctdb[bg][b], y = baby[b]
__global__ void __launch_bounds__(kThreads) k_mac_ct(const u64* __restrict__ baby, const u64* __restrict__ ctdb, u64* __restrict__ inner3,
                                                     int N, int L, int B, long long n_bg, LimbTable lt) {
    const long long LN = (long long)L * N;
    for (long long pos = (long long)blockIdx.x * kThreads + threadIdx.x; pos < LN; pos += (long long)gridDim.x * kThreads) {
        const LimbConst& lc = lt.c[(int)(pos / N)];
        for (long long bg = blockIdx.y; bg < n_bg; bg += gridDim.y) {
            const u64* x = ctdb + bg * B * 2 * LN + pos;
            u64 h0 = 0, l0 = 0, h1 = 0, l1 = 0, h2 = 0, l2 = 0;
            for (int b = 0; b < B; b++) {
                const u64 x0 = __ldcs(x + ((long long)b * 2 + 0) * LN), x1 = __ldcs(x + ((long long)b * 2 + 1) * LN);
                const u64 y0 = baby[((long long)b * 2 + 0) * LN + pos], y1 = baby[((long long)b * 2 + 1) * LN + pos];
                mac128(h0, l0, x0, y0);
                mac128(h1, l1, x0, y1);
                mac128(h1, l1, x1, y0);
                mac128(h2, l2, x1, y1);
            }
            u64* o = inner3 + bg * 3 * LN + pos;
            o[0] = reduce128(h0, l0, lc);
            o[LN] = reduce128(h1, l1, lc);
            o[2 * LN] = reduce128(h2, l2, lc);
        }
    }
}

}  // namespace

// 2-D tiled tensor map over the stored plaintexts of a level: `rows` rows of Ln = L * N/2 64-bit words, boxes of box_rows x 32 words.  The
// encoder is a driver entry point, looked up once (no link against the driver library); false if it cannot be had.
typedef CUresult (*TensorMapEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                           const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                           CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
bool plaintext_map(const u64* pt, long long Ln, long long rows, int box_rows, CUtensorMap* out) {
    static TensorMapEncodeTiledFn encode = [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &res) != cudaSuccess || res != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            fn = nullptr;
        }
        return (TensorMapEncodeTiledFn)fn;
    }();
    if (!encode) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)Ln, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)Ln * 8};
    const cuuint32_t box[2] = {32, (cuuint32_t)box_rows};
    const cuuint32_t elem_strides[2] = {1, 1};
    return encode(out, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, (void*)pt, dims, strides, box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int NG, int BB, int NQ>
void launch_mac_stream(hann_ctx* c, const u64* baby, int64_t baby_stride, const u64* pt, int64_t n_bg, u64* inner,
                       int64_t inner_stride) {
    const long long Ln = (long long)c->L * c->n;
    const int tiles = (int)(Ln / 32);
    bool big_primes = false;  // primes in [2^50, 2^60): the caller lets them through only with the FP64 variant and one query
    for (int l = 0; l < c->L; l++) big_primes = big_primes || c->mod[l] >= (1ULL << 50);
    // split the (blk, g) range over grid.y only as far as needed to fill the machine: every extra split re-reads the
    // baby-step words
    int split = 1;
    while ((long long)tiles * split < 148 * 8 && split < n_bg) split *= 2;
    const int per = (int)((n_bg + split - 1) / split);
    split = (int)((n_bg + per - 1) / per);
    KProf kp(c, KC_MAC);
#ifndef HANN_NO_MAC_BULK
    // one query, up to 32 baby steps, 16-byte aligned plaintexts, row count within a 32-bit coordinate: the tensor-copy
    // kernel
    if constexpr (NQ == 1 && NG * BB <= 32) {
        CUtensorMap map;
        if (((uintptr_t)pt & 15) == 0 && n_bg * (NG * BB) < (1LL << 31) && plaintext_map(pt, Ln, n_bg * (NG * BB), BB, &map)) {
            auto go = [&](auto kern, size_t smem) {
                if (smem > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
                kern<<<dim3(tiles, split), 32 * NG, smem, c->stream>>>(baby, map, inner, c->N, c->L, n_bg, per, c->lt_dev, c->kflag);
            };
            if (!c->mac_f64) go(k_mac_bulk<NG, BB, 0>, mac_bulk_smem<NG, BB, 0>());
            else if (big_primes) go(k_mac_bulk<NG, BB, 2>, mac_bulk_smem<NG, BB, 2>());
            else go(k_mac_bulk<NG, BB, 1>, mac_bulk_smem<NG, BB, 1>());
            return;
        }
    }
#endif
    if constexpr (BB <= 8) {
        if (c->mac_f64 && !big_primes) {
            k_mac_stream<NG, BB, NQ, 1><<<dim3(tiles, split), 32 * NG, 0, c->stream>>>(baby, baby_stride, pt, inner, inner_stride, c->N, c->L,
                                                                                        n_bg, per, c->lt_dev);
            return;
        }
        if constexpr (NQ == 1) {
            if (c->mac_f64) {
                k_mac_stream<NG, BB, 1, 2><<<dim3(tiles, split), 32 * NG, 0, c->stream>>>(baby, baby_stride, pt, inner, inner_stride, c->N, c->L,
                                                                                           n_bg, per, c->lt_dev);
                return;
            }
        }
    }
    // (two queries at more than 16 baby steps exist in the FP64 form only: the three-word partial sums of the integer form
    // do not fit the static shared memory; the caller does not pair queries there)
    if constexpr (!(NQ == 2 && NG * BB > 16))
        k_mac_stream<NG, BB, NQ, 0><<<dim3(tiles, split), 32 * NG, 0, c->stream>>>(baby, baby_stride, pt, inner, inner_stride, c->N, c->L,
                                                                                    n_bg, per, c->lt_dev);
}

// the baby-step words of NQ queries x 2 sides live in registers: 8 BB NQ of them per thread, hence BB <= 8 for one query
// and BB <= 4 for two (B <= 16: with more warps the partial sums would not fit the static shared memory)
template <int NQ>
void launch_mac_stream_b(hann_ctx* c, const u64* baby, int64_t baby_stride, const u64* pt, int64_t n_bg, u64* inner,
                         int64_t inner_stride) {
    switch (c->B) {
        case 1: launch_mac_stream<1, 1, NQ>(c, baby, baby_stride, pt, n_bg, inner, inner_stride); break;
        case 2: launch_mac_stream<2, 1, NQ>(c, baby, baby_stride, pt, n_bg, inner, inner_stride); break;
        case 4: launch_mac_stream<4, 1, NQ>(c, baby, baby_stride, pt, n_bg, inner, inner_stride); break;
        case 8: launch_mac_stream<4, 2, NQ>(c, baby, baby_stride, pt, n_bg, inner, inner_stride); break;
        case 16: launch_mac_stream<4, 4, NQ>(c, baby, baby_stride, pt, n_bg, inner, inner_stride); break;
        case 32:
            if constexpr (NQ == 1) launch_mac_stream<4, 8, NQ>(c, baby, baby_stride, pt, n_bg, inner, inner_stride);
            else launch_mac_stream<8, 4, NQ>(c, baby, baby_stride, pt, n_bg, inner, inner_stride);
            break;
        default:
            if constexpr (NQ == 1) launch_mac_stream<8, 8, NQ>(c, baby, baby_stride, pt, n_bg, inner, inner_stride);
            break;
    }
}

// n_queries baby sets [q][B][2][L][N] against the same n_blocks encoded blocks -> inner [q][n_blocks][G][2][L][N]
int launch_mac_batch(hann_ctx* c, const u64* baby, int n_queries, const u64* pt, int64_t n_blocks, u64* inner) {
    if (n_blocks <= 0 || n_queries <= 0) return HANN_OK;
    const long long LN = (long long)c->L * c->N;
    const long long n_bg = n_blocks * c->G;
    const int64_t baby_stride = (int64_t)c->B * 2 * LN, inner_stride = n_bg * 2 * LN;
    // the streaming kernels: moduli below 2^50, or (their FP64 variant only) below 2^60 with the limbs of the larger primes
    // summed in 128-bit integers
    bool small = c->N >= 64 && c->B <= 64 && (c->B & (c->B - 1)) == 0;
    for (int l = 0; l < c->L; l++) small = small && c->mod[l] < (c->mac_f64 ? (1ULL << 60) : (1ULL << 50));
    if (small) {
        // pairs of queries share one pass over the stored plaintexts where the baby-step words of two queries and both
        // sides fit the register file (B <= 16); a last odd query, and every query of wider baby sets, takes a pass of
        // its own
        int q = 0;
        bool pairs = c->B <= 16 || (c->B == 32 && c->mac_f64 && c->pair_b32);
        for (int l = 0; l < c->L; l++) pairs = pairs && c->mod[l] < (1ULL << 50);
        if (pairs)
            for (; q + 2 <= n_queries; q += 2) launch_mac_stream_b<2>(c, baby + q * baby_stride, baby_stride, pt, n_bg, inner + q * inner_stride, inner_stride);
        for (; q < n_queries; q++) launch_mac_stream_b<1>(c, baby + q * baby_stride, baby_stride, pt, n_bg, inner + q * inner_stride, inner_stride);
        return check_launch(c, "mac_stream");
    }
    int gx = (int)((LN + kThreads - 1) / kThreads);
    int gy = 1;
    // enough CTAs to fill the machine even for a single small block
    while ((long long)gx * gy < 148 * 8 && gy < n_bg) gy *= 2;
    if (gy > n_bg) gy = (int)n_bg;
    for (int q = 0; q < n_queries; q++) {
        KProf kp(c, KC_MAC);
        k_mac<<<dim3(gx, gy), kThreads, 0, c->stream>>>(baby + q * baby_stride, pt, inner + q * inner_stride, c->N, c->L, c->B, c->G, n_bg,
                                                        c->lt);
    }
    return check_launch(c, "mac");
}

int launch_mac(hann_ctx* c, const u64* baby, const u64* pt, int64_t n_blocks, u64* inner) {
    return launch_mac_batch(c, baby, 1, pt, n_blocks, inner);
}

// sums of B <= 2^7 products of residues below 2^62 fit the 128-bit accumulators only for moduli below 2^60 (two products
// per step in d1): checked by the caller
int launch_mac_ct(hann_ctx* c, const u64* baby, const u64* ctdb, int64_t n_bg, u64* inner3) {
    if (n_bg <= 0) return HANN_OK;
    const long long LN = (long long)c->L * c->N;
    bool small = c->N >= 32 && c->B <= 64 && c->B >= 4;
    for (int l = 0; l < c->L; l++) small = small && c->mod[l] < (1ULL << 50);
    if (small) {
        const int tiles = (int)(LN / 32);
        int split = 1;
        while ((long long)tiles * split < 148 * 8 && split < n_bg) split *= 2;
        const int per = (int)((n_bg + split - 1) / split);
        split = (int)((n_bg + per - 1) / per);
        KProf kp(c, KC_MAC);
        const dim3 grid(tiles, split);
        auto go = [&](auto kern, int threads) { kern<<<grid, threads, 0, c->stream>>>(baby, ctdb, inner3, c->N, c->L, n_bg, per, c->lt_dev); };
        if (c->mac_f64) {
            switch (c->B) {
                case 4: go(k_mac_ct_stream<4, 1, true>, 128); break;
                case 8: go(k_mac_ct_stream<4, 2, true>, 128); break;
                case 16: go(k_mac_ct_stream<4, 4, true>, 128); break;
                case 32: go(k_mac_ct_stream<4, 8, true>, 128); break;
                case 64: go(k_mac_ct_stream<8, 8, true>, 256); break;
                default: small = false; break;
            }
        } else {
            switch (c->B) {
                case 4: go(k_mac_ct_stream<4, 1, false>, 128); break;
                case 8: go(k_mac_ct_stream<4, 2, false>, 128); break;
                case 16: go(k_mac_ct_stream<4, 4, false>, 128); break;
                case 32: go(k_mac_ct_stream<4, 8, false>, 128); break;
                case 64: go(k_mac_ct_stream<8, 8, false>, 256); break;
                default: small = false; break;
            }
        }
        if (small) return check_launch(c, "mac_ct_stream");
    }
    int gx = (int)((LN + kThreads - 1) / kThreads), gy = 1;
    while ((long long)gx * gy < 148 * 8 && gy < n_bg) gy *= 2;
    if (gy > n_bg) gy = (int)n_bg;
    {
        KProf kp(c, KC_MAC);
        k_mac_ct<<<dim3(gx, gy), kThreads, 0, c->stream>>>(baby, ctdb, inner3, c->N, c->L, c->B, n_bg, c->lt);
    }
    return check_launch(c, "mac_ct");
}
