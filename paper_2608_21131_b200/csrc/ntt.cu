// Negacyclic number-theoretic transforms over 64-bit RNS limbs.
//
// Forward: Cooley-Tukey butterflies with merged powers of psi, natural order in, bit-reversed order out
// (position k holds the value at psi^(2*brev(k)+1)); inverse: Gentleman-Sande, bit-reversed in, natural out,
// scaled by N^{-1}.
//
// A transform of N = 2^logN points is split into two passes:
//   pass A covers the a = logN - b stages whose butterfly span is >= S = 2^b words (a CTA owns C adjacent columns
//          of the 2^a x S matrix view of the polynomial);
//   pass B covers the b stages inside contiguous chunks of S words (a CTA owns K chunks), b = min(logN, 8).
// Each pass runs its stages in at most two register rounds: a thread loads 2^R words (R <= 4), runs R stages on
// them without touching memory, and the rounds exchange through shared memory.  Stage s of a round whose first
// stage has m0 groups, of which this thread sits in group i0, uses table entry ((m0 + i0) << s) + il, il being the
// group inside the thread's register array: the same rule serves both passes, both rounds and both directions.
//
// Arithmetic.  Three exact implementations of the same modular butterflies, chosen per limb by the size of q:
//   * q < 2^50: binary64.  Residues are held as balanced integers in doubles; a product y*w mod q is
//       h = fl(y*w), l = fma(y, w, -h), c = rint(y * fl(w/q)), t = fma(-c, q, h) + l
//     which is exact (t = y*w - c*q) while |y| <= 8q, with |t| <= (1/2 + k/8) q for |y| <= k q (the quotient estimate
//     is off by at most k/8 before rounding).  A forward stage maps values bounded by b q to values bounded by
//     (b + 1/2 + b/8) q: from reduced inputs (b = 1/2) eight stages reach 1.06, 1.70, 2.41, 3.21, 4.11, 5.12, 6.26,
//     7.55 -- below 8, so a whole pass of eight stages runs without a reduction and every intermediate stays an
//     integer below 2^53; from inputs in (-q, q) (b = 1) four stages reach 4.0.  While the multiplied value is
//     below 4q (the first five stages from reduced inputs) the quotient is rounded inside a multiply-add with
//     1.5 * 2^52 on the FP64 pipe; the later stages use the conversion unit's rint, which runs beside that pipe.
//     An inverse stage doubles a bound, so inverse rounds have at most 4 stages from |x| <= q/2.  Conversions between
//     integers below 2^52 and doubles go through the mantissa of 2^52 + v.  The FP64 pipe sustains about twice
//     the butterflies per second of the integer pipe, which has no native 64-bit multiply.
//   * q < 2^57: 64-bit integers, Shoup multiplication, no correction inside a forward transform (a value grows by
//     at most 2q per stage, 16 stages stay below 33q < 2^63), one chain of conditional subtractions at the end.
//   * otherwise (the ~60-bit special prime): Harvey's lazy butterflies in [0, 4q).
// The inverse integer path keeps values in [0, 2q) throughout.  Between pass A and pass B the words in memory are in
// the private format of the limb's arithmetic (double bits or lazily reduced integers); every polynomial that leaves
// a transform is in [0, q).
#include <algorithm>

#include "internal.h"
#include "bulkcopy.cuh"
#include "nttcore.cuh"

namespace {

constexpr int kThreads = 256;

struct NttArgs {
    u64* data;
    long long stride;  // words between consecutive polynomials
    int logN, a, b;    // a + b = logN
    int logC, K;       // log2(columns per CTA) in pass A, chunks per CTA in pass B
    const void* tw;      // [L+1][N] twiddle pairs in the format of the launch's arithmetic
    const LimbConst* lt;  // per-limb constants (device memory)
    // a launch covers, out of every group of `period` consecutive polynomials, the nsel positions pos[] (their limbs
    // limb[]): all positions whose modulus falls in the launch's arithmetic class
    int period, nsel;
    int tau;  // chunks of 256 positions are stored with their low nibbles swapped (see galois_src)
    // inverse pass B' only (bulk-copy kernel): read group g, position pos from src + g * src_gstride + pos * stride instead
    // of from `data` (nullptr: in place)
    const u64* src;
    long long src_gstride;
    u64 pos4, limb4;  // 4-bit fields: position within the period and limb of selection k (at most 16 selections)
    // forward pass B (bulk-copy kernel) of polynomials that are fixed by X -> 1/X and stored as their first N/2 transform
    // values only: the grid covers the first half of the chunks (stride is then N/2 or more)
    int half;
};

struct Sel {
    long long poly;
    int limb;
};
__device__ __forceinline__ Sel select(const NttArgs& A) {
    const int y = blockIdx.y, k = y % A.nsel;
    Sel s;
    s.poly = (long long)(y / A.nsel) * A.period + (int)((A.pos4 >> (4 * k)) & 15);
    s.limb = (int)((A.limb4 >> (4 * k)) & 15);
    return s;
}

// ---- forward pass A: stages 0 .. a-1 on a tile of 2^a rows x C columns ----------------------------------------

template <int R1, int R2, class AR>
__device__ __forceinline__ void fwd_a_body(const NttArgs& A, const AR ar, u64* __restrict__ base, const typename AR::TW* __restrict__ tw,
                                           u64* __restrict__ sm) {
    const int S = 1 << A.b, logC = A.logC, C = 1 << logC;
    constexpr int G1 = 1 << R2;  // rows >> R1
    for (int w = threadIdx.x; w < (G1 << logC); w += kThreads) {
        const int c = w & (C - 1), g = w >> logC;
        typename AR::T x[1 << R1];
#pragma unroll
        for (int e = 0; e < (1 << R1); e++) x[e] = ar.from_canonical(base[(size_t)(g + G1 * e) * S + c]);
        fwd_round<R1>(ar, x, tw, 1u);
        if (R2 == 0) {
#pragma unroll
            for (int e = 0; e < (1 << R1); e++) base[(size_t)(g + G1 * e) * S + c] = ar.to_mid(x[e]);
        } else {
#pragma unroll
            for (int e = 0; e < (1 << R1); e++) sm[((g + G1 * e) << logC) + c] = ar.to_mid(x[e]);
        }
    }
    if (R2 == 0) return;
    __syncthreads();
    constexpr int G2 = 1 << R1;  // rows >> R2
    constexpr int RR2 = R2 == 0 ? 1 : R2;
    for (int w = threadIdx.x; w < (G2 << logC); w += kThreads) {
        const int c = w & (C - 1), g = w >> logC;
        typename AR::T x[1 << RR2];
#pragma unroll
        for (int e = 0; e < (1 << RR2); e++) x[e] = ar.from_mid(sm[(((g << RR2) + e) << logC) + c]);
        fwd_round<RR2>(ar, x, tw, (unsigned)(G2 + g));
#pragma unroll
        for (int e = 0; e < (1 << RR2); e++) base[(size_t)((g << RR2) + e) * S + c] = ar.to_mid(x[e]);
    }
}

template <int R1, int R2, class AR>
__global__ void __launch_bounds__(kThreads, AR::kMinBlocks) k_ntt_fwd_a(NttArgs A) {
    extern __shared__ u64 sm[];
    const Sel sel = select(A);
    const AR ar(A.lt + sel.limb);
    u64* base = A.data + sel.poly * A.stride + ((long long)blockIdx.x << A.logC);
    fwd_a_body<R1, R2>(A, ar, base, (const typename AR::TW*)A.tw + ((size_t)sel.limb << A.logN), sm);
}

// ---- forward pass B: stages a .. logN-1 inside contiguous chunks of S = 2^(R1+R2) words --------------------------

template <int R1, int R2, class AR>
__device__ __forceinline__ void fwd_b_body(const NttArgs& A, const AR ar, u64* __restrict__ base, int chunk0,
                                           const typename AR::TW* __restrict__ tw, u64* __restrict__ sm) {
    constexpr int S = 1 << (R1 + R2), J1 = 1 << R2, SP = R2 == 0 ? S : S + (S >> R2);
    const int K = A.K;
    const unsigned m0 = 1u << A.a;
    const bool first = A.a == 0;  // no pass A ran: the input is canonical
    for (int w = threadIdx.x; w < K * J1; w += kThreads) {
        const int ch = w / J1, j = w % J1;
        u64* p = base + (size_t)ch * S;
        typename AR::T x[1 << R1];
#pragma unroll
        for (int e = 0; e < (1 << R1); e++) {
            const u64 v = p[j + J1 * e];
            x[e] = first ? ar.from_canonical(v) : ar.from_mid(v);
        }
        fwd_round<R1>(ar, x, tw, m0 + (unsigned)(chunk0 + ch));
        if (R2 == 0) {
#pragma unroll
            for (int e = 0; e < (1 << R1); e++) p[j + J1 * e] = ar.to_canonical(x[e]);
        } else {
#pragma unroll
            for (int e = 0; e < (1 << R1); e++) sm[ch * SP + pad<R2>(j + J1 * e)] = ar.to_mid(x[e]);
        }
    }
    if (R2 == 0) return;
    __syncthreads();
    constexpr int RR2 = R2 == 0 ? 1 : R2;
    constexpr int J2 = 1 << R1;
    for (int w = threadIdx.x; w < K * J2; w += kThreads) {
        const int ch = w / J2, j = w % J2;
        u64* s = sm + ch * SP + pad<R2>(j << RR2);
        typename AR::T x[1 << RR2];
#pragma unroll
        for (int e = 0; e < (1 << RR2); e++) x[e] = ar.from_mid(s[e]);
        fwd_round<RR2>(ar, x, tw, ((m0 + (unsigned)(chunk0 + ch)) << R1) + (unsigned)j);
#pragma unroll
        for (int e = 0; e < (1 << RR2); e++) s[e] = ar.to_canonical(x[e]);
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < K * S; idx += kThreads) base[idx] = sm[(idx / S) * SP + pad<R2>(idx % S)];
}

template <int R1, int R2, class AR>
__global__ void __launch_bounds__(kThreads, AR::kMinBlocks) k_ntt_fwd_b(NttArgs A) {
    extern __shared__ u64 sm[];
    const Sel sel = select(A);
    const AR ar(A.lt + sel.limb);
    const int chunk0 = blockIdx.x * A.K;
    u64* base = A.data + sel.poly * A.stride + ((size_t)chunk0 << (R1 + R2));
    fwd_b_body<R1, R2>(A, ar, base, chunk0, (const typename AR::TW*)A.tw + ((size_t)sel.limb << A.logN), sm);
}

// Forward pass B for rings of at least 2^9 points (chunks of 256 words, two rounds of four stages).  A CTA takes kBK
// chunks of kBPG polynomials that share their modulus (same position in consecutive limb periods): the 255 twiddle pairs
// of each chunk are staged in shared memory once and serve all kBPG polynomials, which cuts the table traffic (two
// table bytes per data byte otherwise) and keeps the twiddles out of the register file.
constexpr int kBK = 4, kBPG = 4;
#ifndef HANN_B8_MINBLOCKS
#define HANN_B8_MINBLOCKS 3
#endif

template <class AR>
__global__ void __launch_bounds__(256, HANN_B8_MINBLOCKS) k_ntt_fwd_b8(NttArgs A, int groups) {
    extern __shared__ u64 smraw[];
    typedef typename AR::TW TW;
    // twiddle cache [kBK][256].  Entries 0..14: pass stages 0..3 (e + 1 = 2^s + il; read by all 16 threads of a chunk at
    // once: broadcast).  Entries 16..255: pass stages 4..7, stored [2^u - 1 + il'][j] so that the 16 threads j of a chunk,
    // which need group j*2^u + il' of stage 4 + u, read consecutive 16-byte words (no bank conflicts).
    TW* tc = (TW*)smraw;
    u64* sm = smraw + kBK * 256 * 2;     // [kBPG][kBK][272] padded chunks
    const int k = blockIdx.y;
    const int pos = (int)((A.pos4 >> (4 * k)) & 15), limb = (int)((A.limb4 >> (4 * k)) & 15);
    const AR ar(A.lt + limb);
    const int chunk0 = blockIdx.x * kBK;
    const TW* tw = (const TW*)A.tw + ((size_t)limb << A.logN);
    const unsigned m0 = 1u << A.a;
    const int t = threadIdx.x >> 6, ch = (threadIdx.x >> 4) & 3, j = threadIdx.x & 15;
    const int ntiles = (groups + kBPG - 1) / kBPG;
    // a CTA walks tiles blockIdx.z, blockIdx.z + gridDim.z, ..: the twiddles are staged once, and the words of the next
    // tile are already in flight while the current one is transformed
    int yg = blockIdx.z;
    const long long tile_stride = (long long)kBPG * A.period * A.stride;  // words between the same polynomial slot of two tiles
    u64* base = A.data + (((long long)yg * kBPG + t) * A.period + pos) * A.stride + ((size_t)(chunk0 + ch) << 8);
    u64 raw[16];
    if ((long long)yg * kBPG + t < groups) {
#pragma unroll
        for (int e = 0; e < 16; e++) raw[e] = base[j + 16 * e];
    }
    for (int i = threadIdx.x; i < kBK * 256; i += 256) {
        const int c2 = i >> 8, e = i & 255;
        if (e < 15) {
            const int st = 31 - __clz(e + 1), il = e + 1 - (1 << st);
            tc[i] = tw[((m0 + (unsigned)(chunk0 + c2)) << st) + il];
        } else if (e >= 16) {
            const int jj = e & 15, r = (e >> 4) - 1;           // r = 2^u - 1 + il'
            const int u = 31 - __clz(r + 1), il = r + 1 - (1 << u);
            tc[i] = tw[((m0 + (unsigned)(chunk0 + c2)) << (4 + u)) + (jj << u) + il];
        }
    }
    __syncthreads();
    const TW* tcc = tc + ch * 256;
    u64* s1 = sm + (t * kBK + ch) * 272;
    for (; yg < ntiles; yg += gridDim.z) {
        const bool valid = (long long)yg * kBPG + t < groups;
        const int yn = yg + gridDim.z;
        u64 nxt[16];
        if (yn < ntiles && (long long)yn * kBPG + t < groups) {
            const u64* nb = base + (long long)gridDim.z * tile_stride;
#pragma unroll
            for (int e = 0; e < 16; e++) nxt[e] = nb[j + 16 * e];
        }
        if (valid) {
            typename AR::T x[16];
#pragma unroll
            for (int e = 0; e < 16; e++) x[e] = ar.from_mid(raw[e]);
            fwd_round_f<4, AR, 4>(ar, x, [=](int st, int il) { return tcc[(1 << st) - 1 + il]; });
#pragma unroll
            for (int e = 0; e < 16; e++) s1[17 * e + j] = ar.to_exch(x[e]);
        }
        __syncwarp();  // the exchange tile of a chunk is private to the 16 lanes that transform it
        if (valid) {
            typename AR::T x[16];
#pragma unroll
            for (int e = 0; e < 16; e++) x[e] = ar.from_mid(s1[17 * j + e]);
            fwd_round_f<4, AR, 1>(ar, x, [=](int u, int il) { return tcc[(((1 << u) + il) << 4) + j]; });
            // logical position 16 j + e goes to word 16 e + j of the chunk (nibble-swapped layout): the 16 threads of a
            // chunk write 128 contiguous bytes per store
#pragma unroll
            for (int e = 0; e < 16; e++) base[16 * e + j] = ar.to_canonical(x[e]);
        }
        __syncwarp();  // round 2 has read the exchange tile; the next tile may overwrite it
#pragma unroll
        for (int e = 0; e < 16; e++) raw[e] = nxt[e];
        base += (long long)gridDim.z * tile_stride;
    }
}

// The same pass with the words brought in by bulk asynchronous copies.  A warp owns the two chunks of ONE polynomial
// (4 KiB, contiguous in memory) and runs its own two-deep pipeline: lane 0 starts the copy of the warp's tile after next
// into the buffer the warp has just finished with, completion is signalled on a per-buffer mbarrier, and no warp ever
// waits for another (the only CTA-wide barrier follows the staging of the twiddles).  The prefetched words therefore
// occupy no registers.  The two rounds exchange IN PLACE in the landing buffer: position 16 r + c of a chunk is kept at
// word 16 r + (c ^ r), which makes the column reads and writes of round 1 and the row reads of round 2 conflict-free
// without padding.  Every wait on an mbarrier is bounded; a warp whose wait runs out raises the context's kernel flag
// and stops.
constexpr int kTK = 2, kTP = 8;       // chunks per CTA, polynomials per tile (= warps per CTA)
template <class AR>
__device__ __forceinline__ void fwd_b8t_body(const NttArgs& A, int groups, int* kflag, int k, u64* smraw) {
    typedef typename AR::TW TW;
    TW* tc = (TW*)smraw;                                 // twiddle cache [kTK][256], layout as in k_ntt_fwd_b8
    u64* bufs = smraw + kTK * 256 * 2;                   // [kTP][2][512] landing / exchange buffers
    u64* bars = bufs + kTP * 2 * 512;                    // [kTP][2] mbarriers
    const int pos = (int)((A.pos4 >> (4 * k)) & 15), limb = (int)((A.limb4 >> (4 * k)) & 15);
    const AR ar(A.lt + limb);
    const int chunk0 = blockIdx.x * kTK;
    const TW* tw = (const TW*)A.tw + ((size_t)limb << A.logN);
    const unsigned m0 = 1u << A.a;
    const int t = threadIdx.x >> 5, lane = threadIdx.x & 31, ch = lane >> 4, j = lane & 15;
    const int ntiles = (groups + kTP - 1) / kTP;
    const long long tile_stride = (long long)kTP * A.period * A.stride;
    u64* wbuf = bufs + t * 1024;
    const unsigned bar0 = smem_addr(bars + t * 2), buf0 = smem_addr(wbuf);
    if (lane == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    // tiles of this CTA: blockIdx.z, blockIdx.z + gridDim.z, ..; this warp's polynomial in tile yg is yg * kTP + t
    const int yg0 = blockIdx.z, ystep = gridDim.z;
    u64* gbase = A.data + (((long long)yg0 * kTP + t) * A.period + pos) * A.stride + ((size_t)chunk0 << 8);
    const int my_tiles = yg0 < ntiles ? (ntiles - yg0 + ystep - 1) / ystep : 0;
    // tile i of this warp is valid when its polynomial exists (only the last tile can be ragged)
    auto tile_valid = [&](int i) { return i < my_tiles && (long long)(yg0 + (long long)i * ystep) * kTP + t < groups; };
    if (lane == 0) {
        for (int i = 0; i < 2; i++)
            if (tile_valid(i)) {
                mbar_expect_tx(bar0 + 8 * i, 4096);
                bulk_load(buf0 + 4096 * i, gbase + (long long)i * ystep * tile_stride, 4096, bar0 + 8 * i);
            }
    }
    for (int i = threadIdx.x; i < kTK * 256; i += 256) {
        const int c2 = i >> 8, e = i & 255;
        if (e < 15) {
            const int st = 31 - __clz(e + 1), il = e + 1 - (1 << st);
            tc[i] = tw[((m0 + (unsigned)(chunk0 + c2)) << st) + il];
        } else if (e >= 16) {
            const int jj = e & 15, r = (e >> 4) - 1;
            const int u = 31 - __clz(r + 1), il = r + 1 - (1 << u);
            tc[i] = tw[((m0 + (unsigned)(chunk0 + c2)) << (4 + u)) + (jj << u) + il];
        }
    }
    __syncthreads();
    const TW* tcc = tc + ch * 256;
    for (int i = 0; i < my_tiles; i++) {
        if (!tile_valid(i)) break;  // warp-uniform
        const int s = i & 1;
        if (!mbar_wait(bar0 + 8 * s, (unsigned)(i >> 1) & 1u)) {
            if (lane == 0) raise_flag(kflag);
            // the copy into the other buffer may still be in flight: give it the same bounded time, then stop
            if (tile_valid(i + 1)) mbar_wait(bar0 + 8 * (s ^ 1), (unsigned)((i + 1) >> 1) & 1u);
            return;
        }
        u64* sb = wbuf + s * 512 + ch * 256;
        typename AR::T x[16];
#pragma unroll
        for (int e = 0; e < 16; e++) x[e] = ar.from_mid(sb[j + 16 * e]);
        __syncwarp();  // every lane holds its words: the buffer may be overwritten
        fwd_round_f<4, AR, 4>(ar, x, [=](int st, int il) { return tcc[(1 << st) - 1 + il]; });
#pragma unroll
        for (int e = 0; e < 16; e++) sb[16 * e + (j ^ e)] = ar.to_exch(x[e]);
        __syncwarp();
#pragma unroll
        for (int e = 0; e < 16; e++) x[e] = ar.from_mid(sb[16 * j + (e ^ j)]);
        fwd_round_f<4, AR, 1>(ar, x, [=](int u, int il) { return tcc[(((1 << u) + il) << 4) + j]; });
        u64* go = gbase + (long long)i * ystep * tile_stride + ((size_t)ch << 8);
#pragma unroll
        for (int e = 0; e < 16; e++) go[16 * e + j] = ar.to_canonical(x[e]);
        // order this warp's shared-memory accesses before the asynchronous copy that refills the buffer
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0 && tile_valid(i + 2)) {
            mbar_expect_tx(bar0 + 8 * s, 4096);
            bulk_load(buf0 + 4096 * s, gbase + (long long)(i + 2) * ystep * tile_stride, 4096, bar0 + 8 * s);
        }
    }
}

template <class AR>
__global__ void __launch_bounds__(256, 3) k_ntt_fwd_b8t(NttArgs A, int groups, int* kflag) {
    extern __shared__ __align__(128) u64 smraw[];
    fwd_b8t_body<AR>(A, groups, kflag, blockIdx.y, smraw);
}

// One launch for the two arithmetic classes of a batch over {q_0 .. q_{L-1}, p} (binary64 limbs and the special prime's
// Harvey integers): the selections of the integer class follow those of the binary64 class along blockIdx.y.  Saves a
// launch per key switch, which matters on levels of one or two blocks.
__global__ void __launch_bounds__(256, 3) k_ntt_fwd_b8t_mixed(NttArgs Af, NttArgs Ai, int groups, int* kflag) {
    extern __shared__ __align__(128) u64 smraw[];
    if ((int)blockIdx.y < Af.nsel) fwd_b8t_body<ArithF64>(Af, groups, kflag, blockIdx.y, smraw);
    else fwd_b8t_body<ArithInt<false>>(Ai, groups, kflag, blockIdx.y - Af.nsel, smraw);
}

// Inverse pass B' (spans 1 .. 128 inside chunks, the first pass of an inverse transform) in the same form: bulk copies
// into per-warp buffers, in-place swizzled exchange, no CTA-wide barrier in the loop.  Input canonical residues in the
// nibble-swapped layout (word 16 e + j holds logical position 16 j + e), output in the private format of the modulus at
// natural positions, as the second inverse pass (k_ntt_inv_a, k_ks_lift) expects.
template <class AR>
__global__ void __launch_bounds__(256, 3) k_ntt_inv_b8t(NttArgs A, int groups, int* kflag) {
    extern __shared__ __align__(128) u64 smraw[];
    typedef typename AR::TW TW;
    // twiddle cache [kTK][256]: stage s of a round of four uses table entries (base << (3 - s)) + il, il < 2^(3 - s); they
    // are kept at row r = 16 - (16 >> s) + il.  Entries 0..14: second round (base = m0 + chunk, read by all 16 lanes of a
    // chunk at once); entries 16 (r + 1) + j: first round of lane j (base = ((m0 + chunk) << 4) + j).
    TW* tc = (TW*)smraw;
    u64* bufs = smraw + kTK * 256 * 2;
    u64* bars = bufs + kTP * 2 * 512;
    const int k = blockIdx.y;
    const int pos = (int)((A.pos4 >> (4 * k)) & 15), limb = (int)((A.limb4 >> (4 * k)) & 15);
    const AR ar(A.lt + limb);
    const int chunk0 = blockIdx.x * kTK;
    const TW* tw = (const TW*)A.tw + ((size_t)limb << A.logN);
    const unsigned m0 = 1u << A.a;
    const int t = threadIdx.x >> 5, lane = threadIdx.x & 31, ch = lane >> 4, j = lane & 15;
    const int ntiles = (groups + kTP - 1) / kTP;
    const long long tile_stride = (long long)kTP * A.period * A.stride;
    u64* wbuf = bufs + t * 1024;
    const unsigned bar0 = smem_addr(bars + t * 2), buf0 = smem_addr(wbuf);
    if (lane == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const int yg0 = blockIdx.z, ystep = gridDim.z;
    u64* gbase = A.data + (((long long)yg0 * kTP + t) * A.period + pos) * A.stride + ((size_t)chunk0 << 8);
    // source of the copies: the same words, or a separately laid out input (group stride src_gstride)
    const u64* sbase = A.src ? A.src + ((long long)yg0 * kTP + t) * A.src_gstride + (long long)pos * A.stride + ((size_t)chunk0 << 8) : gbase;
    const long long stile_stride = A.src ? (long long)kTP * A.src_gstride : (long long)kTP * A.period * A.stride;
    const int my_tiles = yg0 < ntiles ? (ntiles - yg0 + ystep - 1) / ystep : 0;
    auto tile_valid = [&](int i) { return i < my_tiles && (long long)(yg0 + (long long)i * ystep) * kTP + t < groups; };
    if (lane == 0) {
        for (int i = 0; i < 2; i++)
            if (tile_valid(i)) {
                mbar_expect_tx(bar0 + 8 * i, 4096);
                bulk_load(buf0 + 4096 * i, sbase + (long long)i * ystep * stile_stride, 4096, bar0 + 8 * i);
            }
    }
    for (int i = threadIdx.x; i < kTK * 256; i += 256) {
        const int c2 = i >> 8, e = i & 255;
        const unsigned cbase = m0 + (unsigned)(chunk0 + c2);
        const int r = e < 16 ? e : (e >> 4) - 1;  // row 0..14 (e == 15 and rows above 14 are unused)
        if (r < 15 && (e < 15 || e >= 16)) {
            int st = 0;
            while (16 - (16 >> (st + 1)) <= r) st++;
            const int il = r - (16 - (16 >> st));
            const unsigned base = e < 16 ? cbase : (cbase << 4) + (unsigned)(e & 15);
            tc[i] = tw[(base << (3 - st)) + il];
        }
    }
    __syncthreads();
    const TW* tcc = tc + ch * 256;
    for (int i = 0; i < my_tiles; i++) {
        if (!tile_valid(i)) break;  // warp-uniform
        const int s = i & 1;
        if (!mbar_wait(bar0 + 8 * s, (unsigned)(i >> 1) & 1u)) {
            if (lane == 0) raise_flag(kflag);
            if (tile_valid(i + 1)) mbar_wait(bar0 + 8 * (s ^ 1), (unsigned)((i + 1) >> 1) & 1u);
            return;
        }
        u64* sb = wbuf + s * 512 + ch * 256;
        typename AR::T x[16];
#pragma unroll
        for (int e = 0; e < 16; e++) x[e] = ar.inv_input(sb[16 * e + j]);  // logical positions 16 j + e
        __syncwarp();
        inv_round_f<4>(ar, x, [=](int st, int il) { return tcc[((16 - (16 >> st) + il + 1) << 4) + j]; });
#pragma unroll
        for (int e = 0; e < 16; e++) sb[16 * j + (e ^ j)] = ar.to_mid(x[e]);
        __syncwarp();
#pragma unroll
        for (int e = 0; e < 16; e++) x[e] = ar.from_mid(sb[16 * e + (j ^ e)]);  // logical positions j + 16 e
        inv_round_f<4>(ar, x, [=](int st, int il) { return tcc[16 - (16 >> st) + il]; });
        u64* go = gbase + (long long)i * ystep * tile_stride + ((size_t)ch << 8);
#pragma unroll
        for (int e = 0; e < 16; e++) go[j + 16 * e] = ar.to_mid(x[e]);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0 && tile_valid(i + 2)) {
            mbar_expect_tx(bar0 + 8 * s, 4096);
            bulk_load(buf0 + 4096 * s, sbase + (long long)(i + 2) * ystep * stile_stride, 4096, bar0 + 8 * s);
        }
    }
}

// Self-test of the bounded wait: one warp waits on an mbarrier that nothing ever completes, for limit_ns; the wait must
// run out, raise the kernel flag and return -- the error path every bulk-copy kernel takes if a copy never arrives.
__global__ void k_wait_selftest(int* kflag, unsigned long long limit_ns, unsigned long long* waited_ns) {
    __shared__ __align__(8) u64 bar;
    const unsigned b = smem_addr(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const unsigned long long t0 = global_ns();
    const bool arrived = mbar_wait(b, 0, limit_ns);
    if (threadIdx.x == 0) {
        *waited_ns = global_ns() - t0;
        if (!arrived) raise_flag(kflag);
    }
}

// ---- inverse pass B': spans 1 .. S/2 inside contiguous chunks (mirror of forward pass B) -----------------------

template <int R1, int R2, class AR>
__device__ __forceinline__ void inv_b_body(const NttArgs& A, const AR ar, u64* __restrict__ base, int chunk0,
                                           const typename AR::TW* __restrict__ tw, int final_scale, u64* __restrict__ sm) {
    constexpr int S = 1 << (R1 + R2), J1 = 1 << R2, SP = R2 == 0 ? S : S + (S >> R2);
    constexpr int RR2 = R2 == 0 ? 1 : R2;
    constexpr int J2 = 1 << R1;
    const int K = A.K;
    const unsigned m0 = 1u << A.a;
    const typename AR::TW ninv = ar.ninv;
    if (R2 != 0) {
        // memory word idx of a chunk is logical position idx (or its nibble swap, on rings that store chunks that way)
        for (int idx = threadIdx.x; idx < K * S; idx += kThreads) {
            const int p = idx % S;
            sm[(idx / S) * SP + pad<R2>(A.tau ? swap_nibbles(p) : p)] = base[idx];
        }
        __syncthreads();
        for (int w = threadIdx.x; w < K * J2; w += kThreads) {
            const int ch = w / J2, j = w % J2;
            u64* s = sm + ch * SP + pad<R2>(j << RR2);
            typename AR::T x[1 << RR2];
#pragma unroll
            for (int e = 0; e < (1 << RR2); e++) x[e] = ar.inv_input(s[e]);
            inv_round<RR2>(ar, x, tw, ((m0 + (unsigned)(chunk0 + ch)) << R1) + (unsigned)j);
#pragma unroll
            for (int e = 0; e < (1 << RR2); e++) s[e] = ar.to_mid(x[e]);
        }
        __syncthreads();
    }
    for (int w = threadIdx.x; w < K * J1; w += kThreads) {
        const int ch = w / J1, j = w % J1;
        u64* p = base + (size_t)ch * S;
        typename AR::T x[1 << R1];
#pragma unroll
        for (int e = 0; e < (1 << R1); e++) x[e] = R2 == 0 ? ar.inv_input(p[j + J1 * e]) : ar.from_mid(sm[ch * SP + pad<R2>(j + J1 * e)]);
        inv_round<R1>(ar, x, tw, m0 + (unsigned)(chunk0 + ch));
#pragma unroll
        for (int e = 0; e < (1 << R1); e++) p[j + J1 * e] = final_scale ? ar.scaled_output(x[e], ninv) : ar.to_mid(x[e]);
    }
}

template <int R1, int R2, class AR>
__global__ void __launch_bounds__(kThreads, AR::kMinBlocks) k_ntt_inv_b(NttArgs A, int final_scale) {
    extern __shared__ u64 sm[];
    const Sel sel = select(A);
    const AR ar(A.lt + sel.limb);
    const int chunk0 = blockIdx.x * A.K;
    u64* base = A.data + sel.poly * A.stride + ((size_t)chunk0 << (R1 + R2));
    inv_b_body<R1, R2>(A, ar, base, chunk0, (const typename AR::TW*)A.tw + ((size_t)sel.limb << A.logN), final_scale, sm);
}

// ---- inverse pass A': spans S .. N/2 (mirror of forward pass A), then the N^{-1} scaling ------------------------

template <int R1, int R2, class AR>
__device__ __forceinline__ void inv_a_body(const NttArgs& A, const AR ar, u64* __restrict__ base,
                                           const typename AR::TW* __restrict__ tw, u64* __restrict__ sm) {
    const int S = 1 << A.b, logC = A.logC, C = 1 << logC;
    constexpr int G1 = 1 << R2, G2 = 1 << R1;
    constexpr int RR2 = R2 == 0 ? 1 : R2;
    const typename AR::TW ninv = ar.ninv;
    if (R2 != 0) {
        for (int w = threadIdx.x; w < (G2 << logC); w += kThreads) {
            const int c = w & (C - 1), g = w >> logC;
            typename AR::T x[1 << RR2];
#pragma unroll
            for (int e = 0; e < (1 << RR2); e++) x[e] = ar.from_mid(base[(size_t)((g << RR2) + e) * S + c]);
            inv_round<RR2>(ar, x, tw, (unsigned)(G2 + g));
#pragma unroll
            for (int e = 0; e < (1 << RR2); e++) sm[(((g << RR2) + e) << logC) + c] = ar.to_mid(x[e]);
        }
        __syncthreads();
    }
    for (int w = threadIdx.x; w < (G1 << logC); w += kThreads) {
        const int c = w & (C - 1), g = w >> logC;
        typename AR::T x[1 << R1];
#pragma unroll
        for (int e = 0; e < (1 << R1); e++) x[e] = ar.from_mid(R2 == 0 ? base[(size_t)(g + G1 * e) * S + c] : sm[((g + G1 * e) << logC) + c]);
        inv_round<R1>(ar, x, tw, 1u);
#pragma unroll
        for (int e = 0; e < (1 << R1); e++) base[(size_t)(g + G1 * e) * S + c] = ar.scaled_output(x[e], ninv);
    }
}

template <int R1, int R2, class AR>
__global__ void __launch_bounds__(kThreads, AR::kMinBlocks) k_ntt_inv_a(NttArgs A) {
    extern __shared__ u64 sm[];
    const Sel sel = select(A);
    const AR ar(A.lt + sel.limb);
    u64* base = A.data + sel.poly * A.stride + ((long long)blockIdx.x << A.logC);
    inv_a_body<R1, R2>(A, ar, base, (const typename AR::TW*)A.tw + ((size_t)sel.limb << A.logN), sm);
}

// ---- fused key-switch step: inverse pass A' + centred lift + forward pass A for several target moduli -----------------
//
// Both the digit decomposition (ModUp) and ModDown take a polynomial back to coefficients, lift every coefficient to a
// centred integer and re-reduce it into other moduli, whose forward transforms follow.  The last inverse round leaves a
// thread with rows g + G1*e of its column -- exactly the words the first forward round needs -- so the lift and pass A of
// all target transforms run from registers; the coefficient-domain polynomials never travel to memory.

struct LiftArgs {
    u64* src;             // source polynomials after inverse pass B' (private format of their modulus)
    long long src_stride;
    int src_period;
    u64 src_limb4;        // limb of source polynomial sp = nibble (sp % src_period)
    u64* dst;             // target polynomial (sp, ti) at dst + (sp * n_tgt + ti) * N, in forward pass-A output format
    int n_tgt, tgt_limb0;
    int logN;
    const void *tw_inv_int, *tw_inv_f64, *tw_fwd_int, *tw_fwd_f64;
    const LimbConst* lt;
};

template <int R1, int R2, class AR>
__device__ __forceinline__ void lift_inverse(const LiftArgs& A, const AR ar, const typename AR::TW* __restrict__ tw, const u64* __restrict__ base,
                                             u64* __restrict__ sm, int g, int c, bool active, u64 (&v)[1 << R1]) {
    constexpr int G1 = 1 << R2, G2 = 1 << R1;
    constexpr int RR2 = R2 == 0 ? 1 : R2;
    const typename AR::TW ninv = ar.ninv;
    if (R2 != 0) {
        for (int w = threadIdx.x; w < (G2 << 4); w += blockDim.x) {
            const int cc = w & 15, gg = w >> 4;
            typename AR::T x[1 << RR2];
#pragma unroll
            for (int e = 0; e < (1 << RR2); e++) x[e] = ar.from_mid(base[(size_t)((gg << RR2) + e) * 256 + cc]);
            inv_round<RR2>(ar, x, tw, (unsigned)(G2 + gg));
#pragma unroll
            for (int e = 0; e < (1 << RR2); e++) sm[(((gg << RR2) + e) << 4) + cc] = ar.to_mid(x[e]);
        }
        __syncthreads();
    }
    if (active) {
        typename AR::T x[1 << R1];
#pragma unroll
        for (int e = 0; e < (1 << R1); e++) x[e] = ar.from_mid(R2 == 0 ? base[(size_t)(g + G1 * e) * 256 + c] : sm[((g + G1 * e) << 4) + c]);
        inv_round<R1>(ar, x, tw, 1u);
#pragma unroll
        for (int e = 0; e < (1 << R1); e++) v[e] = ar.scaled_output(x[e], ninv);
    }
}

__device__ __forceinline__ double lifted_value(const ArithF64& ar, u64 r, bool neg, u64 q) {
    const double d = ar.from_canonical(r);
    return neg ? -d : d;
}
template <bool S>
__device__ __forceinline__ u64 lifted_value(const ArithInt<S>&, u64 r, bool neg, u64 q) { return (neg && r) ? q - r : r; }

template <int R1, int R2, class AR>
__device__ __forceinline__ void lift_forward(const AR ar, const LimbConst* lc, bool same_modulus, const typename AR::TW* __restrict__ tw,
                                             u64* __restrict__ base, u64* __restrict__ sm, int g, int c, bool active,
                                             const u64 (&v)[1 << R1], u64 src_q, u64 src_half) {
    constexpr int G1 = 1 << R2, G2 = 1 << R1;
    constexpr int RR2 = R2 == 0 ? 1 : R2;
    if (active) {
        typename AR::T x[1 << R1];
#pragma unroll
        for (int e = 0; e < (1 << R1); e++) {
            // centred lift of the coefficient (sign and magnitude), reduced into this modulus
            const bool neg = v[e] > src_half;
            const u64 mag = neg ? src_q - v[e] : v[e];
            x[e] = same_modulus ? ar.from_canonical(v[e]) : lifted_value(ar, barrett64(mag, *lc), neg, lc->q);
        }
        fwd_round<R1, AR, R1>(ar, x, tw, 1u);
#pragma unroll
        for (int e = 0; e < (1 << R1); e++) {
            if (R2 == 0) base[(size_t)(g + G1 * e) * 256 + c] = ar.to_mid(x[e]);
            else sm[((g + G1 * e) << 4) + c] = ar.to_mid(x[e]);
        }
    }
    if (R2 != 0) {
        __syncthreads();
        for (int w = threadIdx.x; w < (G2 << 4); w += blockDim.x) {
            const int cc = w & 15, gg = w >> 4;
            typename AR::T x[1 << RR2];
#pragma unroll
            for (int e = 0; e < (1 << RR2); e++) x[e] = ar.from_mid(sm[(((gg << RR2) + e) << 4) + cc]);
            fwd_round<RR2, AR, RR2>(ar, x, tw, (unsigned)(G2 + gg));
#pragma unroll
            for (int e = 0; e < (1 << RR2); e++) base[(size_t)((gg << RR2) + e) * 256 + cc] = ar.to_mid(x[e]);
        }
        __syncthreads();  // the exchange tile is free for the next target
    }
}

template <int R1, int R2>
__global__ void __launch_bounds__(256, 2) k_ks_lift(LiftArgs A) {
    extern __shared__ u64 sm[];
    constexpr int G1 = 1 << R2;
    const int N = 1 << A.logN;
    const long long sp = blockIdx.y;
    const int c0 = blockIdx.x << 4;
    const int c = threadIdx.x & 15, g = threadIdx.x >> 4;
    const bool active = g < G1;
    const int sl = (int)((A.src_limb4 >> (4 * (sp % A.src_period))) & 15);
    const LimbConst* slc = A.lt + sl;
    const u64* sbase = A.src + sp * A.src_stride + c0;
    u64 v[1 << R1];
    if (slc->q < (1ULL << 50)) {
        const ArithF64 ar(slc);
        lift_inverse<R1, R2>(A, ar, (const double2*)A.tw_inv_f64 + ((size_t)sl << A.logN), sbase, sm, g, c, active, v);
    } else {
        const ArithInt<false> ar(slc);
        lift_inverse<R1, R2>(A, ar, (const ulonglong2*)A.tw_inv_int + ((size_t)sl << A.logN), sbase, sm, g, c, active, v);
    }
    if (R2 != 0) __syncthreads();  // every thread is done with the exchange tile of the inverse rounds
    // a launch too small to fill the machine is cut along the targets as well: gridDim.z CTAs repeat the inverse rounds and
    // share out the targets, which shortens the chain one CTA runs
    for (int ti = blockIdx.z; ti < A.n_tgt; ti += gridDim.z) {
        const int tl = A.tgt_limb0 + ti;
        const LimbConst* tlc = A.lt + tl;
        u64* dbase = A.dst + (sp * A.n_tgt + ti) * (long long)N + c0;
        if (tlc->q < (1ULL << 50)) {
            const ArithF64 ar(tlc);
            lift_forward<R1, R2>(ar, tlc, tl == sl, (const double2*)A.tw_fwd_f64 + ((size_t)tl << A.logN), dbase, sm, g, c, active, v, slc->q, slc->half);
        } else if (tlc->q < (1ULL << 57)) {
            const ArithInt<true> ar(tlc);
            lift_forward<R1, R2>(ar, tlc, tl == sl, (const ulonglong2*)A.tw_fwd_int + ((size_t)tl << A.logN), dbase, sm, g, c, active, v, slc->q, slc->half);
        } else {
            const ArithInt<false> ar(tlc);
            lift_forward<R1, R2>(ar, tlc, tl == sl, (const ulonglong2*)A.tw_fwd_int + ((size_t)tl << A.logN), dbase, sm, g, c, active, v, slc->q, slc->half);
        }
    }
}

typedef void (*KernLift)(LiftArgs);
KernLift pick_lift(int a) {
    switch (a) {
        case 1: return k_ks_lift<1, 0>;
        case 2: return k_ks_lift<2, 0>;
        case 3: return k_ks_lift<3, 0>;
        case 4: return k_ks_lift<4, 0>;
        case 5: return k_ks_lift<4, 1>;
        case 6: return k_ks_lift<4, 2>;
        case 7: return k_ks_lift<4, 3>;
        default: return k_ks_lift<4, 4>;
    }
}

// ---- dispatch ----------------------------------------------------------------------------------------------------

typedef void (*KernA)(NttArgs);
typedef void (*KernIB)(NttArgs, int);

// stages of a pass -> (R1, R2): one round up to 4 stages, else a round of 4 and a round of the rest
#define PICK_TABLE(NAME, KERN, TYPE)                                                                                   \
    template <class AR>                                                                                               \
    TYPE NAME(int stages) {                                                                                           \
        switch (stages) {                                                                                             \
            case 1: return KERN<1, 0, AR>;                                                                            \
            case 2: return KERN<2, 0, AR>;                                                                            \
            case 3: return KERN<3, 0, AR>;                                                                            \
            case 4: return KERN<4, 0, AR>;                                                                            \
            case 5: return KERN<4, 1, AR>;                                                                            \
            case 6: return KERN<4, 2, AR>;                                                                            \
            case 7: return KERN<4, 3, AR>;                                                                            \
            default: return KERN<4, 4, AR>;                                                                           \
        }                                                                                                             \
    }
PICK_TABLE(pick_fwd_a, k_ntt_fwd_a, KernA)
PICK_TABLE(pick_fwd_b, k_ntt_fwd_b, KernA)
PICK_TABLE(pick_inv_a, k_ntt_inv_a, KernA)
PICK_TABLE(pick_inv_b, k_ntt_inv_b, KernIB)

// arithmetic class of a modulus: 0 binary64, 1 lazy integers, 2 Harvey integers
int arith_class(u64 q, bool inverse) {
    if (q < (1ULL << 50)) return 0;
    if (!inverse && q < (1ULL << 57)) return 1;
    return 2;
}

size_t smem_a(const NttArgs& A) { return A.a > 4 ? ((size_t)8 << (A.a + A.logC)) : 0; }
size_t smem_b(const NttArgs& A) {
    if (A.b <= 4) return 0;
    const int S = 1 << A.b, R2 = A.b - 4;
    return (size_t)A.K * (S + (S >> R2)) * 8;
}

bool b8t_eligible(const hann_ctx* c, const NttArgs& A) {
#ifndef HANN_NO_B8T
    return A.b == 8 && A.a > 0 && A.tau && ((c->N >> 8) % kTK) == 0 && ((uintptr_t)A.data & 15) == 0 && (A.stride & 1) == 0;
#else
    (void)c; (void)A;
    return false;
#endif
}
constexpr size_t kB8tSmem = (size_t)kTK * 256 * 16 + (size_t)kTP * 2 * 512 * 8 + (size_t)kTP * 2 * 8;
// tiles per CTA: a CTA stages its twiddles once and its warps prefetch two tiles ahead, but the grid should still fill whole
// waves of the 148 x 3 resident CTAs.  Smallest (waves x (tiles per CTA + staging)), ties to fewer CTAs.
int b8t_zsplit(int per, int ntiles) {
    const int slots = 148 * 3;
    int zs = 1;
    long best = -1;
    for (int z = 1; z <= ntiles && z <= 64; z++) {
        const long waves = ((long)per * z + slots - 1) / slots, tiles = (ntiles + z - 1) / z;
        const long cost = waves * (4 * tiles + 1);
        if (best < 0 || cost < best) {
            best = cost;
            zs = z;
        }
    }
    return zs;
}

// pass B of a batch whose limbs fall into the binary64 class (Af) and the Harvey integer class (Ai): one launch
void launch_fwd_b8t_mixed(hann_ctx* c, const NttArgs& Af, const NttArgs& Ai, int groups) {
    KProf kp(c, KC_NTT_FWD_B);
    cudaFuncSetAttribute(k_ntt_fwd_b8t_mixed, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kB8tSmem);
    const int ranges = (c->N >> 8) / kTK, ntiles = (groups + kTP - 1) / kTP, nsel = Af.nsel + Ai.nsel;
    k_ntt_fwd_b8t_mixed<<<dim3(ranges, nsel, b8t_zsplit(ranges * nsel, ntiles)), 256, kB8tSmem, c->stream>>>(Af, Ai, groups, c->kflag);
}

template <class AR>
void launch_fwd_class(hann_ctx* c, const NttArgs& A, int groups, bool skip_a, bool skip_b = false) {
    if (A.a > 0 && !skip_a) {
        KProf kp(c, KC_NTT_FWD_A);
        pick_fwd_a<AR>(A.a)<<<dim3(1 << (A.b - A.logC), groups * A.nsel), kThreads, smem_a(A), c->stream>>>(A);
    }
    if (skip_b) return;
    KProf kp(c, KC_NTT_FWD_B);
    if (b8t_eligible(c, A)) {
        cudaFuncSetAttribute(k_ntt_fwd_b8t<AR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kB8tSmem);
        const int ranges = ((c->N >> 8) / kTK) >> (A.half ? 1 : 0), ntiles = (groups + kTP - 1) / kTP;
        k_ntt_fwd_b8t<AR><<<dim3(ranges, A.nsel, b8t_zsplit(ranges * A.nsel, ntiles)), 256, kB8tSmem, c->stream>>>(A, groups, c->kflag);
        return;
    }
    if (A.b == 8 && A.a > 0 && A.tau && ((c->N >> 8) % kBK) == 0) {
        const size_t smem = (size_t)kBK * 256 * 16 + (size_t)kBPG * kBK * 272 * 8;
        cudaFuncSetAttribute(k_ntt_fwd_b8<AR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  // 50 KiB > default 48
        // enough CTAs for about four per SM; beyond that a CTA walks several tiles and reuses its staged twiddles
        const int ranges = (c->N >> 8) / kBK, ntiles = (groups + kBPG - 1) / kBPG;
        // tiles per CTA: a CTA that walks several tiles stages its twiddles once, but the grid should still fill whole
        // waves of the 148 x 3 resident CTAs.  Pick the split with the smallest (waves x tiles per CTA), ties to fewer CTAs.
        const int slots = 148 * HANN_B8_MINBLOCKS, per = ranges * A.nsel;
        int zs = 1;
        long best = -1;
        for (int z = 1; z <= ntiles && z <= 64; z++) {
            const long waves = ((long)per * z + slots - 1) / slots, tiles = (ntiles + z - 1) / z;
            const long cost = waves * (4 * tiles + 1);  // staging the twiddles costs about a quarter of a tile
            if (best < 0 || cost < best) {
                best = cost;
                zs = z;
            }
        }
        k_ntt_fwd_b8<AR><<<dim3(ranges, A.nsel, zs), 256, smem, c->stream>>>(A, groups);
        return;
    }
    pick_fwd_b<AR>(A.b)<<<dim3((c->N >> A.b) / A.K, groups * A.nsel), kThreads, smem_b(A), c->stream>>>(A);
}

template <class AR>
void launch_inv_class(hann_ctx* c, const NttArgs& A, int groups, bool skip_a) {
    if (A.b == 8 && A.a > 0 && A.tau && ((c->N >> 8) % kTK) == 0 && ((uintptr_t)A.data & 15) == 0 && (A.stride & 1) == 0 &&
        ((uintptr_t)A.src & 15) == 0 && (A.src_gstride & 1) == 0) {
        KProf kp(c, KC_NTT_INV_B);
        const size_t smem = (size_t)kTK * 256 * 16 + (size_t)kTP * 2 * 512 * 8 + (size_t)kTP * 2 * 8;
        cudaFuncSetAttribute(k_ntt_inv_b8t<AR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        const int ranges = (c->N >> 8) / kTK, ntiles = (groups + kTP - 1) / kTP;
        const int slots = 148 * 3, per = ranges * A.nsel;
        int zs = 1;
        long best = -1;
        for (int z = 1; z <= ntiles && z <= 64; z++) {
            const long waves = ((long)per * z + slots - 1) / slots, tiles = (ntiles + z - 1) / z;
            const long cost = waves * (4 * tiles + 1);
            if (best < 0 || cost < best) {
                best = cost;
                zs = z;
            }
        }
        k_ntt_inv_b8t<AR><<<dim3(ranges, A.nsel, zs), 256, smem, c->stream>>>(A, groups, c->kflag);
    } else {
        KProf kp(c, KC_NTT_INV_B);
        pick_inv_b<AR>(A.b)<<<dim3((c->N >> A.b) / A.K, groups * A.nsel), kThreads, smem_b(A), c->stream>>>(A, A.a == 0 ? 1 : 0);
    }
    if (A.a > 0 && !skip_a) {
        KProf kp(c, KC_NTT_INV_A);
        pick_inv_a<AR>(A.a)<<<dim3(1 << (A.b - A.logC), groups * A.nsel), kThreads, smem_a(A), c->stream>>>(A);
    }
}

// npoly polynomials, `stride` words apart, polynomial p using modulus lm.limb[p % lm.period]; npoly must be a multiple of
// the period.  One set of launches per arithmetic class present in the period.
int launch_ntt(hann_ctx* c, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm, bool inverse, bool skip_a = false,
               const u64* src = nullptr, int64_t src_gstride = 0, bool half = false) {
    if (npoly <= 0) return HANN_OK;
    if (npoly % lm.period) {
        c->err = "transform batch is not a whole number of limb periods";
        return HANN_EINVAL;
    }
    NttArgs A;
    A.stride = stride;
    A.logN = c->logN;
    A.b = c->logN < 8 ? c->logN : 8;
    A.a = c->logN - A.b;
    A.logC = A.b < 4 ? A.b : 4;
    const int chunks = c->N >> A.b;
    A.K = chunks < 16 ? chunks : 16;
    A.lt = c->lt_dev;
    A.tau = c->ntt_tau;
    A.src = src;
    A.src_gstride = src_gstride;
    A.period = lm.period;
    A.half = half ? 1 : 0;
    if (half) {
        bool ok = !inverse && skip_a && ntt_fwd_half_available(c, data, stride);
        for (int i = 0; i < lm.period; i++) ok = ok && arith_class(c->mod[(int)lm.limb[i]], false) == 0;
        if (!ok) {
            c->err = "half-size forward pass B needs the bulk-copy kernel and moduli below 2^50";
            return HANN_EINVAL;
        }
    }
    const int64_t groups_total = npoly / lm.period;
    NttArgs Ac[3];
    for (int cls = 0; cls < 3; cls++) {
        Ac[cls] = A;
        NttArgs& X = Ac[cls];
        X.nsel = 0;
        X.pos4 = X.limb4 = 0;
        for (int i = 0; i < lm.period && i < 16; i++)
            if (arith_class(c->mod[(int)lm.limb[i]], inverse) == cls) {
                X.pos4 |= (u64)i << (4 * X.nsel);
                X.limb4 |= (u64)lm.limb[i] << (4 * X.nsel);
                X.nsel++;
            }
        X.tw = cls == 0 ? (const void*)(inverse ? c->tw_inv_f64 : c->tw_fwd_f64) : (const void*)(inverse ? c->tw_inv : c->tw_fwd);
    }
    // forward, binary64 limbs plus the special prime, bulk-copy kernel applicable: pass B of both classes in one launch
    const bool mixed = !inverse && Ac[0].nsel && Ac[2].nsel && !Ac[1].nsel;
    for (int cls = 0; cls < 3; cls++) {
        NttArgs& X = Ac[cls];
        if (!X.nsel) continue;
        const int64_t gmax = 65535 / (mixed ? Ac[0].nsel + Ac[2].nsel : X.nsel);
        for (int64_t g0 = 0; g0 < groups_total; g0 += gmax) {
            const int groups = (int)std::min<int64_t>(gmax, groups_total - g0);
            X.data = data + g0 * lm.period * stride;
            if (src) X.src = src + g0 * src_gstride;
            const bool merge = mixed && b8t_eligible(c, X);
            if (!inverse) {
                if (cls == 0) launch_fwd_class<ArithF64>(c, X, groups, skip_a, merge);
                else if (cls == 1) launch_fwd_class<ArithInt<true>>(c, X, groups, skip_a);
                else {
                    launch_fwd_class<ArithInt<false>>(c, X, groups, skip_a, merge);
                    if (merge) {
                        Ac[0].data = X.data;
                        launch_fwd_b8t_mixed(c, Ac[0], X, groups);
                    }
                }
            } else {
                if (cls == 0) launch_inv_class<ArithF64>(c, X, groups, skip_a);
                else launch_inv_class<ArithInt<false>>(c, X, groups, skip_a);
            }
        }
    }
    return check_launch(c, inverse ? "ntt_inv" : "ntt_fwd");
}

}  // namespace

LimbMap limbmap_q(const hann_ctx* c) {
    LimbMap m;
    m.period = c->L;
    for (int i = 0; i < c->L; i++) m.limb[i] = (signed char)i;
    return m;
}
LimbMap limbmap_qp(const hann_ctx* c) {
    LimbMap m;
    m.period = c->L + 1;
    for (int i = 0; i <= c->L; i++) m.limb[i] = (signed char)i;
    return m;
}
LimbMap limbmap_first(int nlimbs) {
    LimbMap m;
    m.period = nlimbs;
    for (int i = 0; i < nlimbs; i++) m.limb[i] = (signed char)i;
    return m;
}
LimbMap limbmap_single(int limb) {
    LimbMap m;
    m.period = 1;
    m.limb[0] = (signed char)limb;
    return m;
}

int launch_ntt_fwd(hann_ctx* c, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm) {
    return launch_ntt(c, data, npoly, stride, lm, false);
}

// second half of a forward transform whose pass A was done by another kernel (the fused encoder): the words are in
// the limb's pass-A output format
int launch_ntt_fwd_pass_b(hann_ctx* c, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm) {
    return launch_ntt(c, data, npoly, stride, lm, false, true);
}

// The same for polynomials fixed by X -> 1/X (encodings of real slot vectors), whose values at psi^(2t+1) and at its
// inverse coincide, i.e. position t and position N - 1 - t of the transform: only the first N/2 values are computed and
// kept.  Pass A left out rows 2^(a-1) .. 2^a - 1; polynomial p occupies data + p * stride .. + N/2.
bool ntt_fwd_half_available(const hann_ctx* c, const void* data, int64_t stride) {
#ifndef HANN_NO_B8T
    return c->logN >= 10 && c->ntt_tau && ((c->N >> 8) % (2 * kTK)) == 0 && ((uintptr_t)data & 15) == 0 && (stride & 1) == 0;
#else
    (void)c; (void)data; (void)stride;
    return false;
#endif
}
int launch_ntt_fwd_pass_b_half(hann_ctx* c, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm) {
    return launch_ntt(c, data, npoly, stride, lm, false, true, nullptr, 0, true);
}

namespace {
// full[p][t] = half[p][t < N/2 ? t : N - 1 - t]
__global__ void __launch_bounds__(kThreads) k_unpack_half(const u64* __restrict__ half, u64* __restrict__ full, long long npoly, int N) {
    const long long total = npoly * N;
    const int n = N >> 1;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const long long p = idx / N;
        const int t = (int)(idx % N);
        full[idx] = half[p * n + (t < n ? t : N - 1 - t)];
    }
}
}  // namespace

// stored plaintext polynomials (first N/2 transform values each) -> all N values
int launch_unpack_half(hann_ctx* c, const u64* half, int64_t npoly, u64* full) {
    if (npoly <= 0) return HANN_OK;
    const int64_t total = npoly * c->N;
    const int grid = (int)std::min<int64_t>((total + kThreads - 1) / kThreads, 148 * 16);
    k_unpack_half<<<grid, kThreads, 0, c->stream>>>(half, full, npoly, c->N);
    return check_launch(c, "unpack_half");
}

int launch_ntt_inv(hann_ctx* c, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm) {
    return launch_ntt(c, data, npoly, stride, lm, true);
}

bool ks_lift_available(const hann_ctx* c) { return c->logN >= 9; }

// After inverse pass B' of the nsrc source polynomials (launch_ntt_inv_pass_b): finish their inverse transforms, lift the
// coefficients (centred) into the n_tgt moduli tgt_limb0 .. and run pass A of the target transforms.  The caller finishes
// with launch_ntt_fwd_pass_b over the targets.
int launch_ks_lift(hann_ctx* c, u64* src, int64_t src_stride, int64_t nsrc, const LimbMap& src_lm, u64* dst, int n_tgt, int tgt_limb0) {
    if (nsrc <= 0) return HANN_OK;
    LiftArgs A;
    A.src = src;
    A.src_stride = src_stride;
    A.src_period = src_lm.period;
    A.src_limb4 = 0;
    for (int i = 0; i < src_lm.period && i < 16; i++) A.src_limb4 |= (u64)src_lm.limb[i] << (4 * i);
    A.dst = dst;
    A.n_tgt = n_tgt;
    A.tgt_limb0 = tgt_limb0;
    A.logN = c->logN;
    A.tw_inv_int = c->tw_inv;
    A.tw_inv_f64 = c->tw_inv_f64;
    A.tw_fwd_int = c->tw_fwd;
    A.tw_fwd_f64 = c->tw_fwd_f64;
    A.lt = c->lt_dev;
    const int a = c->logN - 8;
    const size_t smem = a > 4 ? (size_t)(1 << a) * 16 * 8 : 0;
    const int threads = a >= 8 ? 256 : (a == 7 ? 128 : 64);
    for (int64_t s0 = 0; s0 < nsrc; s0 += 65535) {
        const int ns = (int)std::min<int64_t>(65535, nsrc - s0);
        // the source limb of polynomial s0 + y is nibble (s0 + y) % period: 65535 is not a multiple of every period, so shift
        LiftArgs Ap = A;
        Ap.src = src + s0 * src_stride;
        Ap.dst = dst + s0 * n_tgt * (int64_t)c->N;
        Ap.src_limb4 = 0;
        for (int i = 0; i < src_lm.period && i < 16; i++) Ap.src_limb4 |= (u64)src_lm.limb[(s0 + i) % src_lm.period] << (4 * i);
        KProf kp(c, KC_LIFT_DIGITS);
        const int zsplit = (16L * ns * n_tgt <= c->lift_split_ctas) ? n_tgt : 1;  // see hann_ctx::lift_split_ctas
        pick_lift(a)<<<dim3(16, ns, zsplit), threads, smem, c->stream>>>(Ap);
    }
    return check_launch(c, "ks_lift");
}

int launch_ntt_inv_pass_b(hann_ctx* c, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm) {
    return launch_ntt(c, data, npoly, stride, lm, true, true);
}

bool ntt_inv_pass_b_gathers(const hann_ctx* c, const void* src, const void* dst) {
#ifndef HANN_NO_B8T
    return c->logN >= 10 && ((c->N >> 8) % kTK) == 0 && (((uintptr_t)src | (uintptr_t)dst) & 15) == 0;
#else
    (void)c; (void)src; (void)dst;
    return false;
#endif
}

// The same with the input read from elsewhere: group g (lm.period polynomials, `stride` words apart) starts at
// src + g * src_gstride; the output goes to data as above.  Only where ntt_inv_pass_b_gathers(c) holds and both pointers are
// 16-byte aligned (the bulk-copy kernel); the caller copies and uses launch_ntt_inv_pass_b otherwise.
int launch_ntt_inv_pass_b_from(hann_ctx* c, const u64* src, int64_t src_gstride, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm) {
    return launch_ntt(c, data, npoly, stride, lm, true, true, src, src_gstride);
}

int launch_wait_selftest(hann_ctx* c, unsigned long long limit_ns, unsigned long long* waited_ns_dev) {
    k_wait_selftest<<<1, 32, 0, c->stream>>>(c->kflag, limit_ns, waited_ns_dev);
    return check_launch(c, "wait_selftest");
}

int ntt_configure(hann_ctx* c) {
    // every configuration stays below the 48 KiB default of dynamic shared memory (pass A: 2^8 rows x 16 columns x 8 B
    // = 32 KiB; pass B: 16 chunks x 272 words x 8 B = 34 KiB), so nothing to opt in to
    (void)c;
    return HANN_OK;
}
