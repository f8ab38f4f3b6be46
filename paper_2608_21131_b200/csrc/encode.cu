// Canonical CKKS encoding on the device: real slot vector -> integer polynomial -> RNS residues.
//
// m_k = rint((Delta/n) * sum_j z_j cos(pi g_j k / N)), g_j = 5^j mod 2N, evaluated as: y[u_j] = z_j with
// u_j = (g_j - 1)/4, a complex FFT of size n, a twist by exp(-i pi k / N), a scaling by the power of two Delta/n,
// round to nearest even.  To give the same bits as any other IEEE binary64 evaluation of the same data-flow graph,
// the FFT is the radix-2 decimation-in-time graph on bit-reversed input with every product and sum rounded
// separately (explicit __dmul_rn / __dadd_rn / __dsub_rn: never contracted into fused multiply-adds), and the
// twiddles are correctly rounded table values.
//
// Two kernels: pass 1 runs the stages that stay inside contiguous chunks of S1 = 2^b1 points (the input gather
// z_j -> position brev(u_j) is folded into its loads); pass 2 runs the remaining stages on column tiles of the
// (n/S1) x S1 matrix view, then twists, rounds, reduces modulo every ciphertext prime and writes residues.
#include "internal.h"
#include "debugcheck.cuh"

namespace {

constexpr int kThreads = 256;

struct EncArgs {
    // input: candidate rows (rows != nullptr) or one slot vector per plaintext (z != nullptr)
    const float* rows;
    long long rows_in_block;
    int dim, R, B;
    const double* z;
    // tables
    const double2* T;
    const double2* U;
    const int32_t* jinv;
    int logn, b1, K1, C1;
    double scale;  // Delta / n
    double2* buf;  // [P][n], indexed by blockIdx.y
    u64* out;      // [P][L][N] coefficient-domain residues of the launch's plaintexts, indexed by blockIdx.y
    int L;
    int p_first;   // index (g*B + b) of the first plaintext of this launch
};

__device__ __forceinline__ double2 cmul_rn(double2 y, double2 w) {
    double p1 = __dmul_rn(y.x, w.x), p2 = __dmul_rn(y.y, w.y), p3 = __dmul_rn(y.x, w.y), p4 = __dmul_rn(y.y, w.x);
    return make_double2(__dsub_rn(p1, p2), __dadd_rn(p3, p4));
}

__global__ void __launch_bounds__(kThreads) k_fft_a(EncArgs A) {
    extern __shared__ double2 smc[];
    const int n = 1 << A.logn, S1 = 1 << A.b1, K1 = A.K1;
    const int P = blockIdx.y;
    const int g = (A.p_first + P) / A.B, b = (A.p_first + P) % A.B;
    const int pos0 = blockIdx.x * K1 * S1;
    for (int idx = threadIdx.x; idx < K1 * S1; idx += kThreads) {
        const int pos = pos0 + idx;
        const int j = A.jinv[pos];
        if (!HANN_CHECK_INDEX(j, n)) continue;
        double v;
        if (A.rows) {
            int row = j - g * A.B;
            if (row < 0) row += n;
            int col = (j + b) % A.R;
            v = (row < A.rows_in_block && col < A.dim) ? (double)A.rows[(long long)row * A.dim + col] : 0.0;
        } else {
            v = A.z[(long long)P * n + j];
        }
        smc[idx] = make_double2(v, 0.0);
    }
    __syncthreads();
    for (int s = 1; s <= A.b1; s++) {
        const int h = 1 << (s - 1);
        const int tstride = n >> s;  // n / (2h)
        for (int bf = threadIdx.x; bf < K1 * S1 / 2; bf += kThreads) {
            int ch = bf / (S1 / 2), lb = bf % (S1 / 2);
            int grp = lb / h, t = lb % h;
            int i0 = ch * S1 + grp * 2 * h + t, i1 = i0 + h;
            double2 x = smc[i0], y = smc[i1];
            double2 v = cmul_rn(y, A.T[t * tstride]);
            smc[i0] = make_double2(__dadd_rn(x.x, v.x), __dadd_rn(x.y, v.y));
            smc[i1] = make_double2(__dsub_rn(x.x, v.x), __dsub_rn(x.y, v.y));
        }
        __syncthreads();
    }
    double2* o = A.buf + (long long)P * n + pos0;
    for (int idx = threadIdx.x; idx < K1 * S1; idx += kThreads) o[idx] = smc[idx];
}

__global__ void __launch_bounds__(kThreads) k_fft_b(EncArgs A, LimbTable lt) {
    extern __shared__ double2 smc[];
    const int n = 1 << A.logn, N = 2 * n, S1 = 1 << A.b1, rows = n >> A.b1, C1 = A.C1;
    const int P = blockIdx.y;
    const int c0 = blockIdx.x * C1;
    const double2* in = A.buf + (long long)P * n + c0;
    for (int idx = threadIdx.x; idx < rows * C1; idx += kThreads) smc[idx] = in[(long long)(idx / C1) * S1 + (idx % C1)];
    __syncthreads();
    for (int s = A.b1 + 1; s <= A.logn; s++) {
        const int hr = 1 << (s - 1 - A.b1);  // half-size in rows
        const int tstride = n >> s;
        for (int bf = threadIdx.x; bf < (rows / 2) * C1; bf += kThreads) {
            int c = bf % C1, rb = bf / C1;
            int grp = rb / hr, tr = rb % hr;
            int r0 = grp * 2 * hr + tr, r1 = r0 + hr;
            int t = tr * S1 + c0 + c;
            double2 x = smc[r0 * C1 + c], y = smc[r1 * C1 + c];
            double2 v = cmul_rn(y, A.T[(long long)t * tstride]);
            smc[r0 * C1 + c] = make_double2(__dadd_rn(x.x, v.x), __dadd_rn(x.y, v.y));
            smc[r1 * C1 + c] = make_double2(__dsub_rn(x.x, v.x), __dsub_rn(x.y, v.y));
        }
        __syncthreads();
    }
    u64* out = A.out + (long long)P * A.L * N;
    for (int idx = threadIdx.x; idx < rows * C1; idx += kThreads) {
        const int k = (idx / C1) * S1 + c0 + (idx % C1);
        double2 cc = cmul_rn(smc[idx], A.U[k]);
        const i64 mre = __double2ll_rn(__dmul_rn(cc.x, A.scale));
        const i64 mim = __double2ll_rn(__dmul_rn(cc.y, A.scale));
        for (int l = 0; l < A.L; l++) {
            out[(long long)l * N + k] = reduce_signed(mre, lt.c[l]);
            out[(long long)l * N + k + n] = reduce_signed(mim, lt.c[l]);
        }
    }
}

int run_encode(hann_ctx* c, EncArgs& A, int P, int log_scale = -1) {
    const int n = c->n;
    A.T = c->fft_T;
    A.U = c->fft_U;
    A.jinv = c->jinv;
    A.logn = c->logN - 1;
    A.b1 = A.logn < 8 ? A.logn : 8;
    const int S1 = 1 << A.b1, chunks = n >> A.b1;
    A.K1 = chunks < 8 ? chunks : 8;
    A.C1 = S1 < 16 ? S1 : 16;
    A.scale = ldexp(1.0, (log_scale < 0 ? c->prm.log_scale : log_scale) - A.logn);
    A.L = c->L;
    A.R = c->R;
    A.B = c->B;
    {
        KProf kp(c, KC_FFT_A);
        k_fft_a<<<dim3(chunks / A.K1, P), kThreads, (size_t)A.K1 * S1 * sizeof(double2), c->stream>>>(A);
    }
    {
        KProf kp(c, KC_FFT_B);
        k_fft_b<<<dim3(S1 / A.C1, P), kThreads, (size_t)(n >> A.b1) * A.C1 * sizeof(double2), c->stream>>>(A, c->lt);
    }
    return check_launch(c, "encode");
}

}  // namespace

// FFT buffer of one launch group, then the staging area of encode_stage_group() full-size plaintexts (used when the
// half-size transform does not apply: small rings, moduli of 2^50 and more, buffers that are only 8-byte aligned)
int64_t encode_fft_bytes(const hann_ctx* c) {
    const int group = c->encode_group < c->R ? c->encode_group : c->R;
    return ((int64_t)group * c->n * (int64_t)sizeof(double2) + 255) / 256 * 256;
}
int encode_stage_group(const hann_ctx* c) {
    const int group = c->encode_group < c->R ? c->encode_group : c->R;
    return group < 8 ? group : 8;
}
int64_t encode_ws_bytes(const hann_ctx* c) { return encode_fft_bytes(c) + (int64_t)encode_stage_group(c) * c->L * c->N * 8; }

// plaintexts p_first .. p_first+count-1 of one block of candidate rows -> out[count][L][N], coefficient domain (the
// caller transforms them); ws holds count complex vectors of n points
int launch_encode_rows(hann_ctx* c, const float* rows, int64_t rows_in_block, int dim, int p_first, int count, u64* out,
                       void* ws) {
    EncArgs A = {};
    A.rows = rows;
    A.rows_in_block = rows_in_block;
    A.dim = dim;
    A.z = nullptr;
    A.buf = (double2*)ws;
    A.out = out;
    A.p_first = p_first;
    return run_encode(c, A, count);
}

// one slot vector z[n] (device) -> one polynomial [L][N], coefficient domain, at scale 2^log_scale (negative: the context's)
int launch_encode_slots(hann_ctx* c, const double* z_dev, u64* poly_out, void* ws, int log_scale) {
    EncArgs A = {};
    A.rows = nullptr;
    A.z = z_dev;
    A.buf = (double2*)ws;
    A.out = poly_out;
    return run_encode(c, A, 1, log_scale);
}

// =====================================================================================================================
// Fused path (rings with N >= 2^9 whose ciphertext primes are all below 2^50).
//
// Kernel W runs the FFT stages 1..8 (contiguous chunks of 256 points) in two register rounds of four stages; its
// twiddles T[t * n / 2^s] are the same 255 values for every chunk and plaintext and live in shared memory.
// Kernel X owns 16 adjacent columns of one plaintext: it finishes the FFT (the a-1 strided stages, a = logN - 8),
// twists, scales and rounds, and then -- because coefficient k and coefficient k + n are the real and imaginary part of
// the same FFT output -- already holds, per thread, exactly the words the first register round of the forward
// transform's pass A needs.  It runs pass A for every ciphertext prime from those registers and writes the pass-A
// output (binary64 residues) to the plaintext buffer; pass B is the stock kernel.  The integer coefficients never
// travel to HBM, and the operations and their order are those of the two-kernel path, so the results are bit-identical.
#include "nttcore.cuh"

namespace {

struct FusedArgs {
    const float* rows;
    long long rows_in_block;
    int dim, R, B, p_first;
    const double2* T;
    const double2* U;
    const int32_t* jinv;
    int logn, L;
    double scale;
    double2* buf;        // [count][n]
    u64* out;            // limb polynomial l of the launch's plaintext P starts at out + (P * L + l) * out_stride
    long long out_stride;
    const double2* tw;   // forward transform twiddles, binary64 format, [L+1][N]
    const LimbConst* lt;
};

__device__ __forceinline__ void dit(double2& x, double2& y, double2 w) {
    const double2 v = cmul_rn(y, w);
    y = make_double2(__dsub_rn(x.x, v.x), __dsub_rn(x.y, v.y));
    x = make_double2(__dadd_rn(x.x, v.x), __dadd_rn(x.y, v.y));
}

constexpr int kWChunks = 8;  // chunks of 256 points per CTA of kernel W (128 threads)

__global__ void __launch_bounds__(128) k_fft_w(FusedArgs A) {
    __shared__ double2 tc[256];                    // tc[h - 1 + t] = T[t * n / (2h)], h = 1, 2, .., 128
    __shared__ double2 sm[kWChunks * (256 + 16)];  // padded chunk: position pos lives at pos + pos/16
    const int n = 1 << A.logn;
    const int P = blockIdx.y;
    const int g = (A.p_first + P) / A.B, b = (A.p_first + P) % A.B;
    for (int i = threadIdx.x; i < 255; i += 128) {
        const int s = 32 - __clz(i + 1);  // stage 1..8: h = 2^(s-1), entries h-1 .. 2h-2
        const int h = 1 << (s - 1), t = i - (h - 1);
        tc[i] = A.T[(long long)t << (A.logn - s)];
    }
    __syncthreads();
    const int chunk0 = blockIdx.x * kWChunks;
    // round 1: stages 1..4 on 16 consecutive positions
    {
        const int ch = threadIdx.x >> 4, j = threadIdx.x & 15;
        const int pos0 = ((chunk0 + ch) << 8) + (j << 4);
        double2 x[16];
#pragma unroll
        for (int e = 0; e < 16; e++) {
            const int jj = A.jinv[pos0 + e];
            int row = jj - g * A.B;
            if (row < 0) row += n;
            const int col = (jj + b) % A.R;
            const double v = (row < A.rows_in_block && col < A.dim) ? (double)A.rows[(long long)row * A.dim + col] : 0.0;
            x[e] = make_double2(v, 0.0);
        }
#pragma unroll
        for (int s = 0; s < 4; s++) {
            const int span = 1 << s;
#pragma unroll
            for (int e = 0; e < 16; e++)
                if (!(e & span)) dit(x[e], x[e + span], tc[span - 1 + (e & (span - 1))]);
        }
        double2* d = sm + ch * 272 + 17 * j;
#pragma unroll
        for (int e = 0; e < 16; e++) d[e] = x[e];
    }
    __syncthreads();
    // round 2: stages 5..8 on positions j + 16 e
    {
        const int ch = threadIdx.x >> 4, j = threadIdx.x & 15;
        double2 x[16];
#pragma unroll
        for (int e = 0; e < 16; e++) x[e] = sm[ch * 272 + 17 * e + j];
#pragma unroll
        for (int s = 0; s < 4; s++) {
            const int span = 1 << s;  // in units of 16 positions
#pragma unroll
            for (int e = 0; e < 16; e++)
                if (!(e & span)) dit(x[e], x[e + span], tc[16 * span - 1 + j + 16 * (e & (span - 1))]);
        }
        double2* o = A.buf + (long long)P * n + ((long long)(chunk0 + ch) << 8) + j;
#pragma unroll
        for (int e = 0; e < 16; e++) o[16 * e] = x[e];
    }
}

// Kernel W for B >= 8: a CTA takes ONE chunk of 256 FFT positions for EIGHT plaintexts (g, b0 .. b0+7).  For a given
// position the eight plaintexts read eight consecutive columns of the same candidate row, so the gather moves whole
// 32-byte sectors instead of one float per sector, and all of a thread's 16 loads are independent.
__global__ void __launch_bounds__(128, 5) k_fft_w8(FusedArgs A) {
    __shared__ double2 tc[256];
    __shared__ double2 sm[8 * 272];
    // gathered inputs [plaintext][position + position/16]: they live in the tail of the exchange tile until round 1 has
    // read them (38 KiB per CTA: five CTAs per SM)
    float* sin_ = (float*)(sm + 8 * 272) - 8 * 272;
    const int n = 1 << A.logn;
    const int P0 = blockIdx.y * 8;
    const int g = (A.p_first + P0) / A.B, b0 = (A.p_first + P0) % A.B;
    const int chunk = blockIdx.x;
    for (int i = threadIdx.x; i < 255; i += 128) {
        const int s = 32 - __clz(i + 1);
        const int h = 1 << (s - 1), t = i - (h - 1);
        tc[i] = A.T[(long long)t << (A.logn - s)];
    }
#pragma unroll
    for (int i = 0; i < 16; i++) {
        const int idx = threadIdx.x + 128 * i, p = idx >> 3, pl = idx & 7;
        const int jj = A.jinv[(chunk << 8) + p];
        int row = jj - g * A.B;
        if (row < 0) row += n;
        const int col = (jj + b0 + pl) % A.R;
        sin_[pl * 272 + p + (p >> 4)] = (row < A.rows_in_block && col < A.dim) ? A.rows[(long long)row * A.dim + col] : 0.0f;
    }
    __syncthreads();
    const int pl = threadIdx.x >> 4, j = threadIdx.x & 15;
    {
        double2 x[16];
#pragma unroll
        for (int e = 0; e < 16; e++) x[e] = make_double2((double)sin_[pl * 272 + 17 * j + e], 0.0);
#pragma unroll
        for (int s = 0; s < 4; s++) {
            const int span = 1 << s;
#pragma unroll
            for (int e = 0; e < 16; e++)
                if (!(e & span)) dit(x[e], x[e + span], tc[span - 1 + (e & (span - 1))]);
        }
        double2* d = sm + pl * 272 + 17 * j;
        __syncthreads();  // every thread has read its gathered inputs: the tile may be overwritten
#pragma unroll
        for (int e = 0; e < 16; e++) d[e] = x[e];
    }
    __syncthreads();
    {
        double2 x[16];
#pragma unroll
        for (int e = 0; e < 16; e++) x[e] = sm[pl * 272 + 17 * e + j];
#pragma unroll
        for (int s = 0; s < 4; s++) {
            const int span = 1 << s;
#pragma unroll
            for (int e = 0; e < 16; e++)
                if (!(e & span)) dit(x[e], x[e + span], tc[16 * span - 1 + j + 16 * (e & (span - 1))]);
        }
        double2* o = A.buf + (long long)(P0 + pl) * n + ((long long)chunk << 8) + j;
#pragma unroll
        for (int e = 0; e < 16; e++) o[16 * e] = x[e];
    }
}

// R1 + R2 = a = logN - 8 are the register rounds of the transform's pass A (R1 = min(a, 4)); the FFT's a - 1 strided
// stages run as a first round of R2 stages and a last round of R1 - 1 stages
#ifndef HANN_X_MINBLOCKS
#define HANN_X_MINBLOCKS 3
#endif
// SYM: the encoding of a real slot vector is fixed by X -> 1/X, so its transform takes the same value at psi^(2t+1) and
// at the inverse of that root.  After the first stage (which splits modulo X^n - i and X^n + i) only the first half
// carries on; rows 2^(a-1) .. 2^a - 1 of the pass-A output are not produced (out_stride may then be N/2), and pass B
// transforms the first half of the chunks only.
template <int R1, int R2, bool SYM>
__global__ void __launch_bounds__(256, HANN_X_MINBLOCKS) k_encode_x(FusedArgs A) {
    extern __shared__ u64 smx[];
    constexpr int a = R1 + R2;
    constexpr int G1 = 1 << R2;        // row groups of transform round 1 = threads per column
    constexpr int HF = 1 << (R1 - 1);  // complex words a thread holds after the FFT's last round
    constexpr int rows_fft = 1 << (a - 1);
    const int n = 1 << A.logn;
    const int P = blockIdx.y;
    const int c0 = blockIdx.x << 4;
    const double2* in = A.buf + (long long)P * n + c0;
    double2* smc = (double2*)smx;  // [rows_fft][16]
    if (R2 > 0) {
        // FFT round of R2 stages: rows gg*2^R2 + e, spans 1 .. 2^(R2-1) rows
        constexpr int E = 1 << (R2 == 0 ? 1 : R2);
        for (int w = threadIdx.x; w < (rows_fft >> R2) * 16; w += blockDim.x) {
            const int c = w & 15, gg = w >> 4;
            double2 x[E];
#pragma unroll
            for (int e = 0; e < E; e++) x[e] = in[(long long)((gg << R2) + e) * 256 + c];
#pragma unroll
            for (int t = 0; t < R2; t++) {
                const int span = 1 << t;
#pragma unroll
                for (int e = 0; e < E; e++)
                    if (!(e & span)) {
                        const int tr = e & (span - 1);
                        dit(x[e], x[e + span], A.T[(long long)(tr * 256 + c0 + c) << (a - 2 - t)]);
                    }
            }
#pragma unroll
            for (int e = 0; e < E; e++) smc[(((gg << R2) + e) << 4) + c] = x[e];
        }
        __syncthreads();
    }
    // FFT last round (R1 - 1 stages) on rows g + G1*e, then twist, scale, round: one thread per (column, g)
    double m[1 << R1];  // rounded coefficients: rows g + G1*e, e < 2^R1 (second half = imaginary parts)
    const int c = threadIdx.x & 15, g = threadIdx.x >> 4;
    const bool active = g < G1;
    if (active) {
        double2 x[HF];
#pragma unroll
        for (int e = 0; e < HF; e++) x[e] = R2 > 0 ? smc[((g + G1 * e) << 4) + c] : in[(long long)(g + G1 * e) * 256 + c];
#pragma unroll
        for (int u = 0; u < R1 - 1; u++) {
            const int span = 1 << u, t = R2 + u;
#pragma unroll
            for (int e = 0; e < HF; e++)
                if (!(e & span)) {
                    const int tr = g + G1 * (e & (span - 1));
                    dit(x[e], x[e + span], A.T[(long long)(tr * 256 + c0 + c) << (a - 2 - t)]);
                }
        }
#pragma unroll
        for (int e = 0; e < HF; e++) {
            const int k = (g + G1 * e) * 256 + c0 + c;
            const double2 cc = cmul_rn(x[e], A.U[k]);
            m[e] = rint(__dmul_rn(cc.x, A.scale));
            m[e + HF] = rint(__dmul_rn(cc.y, A.scale));
        }
    }
    // pass A of the forward transform for every ciphertext prime, from the registers.  Pass A uses table entries
    // 1 .. 2^a - 1 of a limb, the same for every column: they are staged in shared memory behind the exchange tile.
    constexpr int RR2 = R2 == 0 ? 1 : R2;
    constexpr int G2 = 1 << R1;
    constexpr int NT = 1 << a;  // cached twiddle pairs per limb (entry 0 unused)
    double2* twc = (double2*)(smx + (R2 > 0 ? (size_t)NT * 16 : 0));
    for (int i = threadIdx.x; i < A.L * NT; i += blockDim.x) {
        const int l = i / NT, e = i % NT;
        if (e) twc[i] = A.tw[((size_t)l << (A.logn + 1)) + e];
    }
    if constexpr (SYM && R1 == 4 && R2 == 4) {
        // The half-size second round has work for 128 threads only: two limbs at a time, the first rounds of both by
        // all threads into the two halves of the exchange tile, then threads 0..127 finish one limb and threads
        // 128..255 the other.
        constexpr int HT = (NT / 2) * 16;  // words of a half-size tile
        for (int l = 0; l < A.L; l += 2) {
            __syncthreads();  // the twiddle cache is filled (first pair) / the exchange tile is free again
            for (int h = 0; h < 2 && l + h < A.L; h++) {
                const ArithF64 ar(A.lt + l + h);
                const double2* tw = twc + (l + h) * NT;
                double x[HF];
                const double2 w1 = tw[1];
#pragma unroll
                for (int e = 0; e < HF; e++) x[e] = __dadd_rn(ar.reduce(m[e]), ar.mulmod_small(ar.reduce(m[e + HF]), w1));
                fwd_round<R1 - 1, ArithF64, R1 - 1>(ar, x, tw, 2u);
#pragma unroll
                for (int e = 0; e < HF; e++) smx[h * HT + ((g + G1 * e) << 4) + c] = ar.to_exch(x[e]);
            }
            __syncthreads();
            const int h = threadIdx.x >> 7, ll = l + h;
            if (ll < A.L) {
                const ArithF64 ar(A.lt + ll);
                const double2* tw = twc + ll * NT;
                u64* base = A.out + ((long long)P * A.L + ll) * A.out_stride + c0;
                const int cc = threadIdx.x & 15, gg = (threadIdx.x & 127) >> 4;
                double x[1 << R2];
#pragma unroll
                for (int e = 0; e < (1 << R2); e++) x[e] = ar.from_mid(smx[h * HT + (((gg << R2) + e) << 4) + cc]);
                fwd_round<R2, ArithF64, 5 - R1>(ar, x, tw, (unsigned)(G2 + gg));
#pragma unroll
                for (int e = 0; e < (1 << R2); e++) base[(size_t)((gg << R2) + e) * 256 + cc] = ar.to_mid(x[e]);
            }
        }
    } else
    for (int l = 0; l < A.L; l++) {
        const ArithF64 ar(A.lt + l);
        const double2* tw = twc + l * NT;
        u64* base = A.out + ((long long)P * A.L + l) * A.out_stride + c0;
        __syncthreads();  // the twiddle cache is filled (first limb) / the exchange tile is free again
        if (active && SYM) {
            constexpr int RS = R1 > 1 ? R1 - 1 : 1;
            double x[1 << RS];
            const double2 w1 = tw[1];
#pragma unroll
            for (int e = 0; e < HF; e++) x[e] = __dadd_rn(ar.reduce(m[e]), ar.mulmod_small(ar.reduce(m[e + HF]), w1));
            fwd_round<RS, ArithF64, RS>(ar, x, tw, 2u);
#pragma unroll
            for (int e = 0; e < HF; e++) {
                if (R2 == 0) base[(size_t)(g + G1 * e) * 256 + c] = ar.to_mid(x[e]);
                else smx[((g + G1 * e) << 4) + c] = ar.to_exch(x[e]);
            }
        } else if (active) {
            double x[1 << R1];
#pragma unroll
            for (int e = 0; e < (1 << R1); e++) x[e] = ar.reduce(m[e]);
            fwd_round<R1, ArithF64, R1>(ar, x, tw, 1u);
#pragma unroll
            for (int e = 0; e < (1 << R1); e++) {
                if (R2 == 0) base[(size_t)(g + G1 * e) * 256 + c] = ar.to_mid(x[e]);
                else smx[((g + G1 * e) << 4) + c] = ar.to_exch(x[e]);
            }
        }
        if (R2 > 0) {
            __syncthreads();
            for (int w = threadIdx.x; w < ((SYM ? G2 / 2 : G2) << 4); w += blockDim.x) {
                const int cc = w & 15, gg = w >> 4;
                double x[1 << RR2];
#pragma unroll
                for (int e = 0; e < (1 << RR2); e++) x[e] = ar.from_mid(smx[(((gg << RR2) + e) << 4) + cc]);
                fwd_round<RR2, ArithF64, 5 - R1>(ar, x, tw, (unsigned)(G2 + gg));
#pragma unroll
                for (int e = 0; e < (1 << RR2); e++) base[(size_t)((gg << RR2) + e) * 256 + cc] = ar.to_mid(x[e]);
            }
        }
    }
}

typedef void (*KernX)(FusedArgs);
template <bool SYM>
KernX pick_x_t(int a) {
    switch (a) {
        case 1: return k_encode_x<1, 0, false>;
        case 2: return k_encode_x<2, 0, SYM>;
        case 3: return k_encode_x<3, 0, SYM>;
        case 4: return k_encode_x<4, 0, SYM>;
        case 5: return k_encode_x<4, 1, SYM>;
        case 6: return k_encode_x<4, 2, SYM>;
        case 7: return k_encode_x<4, 3, SYM>;
        default: return k_encode_x<4, 4, SYM>;
    }
}
KernX pick_x(int a, bool sym) { return sym && a >= 2 ? pick_x_t<true>(a) : pick_x_t<false>(a); }

}  // namespace

bool encode_fused_available(const hann_ctx* c) {
    if (c->logN < 9) return false;
    for (int l = 0; l < c->L; l++)
        if (c->mod[l] >= (1ULL << 50)) return false;
    return true;
}

// plaintexts p_first .. p_first+count-1 of one block: encode and run pass A of their forward transforms into
// out[count][L][out_stride]; the caller finishes with launch_ntt_fwd_pass_b over the same polynomials.
// sym: leave the second half of the pass-A rows out (out_stride >= N/2); the caller finishes with launch_ntt_fwd_pass_b_half.
int launch_encode_rows_fused(hann_ctx* c, const float* rows, int64_t rows_in_block, int dim, int p_first, int count, u64* out,
                             int64_t out_stride, void* ws, bool sym) {
    FusedArgs A;
    A.rows = rows;
    A.rows_in_block = rows_in_block;
    A.dim = dim;
    A.R = c->R;
    A.B = c->B;
    A.p_first = p_first;
    A.T = c->fft_T;
    A.U = c->fft_U;
    A.jinv = c->jinv;
    A.logn = c->logN - 1;
    A.L = c->L;
    A.scale = ldexp(1.0, c->prm.log_scale - A.logn);
    A.buf = (double2*)ws;
    A.out = out;
    A.out_stride = out_stride;
    A.tw = (const double2*)c->tw_fwd_f64;
    A.lt = c->lt_dev;
    const int n = c->n, a = c->logN - 8;
    const int chunks = n >> 8;  // >= 1 because logN >= 9
    if (c->B % 8 == 0 && count % 8 == 0 && p_first % 8 == 0) {
        KProf kp(c, KC_FFT_A);
        k_fft_w8<<<dim3(chunks, count / 8), 128, 0, c->stream>>>(A);
    } else if (chunks % kWChunks == 0) {
        KProf kp(c, KC_FFT_A);
        k_fft_w<<<dim3(chunks / kWChunks, count), 128, 0, c->stream>>>(A);
    } else {
        // small rings: the stock first-pass kernel produces the same buffer
        EncArgs E = {};
        E.rows = rows;
        E.rows_in_block = rows_in_block;
        E.dim = dim;
        E.buf = (double2*)ws;
        E.p_first = p_first;
        E.T = c->fft_T;
        E.U = c->fft_U;
        E.jinv = c->jinv;
        E.logn = A.logn;
        E.b1 = 8;
        E.K1 = chunks < 8 ? chunks : 8;
        E.R = c->R;
        E.B = c->B;
        KProf kp(c, KC_FFT_A);
        k_fft_a<<<dim3(chunks / E.K1, count), kThreads, (size_t)E.K1 * 256 * sizeof(double2), c->stream>>>(E);
    }
    {
        // exchange tile (FFT: 2^(a-1) x 16 complex = transform: 2^a x 16 words) when a > 4, then L x 2^a twiddle pairs
        const size_t smem = (a > 4 ? (size_t)(1 << a) * 16 * 8 : 0) + (size_t)c->L * (1 << a) * 16;
        KProf kp(c, KC_FFT_B);
        const int threads = a >= 8 ? 256 : (a == 7 ? 128 : 64);  // 16 columns x 2^R2 row groups, at least two warps
        if (smem > 48 * 1024) cudaFuncSetAttribute(pick_x(a, sym), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        pick_x(a, sym)<<<dim3(16, count), threads, smem, c->stream>>>(A);
    }
    return check_launch(c, "encode_fused");
}

HANN_DEBUG_DEFINE_BIND(debug_bind_encode)
