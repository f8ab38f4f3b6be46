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
    u64* out;      // [..][L][N] coefficient-domain residues, indexed by p_first + blockIdx.y
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
        const int u = (int)(__brev((unsigned)pos) >> (32 - A.logn));
        const int j = A.jinv[u];
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
    u64* out = A.out + (long long)(A.p_first + P) * A.L * N;
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

int run_encode(hann_ctx* c, EncArgs& A, int P) {
    const int n = c->n;
    A.T = c->fft_T;
    A.U = c->fft_U;
    A.jinv = c->jinv;
    A.logn = c->logN - 1;
    A.b1 = A.logn < 8 ? A.logn : 8;
    const int S1 = 1 << A.b1, chunks = n >> A.b1;
    A.K1 = chunks < 8 ? chunks : 8;
    A.C1 = S1 < 16 ? S1 : 16;
    A.scale = ldexp(1.0, c->prm.log_scale - A.logn);
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

int64_t encode_ws_bytes(const hann_ctx* c) {
    const int group = c->encode_group < c->R ? c->encode_group : c->R;
    return (int64_t)group * c->n * (int64_t)sizeof(double2);
}

// plaintexts p_first .. p_first+count-1 of one block of candidate rows -> pt_block[p][L][N], coefficient domain (the
// caller transforms them); ws holds count complex vectors of n points
int launch_encode_rows(hann_ctx* c, const float* rows, int64_t rows_in_block, int dim, int p_first, int count, u64* pt_block,
                       void* ws) {
    EncArgs A = {};
    A.rows = rows;
    A.rows_in_block = rows_in_block;
    A.dim = dim;
    A.z = nullptr;
    A.buf = (double2*)ws;
    A.out = pt_block;
    A.p_first = p_first;
    return run_encode(c, A, count);
}

// one slot vector z[n] (device) -> one polynomial [L][N], coefficient domain
int launch_encode_slots(hann_ctx* c, const double* z_dev, u64* poly_out, void* ws) {
    EncArgs A = {};
    A.rows = nullptr;
    A.z = z_dev;
    A.buf = (double2*)ws;
    A.out = poly_out;
    return run_encode(c, A, 1);
}
