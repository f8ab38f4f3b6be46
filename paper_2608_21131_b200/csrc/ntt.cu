// Negacyclic number-theoretic transforms over 64-bit RNS limbs.
//
// Forward: Cooley-Tukey butterflies with merged powers of psi, natural order in, bit-reversed order out
// (position k holds the value at psi^(2*brev(k)+1)); inverse: Gentleman-Sande, bit-reversed in, natural out,
// scaled by N^{-1}.  Butterflies are lazy (Harvey): forward values stay in [0, 4q), inverse in [0, 2q), one
// correction at the end.  Twiddles are multiplied with Shoup's precomputed quotients.
//
// A transform of N = 2^logN points is split into two passes so that every pass works out of shared memory:
//   pass A covers the a = logN - b stages whose butterfly span is >= S = 2^b words (a CTA owns C adjacent
//          columns of the 2^a x S matrix view, 8*C contiguous bytes per row);
//   pass B covers the b stages inside contiguous chunks of S words (a CTA owns K chunks).
// With b = min(logN, 8) a ring of 2^16 is a 256 x 256 matrix.  The inverse runs B' then A'.
#include "internal.h"

namespace {

constexpr int kThreads = 256;

struct NttArgs {
    u64* data;
    long long stride;  // words between consecutive polynomials
    int logN, a, b;    // a + b = logN
    int C, K;          // columns per CTA in pass A, chunks per CTA in pass B
    const u64* tw;     // [L+1][N]
    const u64* tws;
    LimbMap lm;
};

__global__ void __launch_bounds__(kThreads) k_ntt_fwd_a(NttArgs A, LimbTable lt) {
    extern __shared__ u64 sm[];
    const int N = 1 << A.logN, S = 1 << A.b, rows = 1 << A.a, C = A.C;
    const long long poly = blockIdx.y;
    const int limb = A.lm.limb[poly % A.lm.period];
    const u64 q = lt.c[limb].q, q2 = 2 * q;
    u64* base = A.data + poly * A.stride + (long long)blockIdx.x * C;
    const u64* tw = A.tw + (size_t)limb * N;
    const u64* tws = A.tws + (size_t)limb * N;
    for (int idx = threadIdx.x; idx < rows * C; idx += kThreads) sm[idx] = base[(size_t)(idx / C) * S + (idx % C)];
    __syncthreads();
    for (int s = 0; s < A.a; s++) {
        const int m = 1 << s, tr = rows >> (s + 1);
        for (int bf = threadIdx.x; bf < (rows / 2) * C; bf += kThreads) {
            int c = bf % C, rb = bf / C;
            int i = rb / tr, jr = rb % tr;
            int r0 = i * 2 * tr + jr, r1 = r0 + tr;
            u64 w = tw[m + i], ws = tws[m + i];
            u64 X = sm[r0 * C + c], Y = sm[r1 * C + c];
            X = csub(X, q2);
            u64 T = shoup_mul(Y, w, ws, q);
            sm[r0 * C + c] = X + T;
            sm[r1 * C + c] = X - T + q2;
        }
        __syncthreads();
    }
    for (int idx = threadIdx.x; idx < rows * C; idx += kThreads) base[(size_t)(idx / C) * S + (idx % C)] = sm[idx];
}

__global__ void __launch_bounds__(kThreads) k_ntt_fwd_b(NttArgs A, LimbTable lt) {
    extern __shared__ u64 sm[];
    const int N = 1 << A.logN, S = 1 << A.b, K = A.K;
    const long long poly = blockIdx.y;
    const int limb = A.lm.limb[poly % A.lm.period];
    const u64 q = lt.c[limb].q, q2 = 2 * q;
    const int chunk0 = blockIdx.x * K;
    u64* base = A.data + poly * A.stride + (size_t)chunk0 * S;
    const u64* tw = A.tw + (size_t)limb * N;
    const u64* tws = A.tws + (size_t)limb * N;
    for (int idx = threadIdx.x; idx < K * S; idx += kThreads) sm[idx] = base[idx];
    __syncthreads();
    for (int s = 0; s < A.b; s++) {
        const int m = (N >> A.b) << s, t = S >> (s + 1);
        for (int bf = threadIdx.x; bf < K * S / 2; bf += kThreads) {
            int ch = bf / (S / 2), lb = bf % (S / 2);
            int il = lb / t, jl = lb % t;
            int j0 = ch * S + il * 2 * t + jl, j1 = j0 + t;
            int i = ((chunk0 + ch) << s) + il;
            u64 w = tw[m + i], ws = tws[m + i];
            u64 X = sm[j0], Y = sm[j1];
            X = csub(X, q2);
            u64 T = shoup_mul(Y, w, ws, q);
            sm[j0] = X + T;
            sm[j1] = X - T + q2;
        }
        __syncthreads();
    }
    for (int idx = threadIdx.x; idx < K * S; idx += kThreads) base[idx] = csub(csub(sm[idx], q2), q);
}

// inverse pass B': stages with span 1 .. S/2 inside contiguous chunks
__global__ void __launch_bounds__(kThreads) k_ntt_inv_b(NttArgs A, LimbTable lt, int final_scale) {
    extern __shared__ u64 sm[];
    const int N = 1 << A.logN, S = 1 << A.b, K = A.K;
    const long long poly = blockIdx.y;
    const int limb = A.lm.limb[poly % A.lm.period];
    const u64 q = lt.c[limb].q, q2 = 2 * q;
    const int chunk0 = blockIdx.x * K;
    u64* base = A.data + poly * A.stride + (size_t)chunk0 * S;
    const u64* tw = A.tw + (size_t)limb * N;
    const u64* tws = A.tws + (size_t)limb * N;
    for (int idx = threadIdx.x; idx < K * S; idx += kThreads) sm[idx] = base[idx];
    __syncthreads();
    for (int s = 0; s < A.b; s++) {
        const int t = 1 << s, h = N >> (s + 1);  // h groups of span 2t over the whole polynomial
        for (int bf = threadIdx.x; bf < K * S / 2; bf += kThreads) {
            int ch = bf / (S / 2), lb = bf % (S / 2);
            int il = lb / t, jl = lb % t;
            int j0 = ch * S + il * 2 * t + jl, j1 = j0 + t;
            int i = (chunk0 + ch) * (S / (2 * t)) + il;
            u64 w = tw[h + i], ws = tws[h + i];
            u64 X = sm[j0], Y = sm[j1];
            sm[j0] = csub(X + Y, q2);
            sm[j1] = shoup_mul(X - Y + q2, w, ws, q);
        }
        __syncthreads();
    }
    if (final_scale) {
        const u64 ni = lt.c[limb].ninv, nis = lt.c[limb].ninv_s;
        for (int idx = threadIdx.x; idx < K * S; idx += kThreads) base[idx] = csub(shoup_mul(sm[idx], ni, nis, q), q);
    } else {
        for (int idx = threadIdx.x; idx < K * S; idx += kThreads) base[idx] = sm[idx];
    }
}

// inverse pass A': stages with span S .. N/2, then the N^{-1} scaling
__global__ void __launch_bounds__(kThreads) k_ntt_inv_a(NttArgs A, LimbTable lt) {
    extern __shared__ u64 sm[];
    const int N = 1 << A.logN, S = 1 << A.b, rows = 1 << A.a, C = A.C;
    const long long poly = blockIdx.y;
    const int limb = A.lm.limb[poly % A.lm.period];
    const u64 q = lt.c[limb].q, q2 = 2 * q;
    u64* base = A.data + poly * A.stride + (long long)blockIdx.x * C;
    const u64* tw = A.tw + (size_t)limb * N;
    const u64* tws = A.tws + (size_t)limb * N;
    for (int idx = threadIdx.x; idx < rows * C; idx += kThreads) sm[idx] = base[(size_t)(idx / C) * S + (idx % C)];
    __syncthreads();
    for (int s = 0; s < A.a; s++) {
        const int tr = 1 << s, h = rows >> (s + 1);  // h groups of 2*tr rows
        for (int bf = threadIdx.x; bf < (rows / 2) * C; bf += kThreads) {
            int c = bf % C, rb = bf / C;
            int i = rb / tr, jr = rb % tr;
            int r0 = i * 2 * tr + jr, r1 = r0 + tr;
            u64 w = tw[h + i], ws = tws[h + i];
            u64 X = sm[r0 * C + c], Y = sm[r1 * C + c];
            sm[r0 * C + c] = csub(X + Y, q2);
            sm[r1 * C + c] = shoup_mul(X - Y + q2, w, ws, q);
        }
        __syncthreads();
    }
    const u64 ni = lt.c[limb].ninv, nis = lt.c[limb].ninv_s;
    for (int idx = threadIdx.x; idx < rows * C; idx += kThreads)
        base[(size_t)(idx / C) * S + (idx % C)] = csub(shoup_mul(sm[idx], ni, nis, q), q);
}

NttArgs make_args(const hann_ctx* c, u64* data, long long stride, const LimbMap& lm, bool inverse) {
    NttArgs A;
    A.data = data;
    A.stride = stride;
    A.logN = c->logN;
    A.b = c->logN < 8 ? c->logN : 8;
    A.a = c->logN - A.b;
    int S = 1 << A.b;
    A.C = S < 32 ? S : 32;
    int chunks = c->N >> A.b;
    A.K = chunks < 16 ? chunks : 16;
    A.tw = inverse ? c->tw_inv : c->tw_fwd;
    A.tws = inverse ? c->tw_inv_s : c->tw_fwd_s;
    A.lm = lm;
    return A;
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
LimbMap limbmap_single(int limb) {
    LimbMap m;
    m.period = 1;
    m.limb[0] = (signed char)limb;
    return m;
}

int launch_ntt_fwd(hann_ctx* c, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm) {
    if (npoly <= 0) return HANN_OK;
    NttArgs A = make_args(c, data, stride, lm, false);
    const int S = 1 << A.b;
    for (int64_t p0 = 0; p0 < npoly; p0 += 65535) {
        int np = (int)((npoly - p0) < 65535 ? (npoly - p0) : 65535);
        NttArgs Ap = A;
        Ap.data = data + p0 * stride;
        // the limb of polynomial p0 + y must stay lm.limb[(p0 + y) % period]: rotate the map
        for (int i = 0; i < lm.period; i++) Ap.lm.limb[i] = lm.limb[(p0 + i) % lm.period];
        if (A.a > 0) {
            dim3 grid(S / A.C, np);
            size_t smem = (size_t)(1 << A.a) * A.C * sizeof(u64);
            KProf kp(c, KC_NTT_FWD_A);
            k_ntt_fwd_a<<<grid, kThreads, smem, c->stream>>>(Ap, c->lt);
        }
        dim3 grid((c->N >> A.b) / A.K, np);
        size_t smem = (size_t)A.K * S * sizeof(u64);
        KProf kp(c, KC_NTT_FWD_B);
        k_ntt_fwd_b<<<grid, kThreads, smem, c->stream>>>(Ap, c->lt);
    }
    return check_launch(c, "ntt_fwd");
}

int launch_ntt_inv(hann_ctx* c, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm) {
    if (npoly <= 0) return HANN_OK;
    NttArgs A = make_args(c, data, stride, lm, true);
    const int S = 1 << A.b;
    for (int64_t p0 = 0; p0 < npoly; p0 += 65535) {
        int np = (int)((npoly - p0) < 65535 ? (npoly - p0) : 65535);
        NttArgs Ap = A;
        Ap.data = data + p0 * stride;
        for (int i = 0; i < lm.period; i++) Ap.lm.limb[i] = lm.limb[(p0 + i) % lm.period];
        dim3 grid((c->N >> A.b) / A.K, np);
        size_t smem = (size_t)A.K * S * sizeof(u64);
        {
            KProf kp(c, KC_NTT_INV_B);
            k_ntt_inv_b<<<grid, kThreads, smem, c->stream>>>(Ap, c->lt, A.a == 0 ? 1 : 0);
        }
        if (A.a > 0) {
            dim3 grid2(S / A.C, np);
            size_t smem2 = (size_t)(1 << A.a) * A.C * sizeof(u64);
            KProf kp(c, KC_NTT_INV_A);
            k_ntt_inv_a<<<grid2, kThreads, smem2, c->stream>>>(Ap, c->lt);
        }
    }
    return check_launch(c, "ntt_inv");
}

int ntt_configure(hann_ctx* c) {
    // pass A tiles use up to 2^8 * 32 * 8 = 64 KiB of shared memory: opt in above the 48 KiB default
    cudaError_t e = cudaFuncSetAttribute(k_ntt_fwd_a, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_ntt_inv_a, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
    if (e != cudaSuccess) {
        c->err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e);
        return HANN_ECUDA;
    }
    return HANN_OK;
}
