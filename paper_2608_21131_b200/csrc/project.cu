// Rank reduction under encryption with the projection matrix packed by windows (Sec. 3.1 "How" and Detail): the
// kernels that build the packed diagonals and the 0/1 window masks as slot vectors, and the mask combine that turns two
// slot rotations of the query into one rotation inside every window.  Everything else of the projection (hoisted
// rotations, multiply-accumulate, giant steps, fold, rescale) is the scoring path's own machinery (api.cu).
//
// Layout conventions (n slots viewed with period D = c R; window k of a period = positions k R .. k R + R - 1):
//   query      slot i holds q[i mod D];
//   matrix     W [D][R] row-major; chunk k is the R x R matrix W_k^T[r][col] = W[k R + col][r];
//   packed     plaintext (g, b), slot i with i mod D = k R + j:  W[k R + (j + b) mod R][(j - g B) mod R]  -- diagonal
//              g B + b of every chunk in its own window, shifted inside the window by the giant-step amount;
//   masks      lo_b[i] = 1 if (i mod R) + b < R else 0, hi_b = 1 - lo_b.
#include "internal.h"
#include "debugcheck.cuh"

namespace {

constexpr int kThreads = 256;

inline int grid_for(int64_t work, int cap = 148 * 16) {
    int64_t g = (work + kThreads - 1) / kThreads;
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    return (int)g;
}

// z[i] = W[k R + (j + b) mod R][(j - g B) mod R], i mod D = k R + j        (one packed diagonal as a slot vector)
__global__ void __launch_bounds__(kThreads) k_packed_diagonal(const float* __restrict__ W, int D, int R, int B, int g, int b, int n,
                                                              double* __restrict__ z) {
    for (int i = blockIdx.x * kThreads + threadIdx.x; i < n; i += gridDim.x * kThreads) {
        const int w = i % D, k = w / R, j = w % R;
        int col = (j - g * B) % R;
        if (col < 0) col += R;
        const long long widx = (long long)(k * R + (j + b) % R) * R + col;
        if (!HANN_CHECK_INDEX(widx, (long long)D * R)) continue;
        z[i] = (double)W[widx];
    }
}

// lo[i] = [(i mod R) + b < R], hi = 1 - lo
__global__ void __launch_bounds__(kThreads) k_window_masks(int R, int b, int n, double* __restrict__ lo, double* __restrict__ hi) {
    for (int i = blockIdx.x * kThreads + threadIdx.x; i < n; i += gridDim.x * kThreads) {
        const double v = (i % R) + b < R ? 1.0 : 0.0;
        lo[i] = v;
        hi[i] = 1.0 - v;
    }
}

// cyc[b][comp][l][t] = lo[b][l][t'] * A_b[comp][l][t] + hi[b][l][t'] * H_b[comp][l][t]   (transform domain, elementwise)
// A_0 = ct and no H_0 (hi_0 = 0); A_b = rot_a[b-1], H_b = rot_h[b-1] for b >= 1.  The masks are stored as the first N/2
// transform values of a real slot vector's encoding: position t >= N/2 mirrors position N - 1 - t.
__global__ void __launch_bounds__(kThreads) k_mask_combine(const u64* __restrict__ ct, const u64* __restrict__ rot_a,
                                                           const u64* __restrict__ rot_h, const u64* __restrict__ lo,
                                                           const u64* __restrict__ hi, u64* __restrict__ cyc, int Bn, int N, int L,
                                                           LimbTable lt) {
    const long long LN = (long long)L * N, ctw = 2 * LN, total = (long long)Bn * ctw;
    const int n = N >> 1;
    for (long long idx = (long long)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (long long)gridDim.x * kThreads) {
        const int t = (int)(idx % N);
        const int l = (int)((idx / N) % L);
        const long long b = idx / ctw, rem = idx % ctw;
        const LimbConst& lc = lt.c[l];
        const long long m = (b * L + l) * n + (t < n ? t : N - 1 - t);
        if (!HANN_CHECK_INDEX(m, (long long)Bn * L * n)) continue;
        const u64 a = b == 0 ? ct[rem] : rot_a[(b - 1) * ctw + rem];
        u64 v = mulmod(a, lo[m], lc);
        if (b > 0) v = addmod(v, mulmod(rot_h[(b - 1) * ctw + rem], hi[m], lc), lc.q);
        cyc[idx] = v;
    }
}

}  // namespace

int launch_packed_diagonal(hann_ctx* c, const float* W, int D, int g, int b, double* z) {
    {
        KProf kp(c, KC_OTHER);
        k_packed_diagonal<<<grid_for(c->n), kThreads, 0, c->stream>>>(W, D, c->R, c->B, g, b, c->n, z);
    }
    return check_launch(c, "packed_diagonal");
}

int launch_window_masks(hann_ctx* c, int b, double* lo, double* hi) {
    {
        KProf kp(c, KC_OTHER);
        k_window_masks<<<grid_for(c->n), kThreads, 0, c->stream>>>(c->R, b, c->n, lo, hi);
    }
    return check_launch(c, "window_masks");
}

int launch_mask_combine(hann_ctx* c, const u64* ct, const u64* rot_a, const u64* rot_h, const u64* lo, const u64* hi, u64* cyc) {
    {
        KProf kp(c, KC_OTHER);
        k_mask_combine<<<grid_for((int64_t)c->B * 2 * c->L * c->N, 148 * 32), kThreads, 0, c->stream>>>(ct, rot_a, rot_h, lo, hi, cyc,
                                                                                                      c->B, c->N, c->L, c->lt);
    }
    return check_launch(c, "mask_combine");
}

HANN_DEBUG_DEFINE_BIND(debug_bind_project)
