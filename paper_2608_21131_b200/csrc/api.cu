// C-ABI entry points (see include/hann.h): context set-up, the client half, and the server-side scoring calls,
// each of which is a fixed sequence of kernel launches on the context's stream.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "internal.h"

#define CK(call)                                                                   \
    do {                                                                           \
        cudaError_t e_ = (call);                                                   \
        if (e_ != cudaSuccess) {                                                   \
            c->err = std::string(#call) + ": " + cudaGetErrorString(e_);           \
            return HANN_ECUDA;                                                     \
        }                                                                          \
    } while (0)

#define RET(call)                      \
    do {                               \
        int r_ = (call);               \
        if (r_ != HANN_OK) return r_;  \
    } while (0)

namespace {

int fail(hann_ctx* c, int code, const char* msg) {
    if (c) c->err = msg;
    return code;
}

inline int64_t align256(int64_t x) { return (x + 255) & ~(int64_t)255; }

// Waits for the context's stream, then reads and clears the word a kernel raises when it gives up a bounded wait for an
// asynchronous copy.  Every entry point that synchronises ends with this, so a call that returns HANN_OK has results that
// no aborted kernel produced.  (The word lives in mapped page-locked host memory: reading it costs no copy.)
int sync_and_check(hann_ctx* c) {
    cudaError_t e_ = cudaStreamSynchronize(c->stream);
    if (e_ != cudaSuccess) {
        c->err = std::string("cudaStreamSynchronize: ") + cudaGetErrorString(e_);
        return HANN_ECUDA;
    }
    const int word = *(volatile int*)c->kflag_host;
    if (word) {
        *(volatile int*)c->kflag_host = 0;
        if (word & 0x10000) {
            c->err = "a kernel's index range check failed (debug build), source line " + std::to_string(word & 0xFFFF) +
                     "; the access was skipped, results of the last calls are invalid";
            return HANN_ECUDA;
        }
        return fail(c, HANN_ECUDA, "a kernel gave up a bounded wait for an asynchronous copy; results of the last calls are invalid");
    }
    return HANN_OK;
}

// bump allocator over a caller-provided workspace.  With a context whose canaries are switched on (hann_debug_canaries) every
// sub-buffer is followed by a guard of 256 bytes that is filled with a pattern when it is carved and checked by
// hann_debug_verify: a kernel that writes past the end of its sub-buffer is found without any memory checker.
struct Arena {
    char* base;
    int64_t off, cap;
    hann_ctx* dbg = nullptr;
    template <typename T>
    T* take(int64_t count) {
        int64_t bytes = align256(count * (int64_t)sizeof(T));
        const bool guard = dbg && dbg->canaries;
        if (off + bytes + (guard ? 256 : 0) > cap) return nullptr;
        T* p = (T*)(base + off);
        off += bytes;
        if (guard) {
            // guards of earlier calls that lie inside what is carved now are about to be overwritten legitimately: forget them
            const char *lo = (const char*)p, *hi = base + off + 256;
            auto& gs = dbg->guards;
            gs.erase(std::remove_if(gs.begin(), gs.end(), [&](u64* g) { return (const char*)g + 256 > lo && (const char*)g < hi; }), gs.end());
            if (launch_guard_fill(dbg, (u64*)(base + off)) == HANN_OK) gs.push_back((u64*)(base + off));
            off += 256;
        }
        return p;
    }
};

struct DeviceGuard {
    int prev;
    bool ok;
    explicit DeviceGuard(int dev) {
        ok = cudaGetDevice(&prev) == cudaSuccess && cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        if (ok) cudaSetDevice(prev);
    }
};

int ensure_scratch(hann_ctx* c, int64_t bytes) {
    if (bytes <= c->scratch_bytes) return HANN_OK;
    CK(cudaStreamSynchronize(c->stream));
    if (c->scratch) cudaFree(c->scratch);
    c->scratch = nullptr;
    c->scratch_bytes = 0;
    if (cudaMalloc(&c->scratch, (size_t)bytes) != cudaSuccess) {
        cudaGetLastError();
        return fail(c, HANN_ENOMEM, "device allocation of the exchange scratch failed");
    }
    c->scratch_bytes = bytes;
    return HANN_OK;
}

// per-call timing with CUDA events on the context's stream
struct Timer {
    hann_ctx* c;
    int kind;
    Timer(hann_ctx* c_, int kind_) : c(c_), kind(kind_) {
        if (c->timing) cudaEventRecord(c->ev[kind][0], c->stream);
    }
    ~Timer() {
        if (c->timing) {
            cudaEventRecord(c->ev[kind][1], c->stream);
            c->ev_pending[kind] = 1;
        }
    }
};

int64_t ks_item_words(const hann_ctx* c) {
    // per item: c1 coefficients, digits, u, lifted, one temporary ciphertext
    const int64_t L = c->L, N = c->N;
    return L * N + L * (L + 1) * N + 2 * (L + 1) * N + 2 * L * N + 2 * L * N;
}

// words of workspace the lazy rotate-and-sum needs per block of a round: G-1 terms (c1 coefficients, digits, key product)
// and one ModDown (special-prime limb of the sum, its lift)
int64_t lazy_block_words(const hann_ctx* c) {
    const int64_t L = c->L, N = c->N, G1 = c->G - 1;
    return G1 * (L * N + L * (L + 1) * N + 2 * (L + 1) * N) + 2 * N + 2 * L * N;
}

int64_t prepare_words(const hann_ctx* c) {
    const int64_t L = c->L, N = c->N, nb = std::max(c->B - 1, 1);
    return L * N + L * (L + 1) * N + nb * (2 * (L + 1) * N + 2 * L * N);
}

constexpr int64_t kSlack = 16 * 256;  // room for the alignment of a dozen sub-buffers

// the four sub-buffers of ONE key switch (hann_keyswitch, hann_keyswitch_static): input copy, digits, u, lifted
struct KsBuffers {
    u64 *c1c, *digits, *u, *lifted;
};
bool carve_keyswitch(const hann_ctx* c, Arena& ar, KsBuffers& b) {
    const int64_t L = c->L, N = c->N;
    b.c1c = ar.take<u64>(L * N);
    b.digits = ar.take<u64>(L * (L + 1) * N);
    b.u = ar.take<u64>(2 * (L + 1) * N);
    b.lifted = ar.take<u64>(2 * L * N);
    return b.c1c && b.digits && b.u && b.lifted;
}

// canonical (host or device) -> internal: copy, forward transform of count polynomials of L limbs
int import_polys(hann_ctx* c, const u64* canonical, int64_t npolyL, u64* dst) {
    const int64_t words = npolyL * c->L * c->N;
    CK(cudaMemcpyAsync(dst, canonical, words * 8, cudaMemcpyDefault, c->stream));
    return launch_ntt_fwd(c, dst, npolyL * c->L, c->N, limbmap_q(c));
}

// internal -> canonical through a device staging buffer
int export_polys(hann_ctx* c, const u64* src, int64_t npolyL, u64* staging, u64* canonical_out) {
    const int64_t words = npolyL * c->L * c->N;
    CK(cudaMemcpyAsync(staging, src, words * 8, cudaMemcpyDeviceToDevice, c->stream));
    RET(launch_ntt_inv(c, staging, npolyL * c->L, c->N, limbmap_q(c)));
    CK(cudaMemcpyAsync(canonical_out, staging, words * 8, cudaMemcpyDefault, c->stream));
    return HANN_OK;
}

int polys_of_kind(int kind) {
    switch (kind) {
        case HANN_KIND_POLY:
        case HANN_KIND_PT: return 1;
        case HANN_KIND_CT: return 2;
        default: return 0;
    }
}

// secret key residues in the transform domain for limbs 0..nlimbs-1, into dst[nlimbs][N]; s8 is device scratch [N]
int upload_secret(hann_ctx* c, const int8_t* s_host, int nlimbs, int8_t* s8, u64* dst) {
    CK(cudaMemcpyAsync(s8, s_host, c->N, cudaMemcpyHostToDevice, c->stream));
    RET(launch_lift_i8(c, s8, nlimbs, dst));
    LimbMap lm = nlimbs == c->L + 1 ? limbmap_qp(c) : limbmap_q(c);
    return launch_ntt_fwd(c, dst, nlimbs, c->N, lm);
}

// ---- one key switch round on `items` polynomials ---------------------------------------------------------------
// c1c[items][L][N] (the polynomials to switch, transform domain, item stride L*N; overwritten) -> u, lifted; combine is
// left to the caller because its sources and targets differ between the callers.
// gather_src (optional): the polynomials to switch still lie at gather_src + item * gather_stride (L limbs each); they are
// brought into c1c on the way (by the inverse pass itself where its bulk-copy kernel applies, by a strided copy otherwise).
int ks_digits_to_lifted(hann_ctx* c, u64* c1c, int64_t items, u64* digits, int64_t digit_stride, int rot0, int rot_inc,
                        int64_t u_items, u64* u, u64* lifted, const u64* gather_src = nullptr, int64_t gather_stride = 0) {
    const int L = c->L, N = c->N;
    const int64_t LN = (int64_t)L * N;
    const bool fused_gather = gather_src && ks_lift_available(c) && ntt_inv_pass_b_gathers(c, gather_src, c1c) && (gather_stride & 1) == 0;
    if (gather_src && !fused_gather)
        RET(launch_copy2d(c, c1c, LN, gather_src, gather_stride, LN, items));
    if (ks_lift_available(c)) {
        // c1c arrives in the transform domain: inverse pass B', then one kernel finishes the inverse, lifts the digits
        // and starts their forward transforms; the same again for ModDown
        if (fused_gather) RET(launch_ntt_inv_pass_b_from(c, gather_src, gather_stride, c1c, items * L, N, limbmap_q(c)));
        else RET(launch_ntt_inv_pass_b(c, c1c, items * L, N, limbmap_q(c)));
        RET(launch_ks_lift(c, c1c, N, items * L, limbmap_q(c), digits, L + 1, 0));
        RET(launch_ntt_fwd_pass_b(c, digits, items * L * (L + 1), N, limbmap_qp(c)));
        RET(launch_ks_inner(c, digits, digit_stride, rot0, rot_inc, u_items, u));
        RET(launch_ntt_inv_pass_b(c, u + (int64_t)L * N, u_items * 2, (int64_t)(L + 1) * N, limbmap_single(L)));
        RET(launch_ks_lift(c, u + (int64_t)L * N, (int64_t)(L + 1) * N, u_items * 2, limbmap_single(L), lifted, L, 0));
        RET(launch_ntt_fwd_pass_b(c, lifted, u_items * 2 * L, N, limbmap_q(c)));
        return HANN_OK;
    }
    RET(launch_ntt_inv(c, c1c, items * L, N, limbmap_q(c)));
    RET(launch_lift_digits(c, c1c, (int64_t)L * N, items, digits));
    RET(launch_ntt_fwd(c, digits, items * L * (L + 1), N, limbmap_qp(c)));
    RET(launch_ks_inner(c, digits, digit_stride, rot0, rot_inc, u_items, u));
    // special-prime limbs of u back to coefficients (in place), lift, transform
    RET(launch_ntt_inv(c, u + (int64_t)L * N, u_items * 2, (int64_t)(L + 1) * N, limbmap_single(L)));
    RET(launch_moddown_lift(c, u, u_items * 2, lifted));
    RET(launch_ntt_fwd(c, lifted, u_items * 2 * L, N, limbmap_q(c)));
    return HANN_OK;
}

}  // namespace

int ntt_configure(hann_ctx* c);
int static_scratch_resolve(hann_ctx* c, void** out);

// bytes of 256-byte aligned workspace one hann_keyswitch needs: measured by running its own carving on an empty arena
int64_t keyswitch_ws_bytes(const hann_ctx* c) {
    Arena ar{nullptr, 0, INT64_MAX / 2};
    KsBuffers kb;
    ar.base = (char*)256;  // any non-null base: the carving only does pointer arithmetic
    carve_keyswitch(c, ar, kb);
    return ar.off;
}

// ================================================================================================ context

extern "C" int hann_ctx_create(const hann_params* prm, hann_ctx** out) {
    if (!prm || !out) return HANN_EINVAL;
    if (prm->logN < 4 || prm->logN > 16 || prm->L < 1 || prm->L > HANN_MAX_PRIMES) return HANN_EINVAL;
    const int N = 1 << prm->logN, n = N / 2, L = prm->L;
    if (prm->R < 1 || prm->B < 1 || prm->R % prm->B || n % prm->R) return HANN_EINVAL;
    if (prm->log_scale < 1 || prm->log_scale > 60) return HANN_EINVAL;
    u64 mods[HANN_MAXL1];
    for (int i = 0; i < L; i++) mods[i] = prm->q[i];
    mods[L] = prm->p;
    for (int i = 0; i <= L; i++) {
        if (mods[i] >= (1ULL << 62) || mods[i] < 3 || (mods[i] - 1) % (2 * (u64)N) || !hm::is_prime(mods[i])) return HANN_EINVAL;
        for (int k = 0; k < i; k++)
            if (mods[k] == mods[i]) return HANN_EINVAL;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || prm->device < 0 || prm->device >= ndev) {
        cudaGetLastError();
        return HANN_ECUDA;
    }
    hann_ctx* c = new (std::nothrow) hann_ctx();
    if (!c) return HANN_ENOMEM;
    c->prm = *prm;
    c->logN = prm->logN; c->N = N; c->n = n; c->L = L; c->R = prm->R; c->B = prm->B; c->G = prm->R / prm->B;
    c->ntt_tau = prm->logN >= 10 ? 1 : 0;
    c->host_limbs = L;
    c->device = prm->device;
    c->stream = (cudaStream_t)prm->stream;
    DeviceGuard dg(c->device);
    if (!dg.ok) { delete c; return HANN_ECUDA; }

    // per-limb constants and transform tables
    // tables of (w, floor(w * 2^64 / q)) pairs, [L+1][N][2]
    std::vector<u64> twf((size_t)(L + 1) * N * 2), twi((size_t)(L + 1) * N * 2);
    std::vector<double> twf64((size_t)(L + 1) * N * 2), twi64((size_t)(L + 1) * N * 2);
    std::vector<u64> pw(N), ipw(N);
    for (int i = 0; i <= L; i++) {
        const u64 q = mods[i];
        c->mod[i] = q;
        LimbConst& lc = c->lt.c[i];
        lc.q = q;
        lc.mu = (u64)((((unsigned __int128)1) << 64) / q);
        lc.c64 = (u64)((((unsigned __int128)1) << 64) % q);
        lc.c64s = hm::shoup(lc.c64, q);
        lc.ninv = hm::invmod((u64)N % q, q);
        lc.ninv_s = hm::shoup(lc.ninv, q);
        lc.half = q / 2;
        {
            const double nb = lc.ninv > q / 2 ? -(double)(q - lc.ninv) : (double)lc.ninv;
            lc.ninv_bal = nb;
            lc.ninv_q = nb / (double)q;
        }
        if (i < L) {
            lc.pmod = prm->p % q;
            lc.pinv = hm::invmod(lc.pmod, q);
            lc.pinv_s = hm::shoup(lc.pinv, q);
        } else {
            lc.pmod = 0; lc.pinv = 0; lc.pinv_s = 0;
        }
        const u64 psi = hm::find_psi(q, N), ipsi = hm::invmod(psi, q);
        pw[0] = ipw[0] = 1;
        for (int k = 1; k < N; k++) {
            pw[k] = hm::mulmod(pw[k - 1], psi, q);
            ipw[k] = hm::mulmod(ipw[k - 1], ipsi, q);
        }
        for (int k = 0; k < N; k++) {
            const int br = hm::bitrev(k, c->logN);
            const size_t o = ((size_t)i * N + k) * 2;
            twf[o] = pw[br];  twf[o + 1] = hm::shoup(pw[br], q);
            twi[o] = ipw[br]; twi[o + 1] = hm::shoup(ipw[br], q);
            // balanced copies for the binary64 path (exact for q < 2^53; only used when q < 2^50)
            const double wb = pw[br] > q / 2 ? -(double)(q - pw[br]) : (double)pw[br];
            const double iwb = ipw[br] > q / 2 ? -(double)(q - ipw[br]) : (double)ipw[br];
            twf64[o] = wb;  twf64[o + 1] = wb / (double)q;
            twi64[o] = iwb; twi64[o + 1] = iwb / (double)q;
        }
    }
    // encode tables
    const int nh = std::max(n / 2, 1);
    std::vector<double2> T(nh), U(n);
    c->hU_re.resize(n); c->hU_im.resize(n); c->h_uidx.resize(n);
    for (int t = 0; t < nh; t++) { double cs, sn; hm::unit_root(t, n, &cs, &sn); T[t] = make_double2(cs, -sn + 0.0); }
    for (int k = 0; k < n; k++) {
        double cs, sn; hm::unit_root(k, 2L * N, &cs, &sn);
        U[k] = make_double2(cs, -sn + 0.0);
        c->hU_re[k] = U[k].x; c->hU_im[k] = U[k].y;
    }
    std::vector<int32_t> jinv(n);
    std::vector<unsigned> gal(n);
    {
        long g = 1;
        for (int j = 0; j < n; j++) {
            gal[j] = (unsigned)g;
            c->h_uidx[j] = (int32_t)((g - 1) / 4);
            jinv[(g - 1) / 4] = j;
            g = (g * 5) % (2L * N);
        }
    }
    // the FFT runs on bit-reversed input: position pos of its input array takes slot jinv[brev(pos)]
    std::vector<int32_t> jpos(n);
    for (int pos = 0; pos < n; pos++) jpos[pos] = jinv[hm::bitrev(pos, c->logN - 1)];
    const size_t twb = (size_t)(L + 1) * N * 16;
    bool ok = cudaMalloc(&c->tw_fwd, twb) == cudaSuccess && cudaMalloc(&c->tw_inv, twb) == cudaSuccess &&
              cudaMalloc(&c->tw_fwd_f64, twb) == cudaSuccess && cudaMalloc(&c->tw_inv_f64, twb) == cudaSuccess &&
              cudaMalloc(&c->lt_dev, sizeof(LimbTable)) == cudaSuccess &&
              cudaHostAlloc((void**)&c->kflag_host, sizeof(int), cudaHostAllocMapped) == cudaSuccess &&
              cudaHostGetDevicePointer((void**)&c->kflag, c->kflag_host, 0) == cudaSuccess &&
              cudaMalloc(&c->fft_T, nh * sizeof(double2)) == cudaSuccess && cudaMalloc(&c->fft_U, n * sizeof(double2)) == cudaSuccess &&
              cudaMalloc(&c->jinv, n * sizeof(int32_t)) == cudaSuccess && cudaMalloc(&c->galois_dev, n * sizeof(unsigned)) == cudaSuccess &&
              cudaMalloc(&c->keytab_dev, n * sizeof(u64*)) == cudaSuccess;
    if (ok) {
        *c->kflag_host = 0;
        ok = cudaMemcpy(c->tw_fwd, twf.data(), twb, cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(c->tw_inv, twi.data(), twb, cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(c->tw_fwd_f64, twf64.data(), twb, cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(c->tw_inv_f64, twi64.data(), twb, cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(c->lt_dev, &c->lt, sizeof(LimbTable), cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(c->fft_T, T.data(), nh * sizeof(double2), cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(c->fft_U, U.data(), n * sizeof(double2), cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(c->jinv, jpos.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(c->galois_dev, gal.data(), n * sizeof(unsigned), cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemset(c->keytab_dev, 0, n * sizeof(u64*)) == cudaSuccess;
    }
    c->h_galois = gal;
    c->keytab_host.assign(n, nullptr);
    for (int k = 0; k < HANN_NKINDS && ok; k++)
        ok = cudaEventCreate(&c->ev[k][0]) == cudaSuccess && cudaEventCreate(&c->ev[k][1]) == cudaSuccess;
    if (ok)
        ok = cudaStreamCreateWithFlags(&c->aux_stream, cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 2 && ok; i++)
        ok = cudaStreamCreateWithFlags(&c->lane_stream[i], cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->lane_join[i], cudaEventDisableTiming) == cudaSuccess;
    if (ok)
        ok = cudaStreamCreateWithFlags(&c->up_stream, cudaStreamNonBlocking) == cudaSuccess &&
             cudaStreamCreateWithFlags(&c->down_stream, cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->down_done, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 2 && ok; i++)
        ok = cudaStreamCreateWithFlags(&c->score_stream[i], cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->score_join[i], cudaEventDisableTiming) == cudaSuccess;
    if (ok) ok = cudaEventCreateWithFlags(&c->prep_done, cudaEventDisableTiming) == cudaSuccess;
    if (ok) ok = ntt_configure(c) == HANN_OK;
    // a -DHANN_DEBUG build: the range checks of the kernels report through this context's error word
    if (ok) ok = debug_bind_keyswitch(c->kflag) == 0 && debug_bind_project(c->kflag) == 0 && debug_bind_encode(c->kflag) == 0;
    if (ok) {
        // look up the built-in scratch of hann_keyswitch_static now, while this device is current, so that the request-time
        // call only reads a cached address (a failure here is reported by that call, not by context creation)
        void* unused = nullptr;
        static_scratch_resolve(c, &unused);
        c->err.clear();
    }
    if (!ok) {
        cudaGetLastError();
        hann_ctx_destroy(c);
        return HANN_ECUDA;
    }
    *out = c;
    return HANN_OK;
}

extern "C" void hann_ctx_destroy(hann_ctx* c) {
    if (!c) return;
    DeviceGuard dg(c->device);
    cudaStreamSynchronize(c->stream);
    for (u64* k : c->keytab_host)
        if (k) cudaFree(k);
    cudaFree(c->tw_fwd); cudaFree(c->tw_inv); cudaFree(c->tw_fwd_f64); cudaFree(c->tw_inv_f64); cudaFree(c->lt_dev);
    if (c->kflag_host) cudaFreeHost(c->kflag_host);
    cudaFree(c->fft_T); cudaFree(c->fft_U); cudaFree(c->jinv); cudaFree(c->galois_dev); cudaFree(c->keytab_dev);
    if (c->scratch) cudaFree(c->scratch);
    if (c->aux_stream) {
        cudaStreamSynchronize(c->aux_stream);
        cudaStreamDestroy(c->aux_stream);
    }
    for (int i = 0; i < 2; i++) {
        if (c->lane_stream[i]) {
            cudaStreamSynchronize(c->lane_stream[i]);
            cudaStreamDestroy(c->lane_stream[i]);
        }
        if (c->lane_join[i]) cudaEventDestroy(c->lane_join[i]);
    }
    for (cudaEvent_t e : c->blk_ev) cudaEventDestroy(e);
    for (cudaEvent_t e : c->grp_ev) cudaEventDestroy(e);
    for (cudaEvent_t e : c->enc_ev) cudaEventDestroy(e);
    for (cudaEvent_t e : {c->score_join[0], c->score_join[1], c->prep_done})
        if (e) cudaEventDestroy(e);
    for (cudaStream_t st : {c->up_stream, c->down_stream, c->score_stream[0], c->score_stream[1]})
        if (st) {
            cudaStreamSynchronize(st);
            cudaStreamDestroy(st);
        }
    if (c->down_done) cudaEventDestroy(c->down_done);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_join) cudaEventDestroy(c->ev_join);
    for (auto& r : c->krec) {
        if (r.a) cudaEventDestroy(r.a);
        if (r.b) cudaEventDestroy(r.b);
    }
    for (int k = 0; k < HANN_NKINDS; k++) {
        if (c->ev[k][0]) cudaEventDestroy(c->ev[k][0]);
        if (c->ev[k][1]) cudaEventDestroy(c->ev[k][1]);
    }
    cudaGetLastError();
    delete c;
}

extern "C" int64_t hann_sizeof(const hann_ctx* c, int what) {
    if (!c) return HANN_EINVAL;
    const int64_t L = c->L, N = c->N;
    switch (what) {
        case HANN_SIZE_POLY: return L * N * 8;
        case HANN_SIZE_CT: return 2 * L * N * 8;
        case HANN_SIZE_BABY: return (int64_t)c->B * 2 * L * N * 8;
        case HANN_SIZE_PT_BLOCK: return (int64_t)c->R * L * (N / 2) * 8;
        case HANN_SIZE_INNER: return (int64_t)c->G * 2 * L * N * 8;
        case HANN_SIZE_EVK: return L * 2 * (L + 1) * N * 8;
        case HANN_SIZE_ROWS_PER_BLOCK: return c->n;
        case HANN_SIZE_CTDB_BLOCK: return (int64_t)c->R * 2 * L * N * 8;
        default: return HANN_EINVAL;
    }
}

// hann_query_level and hann_score_level_host cut a level into groups of blocks that are scored (multiply-accumulate,
// rotate-and-sum) on two scoring streams while the following groups are still encoded: number of groups and the
// rotate-and-sum workspace each scoring stream needs
static void level_groups(const hann_ctx* c, int64_t nblk, int* ng_out, int64_t* ws_score_out) {
    int64_t ng = c->host_groups;
    if (ng <= 0) ng = nblk <= 24 ? (nblk + 2) / 3 : (nblk + 3) / 4;  // groups of three to four blocks
    ng = std::max<int64_t>(1, std::min<int64_t>(ng, nblk));
    const int64_t gmax = nblk - nblk * (ng - 1) / ng;
    *ng_out = (int)ng;
    *ws_score_out = ng > 1 ? align256(std::max(ks_item_words(c) * std::min<int64_t>(gmax, 8), lazy_block_words(c) * std::min<int64_t>(gmax, 4)) * 8 + kSlack) : 0;
}

extern "C" int64_t hann_workspace_bytes(const hann_ctx* c, int64_t max_blocks) {
    if (!c || max_blocks < 0) return HANN_EINVAL;
    const int64_t items = std::max<int64_t>(1, std::min<int64_t>(max_blocks, 8));
    int64_t w = std::max(ks_item_words(c) * items, prepare_words(c)) * 8;
    w = std::max(w, (ks_item_words(c) + (int64_t)c->L * c->N) * 8);  // hann_keyswitch permutes its input first
    // hann_score_level_ctdb, hann_multiply: per item one degree-2 sum + its key switch
    w = std::max(w, (ks_item_words(c) + 3 * (int64_t)c->L * c->N) * items * 8);
    w = std::max(w, lazy_block_words(c) * std::min<int64_t>(items, 4) * 8);  // hann_rotate_sum_lazy: up to four blocks per round
    w = std::max(w, encode_ws_bytes(c));
    // hann_query_level runs query_prepare and encode_candidates side by side, each in its own part
    w = std::max(w, align256(prepare_words(c) * 8 + kSlack) + encode_ws_bytes(c));
    // ... and, with more than one group of blocks, the scoring of a group beside the encoding of the next
    int ng = 1;
    int64_t ws_score = 0;
    if (c->host_groups > 1) level_groups(c, std::max<int64_t>(1, max_blocks), &ng, &ws_score);
    w = std::max(w, align256(prepare_words(c) * 8 + kSlack) + align256(encode_ws_bytes(c)) + 2 * ws_score);
    return w + kSlack;
}

extern "C" int64_t hann_keyswitch_bytes(const hann_ctx* c) { return c ? keyswitch_ws_bytes(c) : HANN_EINVAL; }

extern "C" int hann_sync(hann_ctx* c) {
    if (!c) return HANN_EINVAL;
    DeviceGuard dg(c->device);
    return sync_and_check(c);
}

extern "C" int hann_selftest_bounded_wait(hann_ctx* c, int limit_ms, double* waited_ms) {
    if (!c) return HANN_EINVAL;
    if (limit_ms < 1 || limit_ms > 1000) return fail(c, HANN_EINVAL, "hann_selftest_bounded_wait: limit must be 1..1000 ms");
    DeviceGuard dg(c->device);
    RET(ensure_scratch(c, 256));
    unsigned long long* w = (unsigned long long*)c->scratch;
    CK(cudaMemsetAsync(w, 0, 8, c->stream));
    RET(launch_wait_selftest(c, (unsigned long long)limit_ms * 1000000ULL, w));
    unsigned long long ns = 0;
    CK(cudaMemcpyAsync(&ns, w, 8, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    if (waited_ms) *waited_ms = (double)ns * 1e-6;
    return HANN_OK;
}

extern "C" int hann_debug_build(void) {
#ifdef HANN_DEBUG
    return 1;
#else
    return 0;
#endif
}

extern "C" int hann_debug_canaries(hann_ctx* c, int enable) {
    if (!c) return HANN_EINVAL;
    c->canaries = enable ? 1 : 0;
    c->guards.clear();
    return HANN_OK;
}

extern "C" int hann_debug_verify(hann_ctx* c, int64_t* guards_checked, int64_t* guards_damaged) {
    if (!c) return HANN_EINVAL;
    if (!guards_checked || !guards_damaged) return fail(c, HANN_EINVAL, "hann_debug_verify: null pointer");
    DeviceGuard dg(c->device);
    const int64_t ng = (int64_t)c->guards.size();
    *guards_checked = ng;
    *guards_damaged = 0;
    if (ng == 0) return sync_and_check(c);
    // guard addresses and the damage counter go through the exchange scratch (this is a debugging call: it may allocate)
    RET(ensure_scratch(c, align256(ng * 8) + 256));
    u64** list = (u64**)c->scratch;
    unsigned long long* bad = (unsigned long long*)((char*)c->scratch + align256(ng * 8));
    CK(cudaMemcpyAsync(list, c->guards.data(), (size_t)ng * 8, cudaMemcpyHostToDevice, c->stream));
    const unsigned long long init[2] = {0ULL, ~0ULL};   // damaged guards, index of the first one
    CK(cudaMemcpyAsync(bad, init, 16, cudaMemcpyHostToDevice, c->stream));
    RET(launch_guard_verify(c, list, ng, bad));
    unsigned long long res[2] = {0, 0};
    CK(cudaMemcpyAsync(res, bad, 16, cudaMemcpyDeviceToHost, c->stream));
    RET(sync_and_check(c));
    *guards_damaged = (int64_t)res[0];
    c->guards.clear();
    if (res[0]) {
        c->err = "hann_debug_verify: a kernel wrote past the end of a workspace sub-buffer (" + std::to_string(res[0]) + " of " +
                 std::to_string(ng) + " guards damaged, the first one is guard " + std::to_string(res[1]) + " in carving order)";
        return HANN_ECUDA;
    }
    return HANN_OK;
}

extern "C" const char* hann_last_error(const hann_ctx* c) { return c ? c->err.c_str() : "null context"; }

extern "C" int hann_set_timing(hann_ctx* c, int enable) {
    if (!c) return HANN_EINVAL;
    c->timing = enable ? 1 : 0;
    return HANN_OK;
}

extern "C" int hann_set_tuning(hann_ctx* c, int what, int value) {
    if (!c) return HANN_EINVAL;
    switch (what) {
        case HANN_TUNE_ENCODE_GROUP:
            if (value < 1) return fail(c, HANN_EINVAL, "hann_set_tuning: encode group must be positive");
            c->encode_group = value;
            return HANN_OK;
        case HANN_TUNE_HOST_LIMBS:
            if (value < 1 || value > c->L) return fail(c, HANN_EINVAL, "hann_set_tuning: host limbs must be in 1..L");
            c->host_limbs = value;
            return HANN_OK;
        case HANN_TUNE_HOST_GROUPS:
            if (value < 0) return fail(c, HANN_EINVAL, "hann_set_tuning: host groups must be 0 (automatic) or positive");
            c->host_groups = value;
            return HANN_OK;
        case HANN_TUNE_ENCODE_SYMMETRY:
            c->encode_sym = value ? 1 : 0;
            return HANN_OK;
        case HANN_TUNE_GIANT_LAZY:
            c->giant_lazy = value ? 1 : 0;
            return HANN_OK;
        case HANN_TUNE_LAZY_LANES:
            if (value < 1 || value > 4) return fail(c, HANN_EINVAL, "hann_set_tuning: lazy lanes must be 1..4");
            c->lazy_lanes = value;
            return HANN_OK;
        case HANN_TUNE_MAC_F64:
            c->mac_f64 = value ? 4 : 0;
            return HANN_OK;
        case HANN_TUNE_PAIR_B32:
            c->pair_b32 = value ? 1 : 0;
            return HANN_OK;
        default: return fail(c, HANN_EINVAL, "hann_set_tuning: unknown knob");
    }
}

extern "C" int hann_get_stats(hann_ctx* c, hann_stats* out) {
    if (!c || !out) return HANN_EINVAL;
    DeviceGuard dg(c->device);
    float* field[HANN_NKINDS] = {&c->stats.ms_query_prepare, &c->stats.ms_encode, &c->stats.ms_score_level,
                                 &c->stats.ms_rotate_sum, &c->stats.ms_keyswitch};
    for (int k = 0; k < HANN_NKINDS; k++)
        if (c->ev_pending[k]) {
            CK(cudaEventSynchronize(c->ev[k][1]));
            CK(cudaEventElapsedTime(field[k], c->ev[k][0], c->ev[k][1]));
            c->ev_pending[k] = 0;
        }
    *out = c->stats;
    return HANN_OK;
}

static const char* kKernelNames[KC_COUNT] = {"ntt_fwd_a", "ntt_fwd_b", "ntt_inv_b", "ntt_inv_a", "fft_a", "fft_b", "mac",
                                             "lift_digits", "ks_inner", "moddown_lift", "moddown_combine", "permute", "other",
                                             "ks_inner_keys"};

extern "C" int hann_kernel_classes(void) { return KC_COUNT; }
extern "C" const char* hann_kernel_name(int cls) { return cls >= 0 && cls < KC_COUNT ? kKernelNames[cls] : ""; }

extern "C" int hann_kernel_profile(hann_ctx* c, int enable) {
    if (!c) return HANN_EINVAL;
    DeviceGuard dg(c->device);
    CK(cudaStreamSynchronize(c->stream));
    c->kprof = enable ? 1 : 0;
    c->krec_used = 0;
    return HANN_OK;
}

extern "C" int hann_kernel_times(hann_ctx* c, double* ms, uint64_t* launches) {
    if (!c || !ms || !launches) return HANN_EINVAL;
    DeviceGuard dg(c->device);
    CK(cudaStreamSynchronize(c->stream));
    for (int k = 0; k < KC_COUNT; k++) { ms[k] = 0; launches[k] = 0; }
    for (size_t i = 0; i < c->krec_used; i++) {
        float t = 0;
        CK(cudaEventElapsedTime(&t, c->krec[i].a, c->krec[i].b));
        ms[c->krec[i].cls] += t;
        launches[c->krec[i].cls]++;
    }
    c->krec_used = 0;
    return HANN_OK;
}

// ================================================================================================ exchange

extern "C" int hann_import(hann_ctx* c, int kind, const uint64_t* canonical, int64_t count, void* internal_dev) {
    if (!c) return HANN_EINVAL;
    const int pk = polys_of_kind(kind);
    if (!pk || !canonical || !internal_dev || count < 0) return fail(c, HANN_EINVAL, "hann_import: bad argument");
    DeviceGuard dg(c->device);
    if (kind == HANN_KIND_PT) {
        // transformed in full in the scratch, first halves kept (a plaintext is the encoding of a real slot vector)
        const int64_t piece = 64, LN = (int64_t)c->L * c->N;
        RET(ensure_scratch(c, piece * LN * 8));
        for (int64_t p0 = 0; p0 < count; p0 += piece) {
            const int64_t np = std::min(piece, count - p0);
            RET(import_polys(c, canonical + p0 * LN, np, (u64*)c->scratch));
            CK(cudaMemcpy2DAsync((u64*)internal_dev + p0 * (LN / 2), (size_t)c->n * 8, c->scratch, (size_t)c->N * 8, (size_t)c->n * 8,
                                 (size_t)np * c->L, cudaMemcpyDeviceToDevice, c->stream));
        }
        RET(sync_and_check(c));
        return HANN_OK;
    }
    RET(import_polys(c, canonical, count * pk, (u64*)internal_dev));
    RET(sync_and_check(c));
    return HANN_OK;
}

extern "C" int hann_expand_uniform(hann_ctx* c, uint64_t seed, uint64_t stream, uint64_t* a_out) {
    if (!c) return HANN_EINVAL;
    if (!a_out) return fail(c, HANN_EINVAL, "hann_expand_uniform: null pointer");
    DeviceGuard dg(c->device);
    const int64_t LN = (int64_t)c->L * c->N;
    RET(ensure_scratch(c, LN * 8));
    RET(launch_expand_uniform(c, seed, stream, (u64*)c->scratch));
    CK(cudaMemcpyAsync(a_out, c->scratch, LN * 8, cudaMemcpyDefault, c->stream));
    RET(sync_and_check(c));
    return HANN_OK;
}

extern "C" int hann_import_seeded_ct(hann_ctx* c, const uint64_t* c0, uint64_t seed, uint64_t stream, void* ct_dev) {
    if (!c) return HANN_EINVAL;
    if (!c0 || !ct_dev) return fail(c, HANN_EINVAL, "hann_import_seeded_ct: null pointer");
    DeviceGuard dg(c->device);
    const int64_t LN = (int64_t)c->L * c->N;
    u64* ct = (u64*)ct_dev;
    CK(cudaMemcpyAsync(ct, c0, LN * 8, cudaMemcpyDefault, c->stream));
    RET(launch_expand_uniform(c, seed, stream, ct + LN));
    return launch_ntt_fwd(c, ct, 2 * c->L, c->N, limbmap_q(c));
}

extern "C" int hann_export(hann_ctx* c, int kind, const void* internal_dev, int64_t count, uint64_t* canonical_out) {
    if (!c) return HANN_EINVAL;
    const int pk = polys_of_kind(kind);
    if (!pk || !canonical_out || !internal_dev || count < 0) return fail(c, HANN_EINVAL, "hann_export: bad argument");
    DeviceGuard dg(c->device);
    // staged in pieces of at most 64 polynomials so that the scratch stays small
    const int64_t total = count * pk, piece = 64;
    RET(ensure_scratch(c, piece * c->L * c->N * 8));
    for (int64_t p0 = 0; p0 < total; p0 += piece) {
        const int64_t np = std::min(piece, total - p0);
        if (kind == HANN_KIND_PT) {
            const int64_t LN = (int64_t)c->L * c->N;
            RET(launch_unpack_half(c, (const u64*)internal_dev + p0 * (LN / 2), np * c->L, (u64*)c->scratch));
            RET(launch_ntt_inv(c, (u64*)c->scratch, np * c->L, c->N, limbmap_q(c)));
            CK(cudaMemcpyAsync(canonical_out + p0 * LN, c->scratch, np * LN * 8, cudaMemcpyDefault, c->stream));
            continue;
        }
        RET(export_polys(c, (const u64*)internal_dev + p0 * c->L * c->N, np, (u64*)c->scratch, canonical_out + p0 * c->L * c->N));
    }
    RET(sync_and_check(c));
    return HANN_OK;
}

extern "C" int hann_export_limbs(hann_ctx* c, const void* internal_dev, int64_t npoly, int limbs, uint64_t* canonical_out) {
    if (!c) return HANN_EINVAL;
    if (!canonical_out || !internal_dev || npoly < 0) return fail(c, HANN_EINVAL, "hann_export_limbs: bad argument");
    if (limbs < 1 || limbs > c->L) return fail(c, HANN_ESHAPE, "hann_export_limbs: limb count out of range");
    DeviceGuard dg(c->device);
    const int64_t piece = 64, pw = (int64_t)limbs * c->N;
    RET(ensure_scratch(c, piece * pw * 8));
    for (int64_t p0 = 0; p0 < npoly; p0 += piece) {
        const int64_t np = std::min(piece, npoly - p0);
        u64* staging = (u64*)c->scratch;
        CK(cudaMemcpyAsync(staging, (const u64*)internal_dev + p0 * pw, np * pw * 8, cudaMemcpyDeviceToDevice, c->stream));
        RET(launch_ntt_inv(c, staging, np * limbs, c->N, limbmap_first(limbs)));
        CK(cudaMemcpyAsync(canonical_out + p0 * pw, staging, np * pw * 8, cudaMemcpyDefault, c->stream));
    }
    RET(sync_and_check(c));
    return HANN_OK;
}

extern "C" int64_t hann_compact_bytes(const hann_ctx* c, int64_t n_blocks, int keep) {
    if (!c || n_blocks < 0 || keep < 1 || keep > c->L) return HANN_EINVAL;
    return n_blocks * 2 * (int64_t)keep * c->N * 8;
}

extern "C" int hann_compact_scores(hann_ctx* c, const void* score_ct_dev, int64_t n_blocks, int keep, int rescale, void* out_dev,
                                   void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (n_blocks < 0 || (n_blocks > 0 && (!score_ct_dev || !out_dev))) return fail(c, HANN_EINVAL, "hann_compact_scores: bad argument");
    const int L = c->L, N = c->N;
    if (keep < 1 || keep > L - (rescale ? 1 : 0)) return fail(c, HANN_ESHAPE, "hann_compact_scores: keep must be in 1..L-1 (1..L without rescale)");
    if (n_blocks == 0) return HANN_OK;
    DeviceGuard dg(c->device);
    const u64* src = (const u64*)score_ct_dev;
    u64* out = (u64*)out_dev;
    const int64_t npoly = n_blocks * 2;
    if (!rescale) {
        // the first `keep` limbs of every polynomial: c0 + c1 s is the same integer modulo the smaller product
        CK(cudaMemcpy2DAsync(out, (size_t)keep * N * 8, src, (size_t)L * N * 8, (size_t)keep * N * 8, (size_t)npoly, cudaMemcpyDeviceToDevice,
                             c->stream));
        return HANN_OK;
    }
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_compact_scores: workspace missing or not 256-byte aligned");
    // per polynomial: the last limb back in coefficients (N words) and its lift into the kept limbs (keep * N words)
    const int64_t per = (int64_t)(1 + keep) * N * 8;
    int64_t ch = ((int64_t)ws_bytes - kSlack) / per;
    if (ch < 1) return fail(c, HANN_EWORKSPACE, "hann_compact_scores: workspace too small");
    ch = std::min(ch, npoly);
    Arena ar{(char*)ws, 0, (int64_t)ws_bytes, c};
    u64* t = ar.take<u64>(ch * N);
    u64* lifted = ar.take<u64>(ch * keep * N);
    if (!t || !lifted) return fail(c, HANN_EWORKSPACE, "hann_compact_scores: workspace too small");
    for (int64_t p0 = 0; p0 < npoly; p0 += ch) {
        const int64_t np = std::min(ch, npoly - p0);
        CK(cudaMemcpy2DAsync(t, (size_t)N * 8, src + (p0 * L + (L - 1)) * N, (size_t)L * N * 8, (size_t)N * 8, (size_t)np,
                             cudaMemcpyDeviceToDevice, c->stream));
        RET(launch_ntt_inv(c, t, np, N, limbmap_single(L - 1)));
        RET(launch_rescale_lift(c, t, np, keep, lifted));
        RET(launch_ntt_fwd(c, lifted, np * keep, N, limbmap_first(keep)));
        RET(launch_rescale_combine(c, src + p0 * L * N, lifted, np, keep, out + p0 * keep * N));
    }
    return HANN_OK;
}

// ================================================================================================ client side

extern "C" int hann_keygen_from_samples(hann_ctx* c, const int8_t* s, int n_rot, const int32_t* rot, const uint64_t* a,
                                        const int8_t* e, uint64_t* evk_out) {
    if (!c) return HANN_EINVAL;
    if (!s || !rot || !a || !e || !evk_out || n_rot < 0) return fail(c, HANN_EINVAL, "hann_keygen_from_samples: bad argument");
    const int L = c->L, N = c->N;
    for (int i = 0; i < n_rot; i++)
        if (rot[i] < 1 || rot[i] >= c->n) return fail(c, HANN_ESHAPE, "hann_keygen_from_samples: rotation out of range");
    DeviceGuard dg(c->device);
    const int64_t W = (int64_t)N, keyw = (int64_t)L * (L + 1) * W;
    // scratch: s_hat[L+1][N], A[L][L+1][N], AS[L][L+1][N], int8: s, s', e[L][N]
    const int64_t words = (L + 1) * W + 2 * keyw;
    RET(ensure_scratch(c, words * 8 + align256(N) * 2 + align256((int64_t)L * N) + kSlack));
    Arena ar{(char*)c->scratch, 0, c->scratch_bytes};
    u64* shat = ar.take<u64>((L + 1) * W);
    u64* A = ar.take<u64>(keyw);
    u64* AS = ar.take<u64>(keyw);
    int8_t* s8 = ar.take<int8_t>(N);
    int8_t* sp8 = ar.take<int8_t>(N);
    int8_t* e8 = ar.take<int8_t>((int64_t)L * N);
    RET(upload_secret(c, s, L + 1, s8, shat));
    std::vector<int8_t> sprime(N);
    for (int r = 0; r < n_rot; r++) {
        const unsigned k = c->h_galois[rot[r]];
        for (long i = 0; i < N; i++) {  // s'(X) = s(X^k)
            long ex = (i * (long)k) % (2L * N);
            if (ex < N) sprime[ex] = s[i];
            else sprime[ex - N] = (int8_t)(-s[i]);
        }
        const u64* a_r = a + (int64_t)r * keyw;
        CK(cudaMemcpyAsync(A, a_r, keyw * 8, cudaMemcpyHostToDevice, c->stream));
        CK(cudaMemcpyAsync(sp8, sprime.data(), N, cudaMemcpyHostToDevice, c->stream));
        CK(cudaMemcpyAsync(e8, e + (int64_t)r * L * N, (size_t)L * N, cudaMemcpyHostToDevice, c->stream));
        RET(launch_ntt_fwd(c, A, (int64_t)L * (L + 1), N, limbmap_qp(c)));
        RET(launch_mul(c, A, shat, L + 1, AS, (int64_t)L * (L + 1), limbmap_qp(c)));
        RET(launch_ntt_inv(c, AS, (int64_t)L * (L + 1), N, limbmap_qp(c)));
        RET(launch_evk_finish(c, AS, e8, sp8, AS));
        u64* out_r = evk_out + (int64_t)r * 2 * keyw;
        for (int j = 0; j < L; j++) {
            CK(cudaMemcpyAsync(out_r + ((int64_t)j * 2 + 0) * (L + 1) * W, AS + (int64_t)j * (L + 1) * W, (size_t)(L + 1) * W * 8,
                               cudaMemcpyDeviceToHost, c->stream));
            memcpy(out_r + ((int64_t)j * 2 + 1) * (L + 1) * W, a_r + (int64_t)j * (L + 1) * W, (size_t)(L + 1) * W * 8);
        }
        RET(sync_and_check(c));  // sprime (host) is reused by the next rotation
    }
    return HANN_OK;
}

extern "C" int hann_keygen_seeded(hann_ctx* c, uint64_t seed, int n_rot, const int32_t* rot, int8_t* s_out, uint64_t* evk_out) {
    if (!c) return HANN_EINVAL;
    if (!rot || !s_out || !evk_out || n_rot < 0) return fail(c, HANN_EINVAL, "hann_keygen_seeded: bad argument");
    const int L = c->L, N = c->N;
    for (int i = 0; i < n_rot; i++)
        if (rot[i] < 1 || rot[i] >= c->n) return fail(c, HANN_ESHAPE, "hann_keygen_seeded: rotation out of range");
    // streams of the counter hash: 16 secret, 17 uniform halves of the keys, 18/19 the two Box-Muller sub-streams
    hm::seeded_ternary(seed, 16, N, s_out);
    const int64_t keyw = (int64_t)L * (L + 1) * N;
    std::vector<u64> a((size_t)keyw);
    std::vector<int8_t> e((size_t)L * N);
    for (int r = 0; r < n_rot; r++) {
        {
            DeviceGuard dg(c->device);
            RET(ensure_scratch(c, keyw * 8));
            // counters are keyed by the ROTATION, not by its place in the list: a rotation's key does not depend on
            // which other keys are generated with it
            RET(launch_expand_uniform_qp(c, seed, 17, (u64)rot[r] * (u64)keyw, (u64*)c->scratch));
            CK(cudaMemcpyAsync(a.data(), c->scratch, keyw * 8, cudaMemcpyDeviceToHost, c->stream));
            RET(sync_and_check(c));
        }
        hm::seeded_gaussian(seed, 18, (u64)rot[r] * (u64)L * N, (long)L * N, 3.2, e.data());
        RET(hann_keygen_from_samples(c, s_out, 1, rot + r, a.data(), e.data(), evk_out + (int64_t)r * 2 * keyw));
    }
    return HANN_OK;
}

extern "C" int hann_keygen_relin_from_samples(hann_ctx* c, const int8_t* s, const uint64_t* a, const int8_t* e, uint64_t* evk_out) {
    if (!c) return HANN_EINVAL;
    if (!s || !a || !e || !evk_out) return fail(c, HANN_EINVAL, "hann_keygen_relin_from_samples: bad argument");
    const int L = c->L, N = c->N;
    DeviceGuard dg(c->device);
    const int64_t W = (int64_t)N, keyw = (int64_t)L * (L + 1) * W;
    RET(ensure_scratch(c, (2 * (L + 1) * W + 2 * keyw) * 8 + align256(N) + align256((int64_t)L * N) + kSlack));
    Arena ar{(char*)c->scratch, 0, c->scratch_bytes};
    u64* shat = ar.take<u64>((L + 1) * W);
    u64* s2 = ar.take<u64>((L + 1) * W);
    u64* A = ar.take<u64>(keyw);
    u64* AS = ar.take<u64>(keyw);
    int8_t* s8 = ar.take<int8_t>(N);
    int8_t* e8 = ar.take<int8_t>((int64_t)L * N);
    RET(upload_secret(c, s, L + 1, s8, shat));
    // s' = s^2: squared in the transform domain, back to coefficient-domain residues for the finish kernel
    RET(launch_mul(c, shat, shat, L + 1, s2, L + 1, limbmap_qp(c)));
    RET(launch_ntt_inv(c, s2, L + 1, N, limbmap_qp(c)));
    CK(cudaMemcpyAsync(A, a, keyw * 8, cudaMemcpyHostToDevice, c->stream));
    CK(cudaMemcpyAsync(e8, e, (size_t)L * N, cudaMemcpyHostToDevice, c->stream));
    RET(launch_ntt_fwd(c, A, (int64_t)L * (L + 1), N, limbmap_qp(c)));
    RET(launch_mul(c, A, shat, L + 1, AS, (int64_t)L * (L + 1), limbmap_qp(c)));
    RET(launch_ntt_inv(c, AS, (int64_t)L * (L + 1), N, limbmap_qp(c)));
    RET(launch_rlk_finish(c, AS, e8, s2, AS));
    for (int j = 0; j < L; j++) {
        CK(cudaMemcpyAsync(evk_out + ((int64_t)j * 2 + 0) * (L + 1) * W, AS + (int64_t)j * (L + 1) * W, (size_t)(L + 1) * W * 8,
                           cudaMemcpyDeviceToHost, c->stream));
        memcpy(evk_out + ((int64_t)j * 2 + 1) * (L + 1) * W, a + (int64_t)j * (L + 1) * W, (size_t)(L + 1) * W * 8);
    }
    RET(sync_and_check(c));
    return HANN_OK;
}

extern "C" int hann_encrypt_block(hann_ctx* c, const int8_t* s, const void* pt_dev, const uint64_t* a, const int8_t* e, void* ctdb_dev) {
    if (!c) return HANN_EINVAL;
    if (!s || !pt_dev || !a || !e || !ctdb_dev) return fail(c, HANN_EINVAL, "hann_encrypt_block: bad argument");
    const int L = c->L, N = c->N, R = c->R;
    const int64_t LN = (int64_t)L * N;
    DeviceGuard dg(c->device);
    // pieces of up to 16 plaintexts: a (transformed) lands in the ciphertext's second half, a*s and the transformed error in
    // the scratch
    const int piece = 16;
    RET(ensure_scratch(c, (LN + 2 * piece * LN) * 8 + align256(N) + align256((int64_t)piece * N) + kSlack));
    Arena ar{(char*)c->scratch, 0, c->scratch_bytes};
    u64* shat = ar.take<u64>(LN);
    u64* AS = ar.take<u64>(piece * LN);
    u64* EH = ar.take<u64>(piece * LN);
    int8_t* s8 = ar.take<int8_t>(N);
    int8_t* e8 = ar.take<int8_t>((int64_t)piece * N);
    RET(upload_secret(c, s, L, s8, shat));
    u64* ct = (u64*)ctdb_dev;
    const u64* pt = (const u64*)pt_dev;
    for (int r0 = 0; r0 < R; r0 += piece) {
        const int np = std::min(piece, R - r0);
        // c1 = transform of a, straight into place (polynomial r at ct + (2 r + 1) * LN)
        CK(cudaMemcpy2DAsync(ct + ((int64_t)r0 * 2 + 1) * LN, (size_t)2 * LN * 8, a + (int64_t)r0 * LN, (size_t)LN * 8, (size_t)LN * 8, (size_t)np,
                             cudaMemcpyDefault, c->stream));
        for (int r = 0; r < np; r++) RET(launch_ntt_fwd(c, ct + ((int64_t)(r0 + r) * 2 + 1) * LN, L, N, limbmap_q(c)));
        CK(cudaMemcpyAsync(e8, e + (int64_t)r0 * N, (size_t)np * N, cudaMemcpyHostToDevice, c->stream));
        for (int r = 0; r < np; r++) {
            RET(launch_mul(c, ct + ((int64_t)(r0 + r) * 2 + 1) * LN, shat, L, AS + (int64_t)r * LN, L, limbmap_q(c)));
            RET(launch_lift_i8(c, e8 + (int64_t)r * N, L, EH + (int64_t)r * LN));
        }
        RET(launch_ntt_fwd(c, EH, (int64_t)np * L, N, limbmap_q(c)));
        // c0 = pt - a*s + e, written at ct + 2 r * LN (the finish kernel strides its output by 2 * LN)
        RET(launch_encrypt_block_finish(c, pt + (int64_t)r0 * (LN / 2), AS, EH, ct + (int64_t)r0 * 2 * LN, np));
        RET(sync_and_check(c));  // e8 is reused by the next piece
    }
    return HANN_OK;
}

extern "C" int hann_encrypt_query(hann_ctx* c, const int8_t* s, const float* q, int dim, const uint64_t* a, const int8_t* e,
                                  uint64_t* ct_out) {
    if (!c) return HANN_EINVAL;
    if (!s || !q || !a || !e || !ct_out) return fail(c, HANN_EINVAL, "hann_encrypt_query: null pointer");
    if (dim < 1 || dim > c->R) return fail(c, HANN_ESHAPE, "hann_encrypt_query: dim must be in 1..R");
    const int L = c->L, N = c->N, n = c->n;
    DeviceGuard dg(c->device);
    const int64_t LN = (int64_t)L * N;
    RET(ensure_scratch(c, (4 * LN) * 8 + n * 8 + n * 16 + 2 * align256(N) + kSlack));
    Arena ar{(char*)c->scratch, 0, c->scratch_bytes};
    u64* shat = ar.take<u64>(LN);
    u64* A = ar.take<u64>(LN);
    u64* AS = ar.take<u64>(LN);
    u64* M = ar.take<u64>(LN);
    double* z = ar.take<double>(n);
    double2* fbuf = ar.take<double2>(n);
    int8_t* s8 = ar.take<int8_t>(N);
    int8_t* e8 = ar.take<int8_t>(N);
    std::vector<double> zh(n);
    for (int i = 0; i < n; i++) {
        int d = i % c->R;
        zh[i] = d < dim ? (double)q[d] : 0.0;
    }
    CK(cudaMemcpyAsync(z, zh.data(), n * 8, cudaMemcpyHostToDevice, c->stream));
    CK(cudaMemcpyAsync(A, a, LN * 8, cudaMemcpyHostToDevice, c->stream));
    CK(cudaMemcpyAsync(e8, e, N, cudaMemcpyHostToDevice, c->stream));
    RET(upload_secret(c, s, L, s8, shat));
    RET(launch_encode_slots(c, z, M, fbuf));
    RET(launch_ntt_fwd(c, A, L, N, limbmap_q(c)));
    RET(launch_mul(c, A, shat, L, AS, L, limbmap_q(c)));
    RET(launch_ntt_inv(c, AS, L, N, limbmap_q(c)));
    RET(launch_encrypt_finish(c, AS, e8, M, AS));
    CK(cudaMemcpyAsync(ct_out, AS, LN * 8, cudaMemcpyDeviceToHost, c->stream));
    RET(sync_and_check(c));
    memcpy(ct_out + LN, a, LN * 8);
    return HANN_OK;
}

// count ciphertexts of nl limbs each, ct [count][2][nl][N] canonical, plaintext scale 1 / inv_scale
static int decrypt_impl(hann_ctx* c, const int8_t* s, const uint64_t* ct, int64_t count, int nl, long double inv_scale,
                        double* scores, double* imag_or_null) {
    const int N = c->N, n = c->n;
    DeviceGuard dg(c->device);
    const int64_t LN = (int64_t)nl * N;
    RET(ensure_scratch(c, 4 * LN * 8 + align256(N) + kSlack));
    Arena ar{(char*)c->scratch, 0, c->scratch_bytes};
    u64* shat = ar.take<u64>(LN);
    u64* CT = ar.take<u64>(2 * LN);
    u64* MU = ar.take<u64>(LN);
    int8_t* s8 = ar.take<int8_t>(N);
    const LimbMap lm = limbmap_first(nl);
    CK(cudaMemcpyAsync(s8, s, N, cudaMemcpyHostToDevice, c->stream));
    RET(launch_lift_i8(c, s8, nl, shat));
    RET(launch_ntt_fwd(c, shat, nl, N, lm));
    std::vector<u64> mu(LN);
    std::vector<long double> real(N);
    std::vector<double> re(n), im(n);
    for (int64_t i = 0; i < count; i++) {
        CK(cudaMemcpyAsync(CT, ct + i * 2 * LN, 2 * LN * 8, cudaMemcpyDefault, c->stream));
        RET(launch_ntt_fwd(c, CT, 2 * nl, N, lm));
        RET(launch_mul(c, CT + LN, shat, nl, MU, nl, lm));   // c1 * s
        RET(launch_add(c, MU, CT, MU, nl, lm));              // + c0
        RET(launch_ntt_inv(c, MU, nl, N, lm));
        CK(cudaMemcpyAsync(mu.data(), MU, LN * 8, cudaMemcpyDeviceToHost, c->stream));
        RET(sync_and_check(c));
        hm::crt_to_real(mu.data(), nl, N, c->mod, real.data());
        // slots: a_k = (mu_k + i mu_{k+n}) conj(U[k]);  z_j * scale = sum_k a_k exp(+2 pi i u_j k / n)
        for (int k = 0; k < n; k++) {
            const double mr = (double)(real[k] * inv_scale), mi = (double)(real[k + n] * inv_scale);
            const double ur = c->hU_re[k], ui = -c->hU_im[k];
            re[k] = mr * ur - mi * ui;
            im[k] = mr * ui + mi * ur;
        }
        hm::fft_inplace(re.data(), im.data(), n, c->logN - 1, +1);
        for (int j = 0; j < n; j++) {
            scores[i * n + j] = re[c->h_uidx[j]];
            if (imag_or_null) imag_or_null[i * n + j] = im[c->h_uidx[j]];
        }
    }
    return HANN_OK;
}

extern "C" int hann_decrypt_scores(hann_ctx* c, const int8_t* s, const uint64_t* ct, int64_t count, int log_scale_out,
                                   double* scores, double* imag_or_null) {
    if (!c) return HANN_EINVAL;
    if (!s || !ct || !scores || count < 0) return fail(c, HANN_EINVAL, "hann_decrypt_scores: bad argument");
    return decrypt_impl(c, s, ct, count, c->L, ldexpl(1.0L, -log_scale_out), scores, imag_or_null);
}

extern "C" int hann_decrypt_compact(hann_ctx* c, const int8_t* s, const uint64_t* ct, int64_t count, int limbs, int rescaled,
                                    int log_scale_in, double* scores, double* imag_or_null) {
    if (!c) return HANN_EINVAL;
    if (!s || !ct || !scores || count < 0) return fail(c, HANN_EINVAL, "hann_decrypt_compact: bad argument");
    if (limbs < 1 || limbs > c->L - (rescaled ? 1 : 0)) return fail(c, HANN_ESHAPE, "hann_decrypt_compact: limb count out of range");
    long double inv_scale = ldexpl(1.0L, -log_scale_in);
    if (rescaled) inv_scale *= (long double)c->mod[c->L - 1];
    return decrypt_impl(c, s, ct, count, limbs, inv_scale, scores, imag_or_null);
}

// ================================================================================================ server side

extern "C" int hann_load_keys(hann_ctx* c, const uint64_t* evk, int n_rot, const int32_t* rot) {
    if (!c) return HANN_EINVAL;
    if (!evk || !rot || n_rot < 0) return fail(c, HANN_EINVAL, "hann_load_keys: bad argument");
    const int L = c->L, N = c->N;
    for (int i = 0; i < n_rot; i++)
        if (rot[i] < 0 || rot[i] >= c->n) return fail(c, HANN_ESHAPE, "hann_load_keys: rotation out of range");
    DeviceGuard dg(c->device);
    const int64_t keyw = (int64_t)L * 2 * (L + 1) * N;
    RET(ensure_scratch(c, keyw * 8));
    for (int i = 0; i < n_rot; i++) {
        const int r = rot[i];
        if (!c->keytab_host[r]) {
            u64* buf = nullptr;
            if (cudaMalloc(&buf, keyw * 8) != cudaSuccess) {
                cudaGetLastError();
                return fail(c, HANN_ENOMEM, "hann_load_keys: device allocation failed");
            }
            c->keytab_host[r] = buf;
        }
        u64* tmp = (u64*)c->scratch;
        CK(cudaMemcpyAsync(tmp, evk + (int64_t)i * keyw, keyw * 8, cudaMemcpyDefault, c->stream));
        RET(launch_ntt_fwd(c, tmp, (int64_t)L * 2 * (L + 1), N, limbmap_qp(c)));
        // store phi_k^{-1}(key): the inner product then runs on unpermuted digits and the automorphism is applied
        // once, to its much smaller result
        const unsigned k = c->h_galois[r];
        const unsigned kinv = c->h_galois[(c->n - r) % c->n];  // 5^{-r} = 5^{n-r} (5 has order n modulo 2N)
        (void)k;
        RET(launch_permute(c, tmp, c->keytab_host[r], (int64_t)L * 2 * (L + 1), kinv));
        RET(sync_and_check(c));
    }
    CK(cudaMemcpy(c->keytab_dev, c->keytab_host.data(), c->keytab_host.size() * sizeof(u64*), cudaMemcpyHostToDevice));
    return HANN_OK;
}

// out[i] = rot_{rot0 + i}(ct), i < count: one digit decomposition of c1, count keys, one ModDown round
static int rotate_hoisted(hann_ctx* c, const char* who, const u64* ct, int rot0, int count, u64* out, void* ws, size_t ws_bytes) {
    const int L = c->L, N = c->N;
    const int64_t LN = (int64_t)L * N, L1N = (int64_t)(L + 1) * N, ctw = 2 * LN;
    if (count <= 0) return HANN_OK;
    if (rot0 < 1 || rot0 + count > c->n) return fail(c, HANN_ESHAPE, (std::string(who) + ": rotation out of range").c_str());
    for (int r = rot0; r < rot0 + count; r++)
        if (!c->keytab_host[r]) return fail(c, HANN_ENOKEY, (std::string(who) + ": a rotation key is not loaded").c_str());
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, (std::string(who) + ": workspace missing or not 256-byte aligned").c_str());
    Arena ar{(char*)ws, 0, (int64_t)ws_bytes, c};
    u64* c1c = ar.take<u64>(LN);
    u64* digits = ar.take<u64>(L * L1N);
    u64* u = ar.take<u64>((int64_t)count * 2 * L1N);
    u64* lifted = ar.take<u64>((int64_t)count * 2 * LN);
    if (!c1c || !digits || !u || !lifted) return fail(c, HANN_EWORKSPACE, (std::string(who) + ": workspace too small").c_str());
    // one digit set, count keys: item i uses rotation rot0 + i
    RET(ks_digits_to_lifted(c, c1c, 1, digits, 0, rot0, 1, count, u, lifted, ct + LN, 2 * LN));
    RET(launch_moddown_combine(c, u, lifted, count, rot0, 1, ct, 0, nullptr, 0, out, out + LN, ctw));
    return HANN_OK;
}

extern "C" int hann_query_prepare(hann_ctx* c, const void* ct_dev, void* baby_dev, void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (!ct_dev || !baby_dev) return fail(c, HANN_EINVAL, "hann_query_prepare: null pointer");
    const int64_t ctw = 2 * (int64_t)c->L * c->N;
    for (int r = 1; r < c->B; r++)
        if (!c->keytab_host[r]) return fail(c, HANN_ENOKEY, "hann_query_prepare: a baby-step rotation key is not loaded");
    DeviceGuard dg(c->device);
    Timer tm(c, 0);
    const u64* ct = (const u64*)ct_dev;
    u64* baby = (u64*)baby_dev;
    RET(launch_copy2d(c, baby, ctw, ct, ctw, ctw, 1));  // rotation 0
    return rotate_hoisted(c, "hann_query_prepare", ct, 1, c->B - 1, baby + ctw, ws, ws_bytes);
}

extern "C" int hann_rotate_hoisted(hann_ctx* c, const void* ct_dev, int rot0, int count, void* out_dev, void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (!ct_dev || !out_dev || count < 0) return fail(c, HANN_EINVAL, "hann_rotate_hoisted: bad argument");
    DeviceGuard dg(c->device);
    return rotate_hoisted(c, "hann_rotate_hoisted", (const u64*)ct_dev, rot0, count, (u64*)out_dev, ws, ws_bytes);
}

extern "C" int hann_encode_candidates(hann_ctx* c, const float* rows_dev, int64_t n_rows, int dim, void* pt_dev, void* ws,
                                      size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (n_rows < 0 || (n_rows > 0 && (!rows_dev || !pt_dev))) return fail(c, HANN_EINVAL, "hann_encode_candidates: bad argument");
    if (dim < 1 || dim > c->R) return fail(c, HANN_ESHAPE, "hann_encode_candidates: dim must be in 1..R");
    if (n_rows == 0) return HANN_OK;
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_encode_candidates: workspace missing or not 256-byte aligned");
    if ((int64_t)ws_bytes < encode_ws_bytes(c)) return fail(c, HANN_EWORKSPACE, "hann_encode_candidates: workspace too small");
    DeviceGuard dg(c->device);
    Timer tm(c, 1);
    // a stored plaintext is the first N/2 values of each limb's transform (the rest is their mirror image)
    const int64_t n = c->n, nblk = (n_rows + n - 1) / n, Ln = (int64_t)c->L * n, ptw = (int64_t)c->R * Ln;
    const bool fused = encode_fused_available(c);
    for (int64_t blk = 0; blk < nblk; blk++) {
        const int64_t rows_here = std::min(n, n_rows - blk * n);
        const float* rows = rows_dev + blk * n * dim;
        u64* pt = (u64*)pt_dev + blk * ptw;
        // a few plaintexts at a time: FFT buffer and residues of a group are re-read from L2, not from HBM
        for (int p0 = 0; p0 < c->R; p0 += c->encode_group) {
            const int cnt = std::min(c->encode_group, c->R - p0);
            u64* polys = pt + (int64_t)p0 * Ln;
            if (fused && c->encode_sym && ntt_fwd_half_available(c, polys, n)) {
                // half of every transform is computed, straight into place
                RET(launch_encode_rows_fused(c, rows, rows_here, dim, p0, cnt, polys, n, ws, true));
                RET(launch_ntt_fwd_pass_b_half(c, polys, (int64_t)cnt * c->L, n, limbmap_q(c)));
                continue;
            }
            // full transforms of a few plaintexts at a time in the staging area, first halves copied into place
            u64* stage = (u64*)((char*)ws + encode_fft_bytes(c));
            const int sg = encode_stage_group(c);
            for (int s0 = 0; s0 < cnt; s0 += sg) {
                const int sn = std::min(sg, cnt - s0);
                if (fused) {
                    RET(launch_encode_rows_fused(c, rows, rows_here, dim, p0 + s0, sn, stage, c->N, ws, false));
                    RET(launch_ntt_fwd_pass_b(c, stage, (int64_t)sn * c->L, c->N, limbmap_q(c)));
                } else {
                    RET(launch_encode_rows(c, rows, rows_here, dim, p0 + s0, sn, stage, ws));
                    RET(launch_ntt_fwd(c, stage, (int64_t)sn * c->L, c->N, limbmap_q(c)));
                }
                RET(launch_copy2d(c, polys + (int64_t)s0 * Ln, n, stage, c->N, n, (int64_t)sn * c->L));
            }
        }
    }
    return HANN_OK;
}

extern "C" int hann_score_level(hann_ctx* c, const void* baby_dev, const void* pt_dev, int64_t n_blocks, void* inner_dev,
                                void* ws, size_t ws_bytes) {
    (void)ws; (void)ws_bytes;  // the multiply-accumulate needs no scratch
    if (!c) return HANN_EINVAL;
    if (n_blocks < 0 || (n_blocks > 0 && (!baby_dev || !pt_dev || !inner_dev))) return fail(c, HANN_EINVAL, "hann_score_level: bad argument");
    DeviceGuard dg(c->device);
    Timer tm(c, 2);
    return launch_mac(c, (const u64*)baby_dev, (const u64*)pt_dev, n_blocks, (u64*)inner_dev);
}

extern "C" int hann_score_level_batch(hann_ctx* c, const void* baby_dev, int n_queries, const void* pt_dev, int64_t n_blocks,
                                      void* inner_dev, void* ws, size_t ws_bytes) {
    (void)ws; (void)ws_bytes;  // the multiply-accumulate needs no scratch
    if (!c) return HANN_EINVAL;
    if (n_blocks < 0 || n_queries < 0 || (n_blocks > 0 && n_queries > 0 && (!baby_dev || !pt_dev || !inner_dev)))
        return fail(c, HANN_EINVAL, "hann_score_level_batch: bad argument");
    DeviceGuard dg(c->device);
    Timer tm(c, 2);
    return launch_mac_batch(c, (const u64*)baby_dev, n_queries, (const u64*)pt_dev, n_blocks, (u64*)inner_dev);
}

extern "C" int hann_score_level_ctdb(hann_ctx* c, const void* baby_dev, const void* ctdb_dev, int64_t n_blocks, void* inner_dev,
                                     void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (n_blocks < 0 || (n_blocks > 0 && (!baby_dev || !ctdb_dev || !inner_dev))) return fail(c, HANN_EINVAL, "hann_score_level_ctdb: bad argument");
    if (n_blocks == 0) return HANN_OK;
    const int L = c->L, N = c->N, G = c->G;
    for (int l = 0; l < L; l++)
        if (c->mod[l] >= (1ULL << 60)) return fail(c, HANN_ESHAPE, "hann_score_level_ctdb: ciphertext primes must be below 2^60");
    if (c->B > 128) return fail(c, HANN_ESHAPE, "hann_score_level_ctdb: at most 128 baby steps");
    if (!c->keytab_host[0]) return fail(c, HANN_ENOKEY, "hann_score_level_ctdb: the relinearisation key (rotation 0) is not loaded");
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_score_level_ctdb: workspace missing or not 256-byte aligned");
    DeviceGuard dg(c->device);
    Timer tm(c, 2);
    const int64_t LN = (int64_t)L * N, L1N = (int64_t)(L + 1) * N, ctw = 2 * LN;
    // per (blk, g) item: the degree-2 sum (3 polynomials) and one key switch (its own copy of d2, digits, u, lifted)
    const int64_t per = (3 * LN + ks_item_words(c)) * 8;
    int64_t ch = ((int64_t)ws_bytes - kSlack) / per;
    if (ch < 1) return fail(c, HANN_EWORKSPACE, "hann_score_level_ctdb: workspace too small");
    const int64_t items = n_blocks * G;
    ch = std::min<int64_t>(std::min<int64_t>(ch, items), 8 * G);
    Arena ar{(char*)ws, 0, (int64_t)ws_bytes, c};
    u64* d = ar.take<u64>(ch * 3 * LN);
    u64* c1c = ar.take<u64>(ch * LN);
    u64* digits = ar.take<u64>(ch * L * L1N);
    u64* u = ar.take<u64>(ch * 2 * L1N);
    u64* lifted = ar.take<u64>(ch * 2 * LN);
    if (!d || !c1c || !digits || !u || !lifted) return fail(c, HANN_EWORKSPACE, "hann_score_level_ctdb: workspace too small");
    const u64* ctdb = (const u64*)ctdb_dev;
    u64* inner = (u64*)inner_dev;
    for (int64_t i0 = 0; i0 < items; i0 += ch) {
        const int64_t ni = std::min(ch, items - i0);
        RET(launch_mac_ct(c, (const u64*)baby_dev, ctdb + i0 * c->B * ctw, ni, d));
        // relinearise: (d0 + ks0, d1 + ks1) with (ks0, ks1) the key switch of d2 under the key of s^2 ("rotation 0": no
        // automorphism)
        RET(launch_copy2d(c, c1c, LN, d + 2 * LN, 3 * LN, LN, ni));
        RET(ks_digits_to_lifted(c, c1c, ni, digits, (int64_t)L * L1N, 0, 0, ni, u, lifted));
        RET(launch_moddown_combine(c, u, lifted, ni, 0, 0, nullptr, 0, d, 3 * LN, inner + i0 * ctw, inner + i0 * ctw + LN, ctw));
    }
    return HANN_OK;
}

extern "C" int hann_multiply(hann_ctx* c, const void* a_dev, const void* b_dev, int64_t count, void* out_dev, void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (count < 0 || (count > 0 && (!a_dev || !b_dev || !out_dev))) return fail(c, HANN_EINVAL, "hann_multiply: bad argument");
    if (count == 0) return HANN_OK;
    const int L = c->L, N = c->N;
    for (int l = 0; l < L; l++)
        if (c->mod[l] >= (1ULL << 62)) return fail(c, HANN_ESHAPE, "hann_multiply: ciphertext primes must be below 2^62");
    if (!c->keytab_host[0]) return fail(c, HANN_ENOKEY, "hann_multiply: the relinearisation key (rotation 0) is not loaded");
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_multiply: workspace missing or not 256-byte aligned");
    DeviceGuard dg(c->device);
    Timer tm(c, 2);
    const int64_t LN = (int64_t)L * N, L1N = (int64_t)(L + 1) * N, ctw = 2 * LN;
    // per pair: the degree-2 product (3 polynomials) and one key switch (its own copy of d2, digits, u, lifted)
    const int64_t per = (3 * LN + ks_item_words(c)) * 8;
    int64_t ch = ((int64_t)ws_bytes - kSlack) / per;
    if (ch < 1) return fail(c, HANN_EWORKSPACE, "hann_multiply: workspace too small");
    ch = std::min<int64_t>(std::min<int64_t>(ch, count), 32);
    Arena ar{(char*)ws, 0, (int64_t)ws_bytes, c};
    u64* d = ar.take<u64>(ch * 3 * LN);
    u64* c1c = ar.take<u64>(ch * LN);
    u64* digits = ar.take<u64>(ch * L * L1N);
    u64* u = ar.take<u64>(ch * 2 * L1N);
    u64* lifted = ar.take<u64>(ch * 2 * LN);
    if (!d || !c1c || !digits || !u || !lifted) return fail(c, HANN_EWORKSPACE, "hann_multiply: workspace too small");
    const u64 *a = (const u64*)a_dev, *b = (const u64*)b_dev;
    u64* out = (u64*)out_dev;
    for (int64_t i0 = 0; i0 < count; i0 += ch) {
        const int64_t ni = std::min(ch, count - i0);
        RET(launch_mul_ct(c, a + i0 * ctw, b + i0 * ctw, ni, d));
        // relinearise: (d0 + ks0, d1 + ks1), (ks0, ks1) the key switch of d2 under the key of s^2 ("rotation 0")
        RET(launch_copy2d(c, c1c, LN, d + 2 * LN, 3 * LN, LN, ni));
        RET(ks_digits_to_lifted(c, c1c, ni, digits, (int64_t)L * L1N, 0, 0, ni, u, lifted));
        RET(launch_moddown_combine(c, u, lifted, ni, 0, 0, nullptr, 0, d, 3 * LN, out + i0 * ctw, out + i0 * ctw + LN, ctw));
    }
    return HANN_OK;
}

extern "C" int hann_rotate_sum(hann_ctx* c, const void* inner_dev, int64_t n_blocks, void* score_ct_dev, void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (n_blocks < 0 || (n_blocks > 0 && (!inner_dev || !score_ct_dev))) return fail(c, HANN_EINVAL, "hann_rotate_sum: bad argument");
    if (n_blocks == 0) return HANN_OK;
    const int L = c->L, N = c->N, G = c->G, B = c->B;
    const int64_t LN = (int64_t)L * N, L1N = (int64_t)(L + 1) * N, ctw = 2 * LN;
    const u64* inner = (const u64*)inner_dev;
    u64* score = (u64*)score_ct_dev;
    if (c->giant_lazy && G > 1) return hann_rotate_sum_lazy(c, inner_dev, n_blocks, score_ct_dev, ws, ws_bytes);
    DeviceGuard dg(c->device);
    Timer tm(c, 3);
    if (G == 1) {
        RET(launch_copy2d(c, score, ctw, inner, ctw, n_blocks * ctw, 1));
        return HANN_OK;
    }
    if (!c->keytab_host[B]) return fail(c, HANN_ENOKEY, "hann_rotate_sum: the key of rotation B is not loaded");
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_rotate_sum: workspace missing or not 256-byte aligned");
    // Horner over the giant steps for blocks [b_lo, b_hi), as many blocks per round as the given part of the workspace
    // holds, on the context's current stream
    auto run_range = [&](int64_t b_lo, int64_t b_hi, char* wsp, int64_t wsp_bytes) -> int {
        int64_t ch = (wsp_bytes - kSlack) / (ks_item_words(c) * 8);
        if (ch < 1) return fail(c, HANN_EWORKSPACE, "hann_rotate_sum: workspace too small");
        ch = std::min<int64_t>(std::min<int64_t>(ch, b_hi - b_lo), 8);
        Arena ar{wsp, 0, wsp_bytes, c};
        u64* c1c = ar.take<u64>(ch * LN);
        u64* digits = ar.take<u64>(ch * L * L1N);
        u64* u = ar.take<u64>(ch * 2 * L1N);
        u64* lifted = ar.take<u64>(ch * 2 * LN);
        u64* tmp = ar.take<u64>(ch * ctw);
        if (!c1c || !digits || !u || !lifted || !tmp) return fail(c, HANN_EWORKSPACE, "hann_rotate_sum: workspace too small");
        for (int64_t b0 = b_lo; b0 < b_hi; b0 += ch) {
            const int64_t nb = std::min(ch, b_hi - b0);
            const u64* old = inner + (b0 * G + (G - 1)) * ctw;  // acc = inner[G-1]
            int64_t old_stride = (int64_t)G * ctw;
            for (int g = G - 2; g >= 0; g--) {
                u64* out = (g % 2 == 0) ? score + b0 * ctw : tmp;
                // c1 of every accumulator, still in the transform domain; the key-switch round takes it from there
                RET(ks_digits_to_lifted(c, c1c, nb, digits, (int64_t)L * L1N, B, 0, nb, u, lifted, old + LN, old_stride));
                RET(launch_moddown_combine(c, u, lifted, nb, B, 0, old, old_stride, inner + (b0 * G + g) * ctw, (int64_t)G * ctw, out,
                                           out + LN, ctw));
                old = out;
                old_stride = ctw;
            }
        }
        return HANN_OK;
    };
    // Blocks are independent: up to four ranges run side by side on the context's stream and the helper streams, each in
    // its own part of the workspace, which keeps the machine busy through the many small launches of a key switch.
    // (One lane while the per-launch profile is on, so that its kernel times do not overlap.)
    int lanes = (int)std::min<int64_t>(c->max_lanes, n_blocks);
    if (c->stream == c->aux_stream || c->kprof) lanes = 1;
    while (lanes > 1 && (((int64_t)ws_bytes / lanes) & ~(int64_t)255) < ks_item_words(c) * 8 + kSlack) lanes--;
    if (lanes <= 1) {
        const int saved = c->lift_split_ctas;
        if (n_blocks <= 2) c->lift_split_ctas = 320;
        const int r = run_range(0, n_blocks, (char*)ws, (int64_t)ws_bytes);
        c->lift_split_ctas = saved;
        return r;
    }
    const int64_t part = ((int64_t)ws_bytes / lanes) & ~(int64_t)255;
    cudaStream_t main_stream = c->stream;
    cudaStream_t helper[3] = {c->aux_stream, c->lane_stream[0], c->lane_stream[1]};
    cudaEvent_t joined[3] = {c->ev_join, c->lane_join[0], c->lane_join[1]};
    CK(cudaEventRecord(c->ev_fork, main_stream));
    int rc = HANN_OK;
    cudaError_t ce = cudaSuccess;
    for (int ln = 1; ln < lanes; ln++) {
        const int64_t lo = n_blocks * ln / lanes, hi = n_blocks * (ln + 1) / lanes;
        cudaError_t e = cudaStreamWaitEvent(helper[ln - 1], c->ev_fork, 0);
        c->stream = helper[ln - 1];
        const int r = e == cudaSuccess ? run_range(lo, hi, (char*)ws + ln * part, part) : HANN_ECUDA;
        c->stream = main_stream;
        if (e == cudaSuccess) e = cudaEventRecord(joined[ln - 1], helper[ln - 1]);
        if (rc == HANN_OK) rc = r;
        if (ce == cudaSuccess) ce = e;
    }
    const int r0 = run_range(0, n_blocks / lanes, (char*)ws, part);
    if (rc == HANN_OK) rc = r0;
    // join every helper before reporting anything: no helper stream runs past this call unobserved
    for (int ln = 1; ln < lanes; ln++) {
        cudaError_t e = cudaStreamWaitEvent(main_stream, joined[ln - 1], 0);
        if (ce == cudaSuccess) ce = e;
    }
    RET(rc);
    CK(ce);
    return HANN_OK;
}

extern "C" int hann_rotate_sum_lazy(hann_ctx* c, const void* inner_dev, int64_t n_blocks, void* score_ct_dev, void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (n_blocks < 0 || (n_blocks > 0 && (!inner_dev || !score_ct_dev))) return fail(c, HANN_EINVAL, "hann_rotate_sum_lazy: bad argument");
    if (n_blocks == 0) return HANN_OK;
    const int L = c->L, N = c->N, G = c->G, B = c->B;
    const int64_t LN = (int64_t)L * N, L1N = (int64_t)(L + 1) * N, ctw = 2 * LN;
    const u64* inner = (const u64*)inner_dev;
    u64* score = (u64*)score_ct_dev;
    DeviceGuard dg(c->device);
    Timer tm(c, 3);
    if (G == 1) return launch_copy2d(c, score, ctw, inner, ctw, n_blocks * ctw, 1);
    for (int g = 1; g < G; g++)
        if (!c->keytab_host[g * B]) return fail(c, HANN_ENOKEY, "hann_rotate_sum_lazy: the keys of rotations B, 2B, .., (G-1)B must be loaded");
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_rotate_sum_lazy: workspace missing or not 256-byte aligned");
    const bool lift = ks_lift_available(c);
    // blocks [b_lo, b_hi), as many per round as the given part of the workspace holds, on the context's current stream
    auto run_range = [&](int64_t b_lo, int64_t b_hi, char* wsp, int64_t wsp_bytes) -> int {
        int64_t ch = (wsp_bytes - kSlack) / (lazy_block_words(c) * 8);
        if (ch < 1) return fail(c, HANN_EWORKSPACE, "hann_rotate_sum_lazy: workspace too small");
        ch = std::min<int64_t>(std::min<int64_t>(ch, b_hi - b_lo), 16);
        Arena ar{wsp, 0, wsp_bytes, c};
        const int64_t items_max = ch * (G - 1);
        u64* c1c = ar.take<u64>(items_max * LN);
        u64* digits = ar.take<u64>(items_max * L * L1N);
        u64* u = ar.take<u64>(items_max * 2 * L1N);
        u64* up = ar.take<u64>(ch * 2 * N);
        u64* lifted = ar.take<u64>(ch * 2 * LN);
        if (!c1c || !digits || !u || !up || !lifted) return fail(c, HANN_EWORKSPACE, "hann_rotate_sum_lazy: workspace too small");
        for (int64_t b0 = b_lo; b0 < b_hi; b0 += ch) {
            const int64_t nb = std::min(ch, b_hi - b0), items = nb * (G - 1);
            // c1 of term (g, blk), still in the transform domain, into c1c[(g - 1) * nb + blk]
            bool all_fused = lift;
            for (int g = 1; g < G; g++) {
                const u64* src = inner + (b0 * G + g) * ctw + LN;
                u64* dst = c1c + (int64_t)(g - 1) * nb * LN;
                const bool fused = lift && ntt_inv_pass_b_gathers(c, src, dst);
                all_fused = all_fused && fused;
                if (fused) RET(launch_ntt_inv_pass_b_from(c, src, (int64_t)G * ctw, dst, nb * L, N, limbmap_q(c)));
                else RET(launch_copy2d(c, dst, LN, src, (int64_t)G * ctw, LN, nb));
            }
            if (lift) {
                if (!all_fused) {
                    // the terms whose inverse pass ran while gathering are finished; the copied ones still need it
                    for (int g = 1; g < G; g++) {
                        const u64* src = inner + (b0 * G + g) * ctw + LN;
                        u64* dst = c1c + (int64_t)(g - 1) * nb * LN;
                        if (!ntt_inv_pass_b_gathers(c, src, dst)) RET(launch_ntt_inv_pass_b(c, dst, nb * L, N, limbmap_q(c)));
                    }
                }
                RET(launch_ks_lift(c, c1c, N, items * L, limbmap_q(c), digits, L + 1, 0));
                RET(launch_ntt_fwd_pass_b(c, digits, items * L * (L + 1), N, limbmap_qp(c)));
            } else {
                RET(launch_ntt_inv(c, c1c, items * L, N, limbmap_q(c)));
                RET(launch_lift_digits(c, c1c, LN, items, digits));
                RET(launch_ntt_fwd(c, digits, items * L * (L + 1), N, limbmap_qp(c)));
            }
            // every giant step under its own key, all in one launch; then the special-prime limb of the SUM of the (permuted)
            // products, its inverse transform, centred lift and forward transforms: one ModDown per block
            RET(launch_ks_inner_batches(c, digits, (int64_t)L * L1N, B, B, G - 1, nb, u));
            RET(launch_giant_sum_p(c, u, nb, up));
            if (lift) {
                RET(launch_ntt_inv_pass_b(c, up, nb * 2, N, limbmap_single(L)));
                RET(launch_ks_lift(c, up, N, nb * 2, limbmap_single(L), lifted, L, 0));
                RET(launch_ntt_fwd_pass_b(c, lifted, nb * 2 * L, N, limbmap_q(c)));
            } else {
                RET(launch_ntt_inv(c, up, nb * 2, N, limbmap_single(L)));
                RET(launch_lift_p(c, up, nb * 2, lifted));
                RET(launch_ntt_fwd(c, lifted, nb * 2 * L, N, limbmap_q(c)));
            }
            RET(launch_giant_combine(c, u, lifted, inner + b0 * G * ctw, nb, score + b0 * ctw));
        }
        return HANN_OK;
    };
    // Block ranges are independent: up to `lazy_lanes` of them run side by side on the context's stream and its helper
    // streams, each in its own part of the workspace, so that the short launches of one range (the ModDown of a few
    // polynomials is a latency chain on a fraction of the machine) overlap the long ones of another.  One lane while the
    // per-launch profile is on (its kernel times must not overlap) and when the caller already is on a helper stream.
    int lanes = (int)std::min<int64_t>(c->lazy_lanes, n_blocks);
    if (c->stream == c->aux_stream || c->kprof || c->max_lanes <= 1) lanes = 1;
    while (lanes > 1 && (((int64_t)ws_bytes / lanes) & ~(int64_t)255) < lazy_block_words(c) * 8 + kSlack) lanes--;
    if (lanes <= 1) return run_range(0, n_blocks, (char*)ws, (int64_t)ws_bytes);
    const int64_t part = ((int64_t)ws_bytes / lanes) & ~(int64_t)255;
    cudaStream_t main_stream = c->stream;
    cudaStream_t helper[3] = {c->aux_stream, c->lane_stream[0], c->lane_stream[1]};
    cudaEvent_t joined[3] = {c->ev_join, c->lane_join[0], c->lane_join[1]};
    CK(cudaEventRecord(c->ev_fork, main_stream));
    int rc = HANN_OK;
    cudaError_t ce = cudaSuccess;
    for (int ln = 1; ln < lanes; ln++) {
        const int64_t lo = n_blocks * ln / lanes, hi = n_blocks * (ln + 1) / lanes;
        cudaError_t e = cudaStreamWaitEvent(helper[ln - 1], c->ev_fork, 0);
        c->stream = helper[ln - 1];
        const int r = e == cudaSuccess ? run_range(lo, hi, (char*)ws + ln * part, part) : HANN_ECUDA;
        c->stream = main_stream;
        if (e == cudaSuccess) e = cudaEventRecord(joined[ln - 1], helper[ln - 1]);
        if (rc == HANN_OK) rc = r;
        if (ce == cudaSuccess) ce = e;
    }
    const int r0 = run_range(0, n_blocks / lanes, (char*)ws, part);
    if (rc == HANN_OK) rc = r0;
    // join every helper before reporting anything: no helper stream runs past this call unobserved
    for (int ln = 1; ln < lanes; ln++) {
        cudaError_t e = cudaStreamWaitEvent(main_stream, joined[ln - 1], 0);
        if (ce == cudaSuccess) ce = e;
    }
    RET(rc);
    CK(ce);
    return HANN_OK;
}

// ================================================================================================ packed projection

// count real slot vectors z [count][n] (device doubles) -> stored plaintexts [count][L][N/2] at scale 2^log_scale: canonical
// encode, full transform in the staging area, first half kept
static int encode_slot_vectors(hann_ctx* c, const double* z, int64_t count, int log_scale, u64* pt, void* ws, size_t ws_bytes) {
    if ((int64_t)ws_bytes < encode_ws_bytes(c)) return fail(c, HANN_EWORKSPACE, "slot-vector encoding: workspace too small");
    u64* stage = (u64*)((char*)ws + encode_fft_bytes(c));
    const int64_t n = c->n, Ln = (int64_t)c->L * n;
    for (int64_t i = 0; i < count; i++) {
        RET(launch_encode_slots(c, z + i * n, stage, ws, log_scale));
        RET(launch_ntt_fwd(c, stage, c->L, c->N, limbmap_q(c)));
        RET(launch_copy2d(c, pt + i * Ln, n, stage, c->N, n, c->L));
    }
    return HANN_OK;
}

extern "C" int hann_encode_slots(hann_ctx* c, const double* z_dev, int64_t count, int log_scale, void* pt_dev, void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (count < 0 || (count > 0 && (!z_dev || !pt_dev))) return fail(c, HANN_EINVAL, "hann_encode_slots: bad argument");
    if (log_scale < 1 || log_scale > 60) return fail(c, HANN_EINVAL, "hann_encode_slots: scale must be 2^1 .. 2^60");
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_encode_slots: workspace missing or not 256-byte aligned");
    DeviceGuard dg(c->device);
    return encode_slot_vectors(c, z_dev, count, log_scale, (u64*)pt_dev, ws, ws_bytes);
}

extern "C" int hann_project_enrol(hann_ctx* c, const float* W_dev, int D, int log_scale_w, void* pt_dev, void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (!W_dev || !pt_dev) return fail(c, HANN_EINVAL, "hann_project_enrol: null pointer");
    if (D < c->R || D % c->R || c->n % D) return fail(c, HANN_ESHAPE, "hann_project_enrol: D must be a multiple of R that divides n");
    if (log_scale_w < 1 || log_scale_w > 60) return fail(c, HANN_EINVAL, "hann_project_enrol: scale must be 2^1 .. 2^60");
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_project_enrol: workspace missing or not 256-byte aligned");
    const int64_t zb = align256((int64_t)c->n * 8);
    if ((int64_t)ws_bytes < zb + encode_ws_bytes(c)) return fail(c, HANN_EWORKSPACE, "hann_project_enrol: workspace too small");
    DeviceGuard dg(c->device);
    double* z = (double*)ws;
    const int64_t Ln = (int64_t)c->L * c->n;
    for (int g = 0; g < c->G; g++)
        for (int b = 0; b < c->B; b++) {
            RET(launch_packed_diagonal(c, W_dev, D, g, b, z));
            RET(encode_slot_vectors(c, z, 1, log_scale_w, (u64*)pt_dev + ((int64_t)g * c->B + b) * Ln, (char*)ws + zb, ws_bytes - (size_t)zb));
        }
    return HANN_OK;
}

extern "C" int hann_project_masks(hann_ctx* c, int log_scale_m, void* lo_dev, void* hi_dev, void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (!lo_dev || !hi_dev) return fail(c, HANN_EINVAL, "hann_project_masks: null pointer");
    if (log_scale_m < 1 || log_scale_m > 60) return fail(c, HANN_EINVAL, "hann_project_masks: scale must be 2^1 .. 2^60");
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_project_masks: workspace missing or not 256-byte aligned");
    const int64_t zb = align256((int64_t)c->n * 8);
    if ((int64_t)ws_bytes < 2 * zb + encode_ws_bytes(c)) return fail(c, HANN_EWORKSPACE, "hann_project_masks: workspace too small");
    DeviceGuard dg(c->device);
    double *lo = (double*)ws, *hi = (double*)((char*)ws + zb);
    const int64_t Ln = (int64_t)c->L * c->n;
    for (int b = 0; b < c->B; b++) {
        RET(launch_window_masks(c, b, lo, hi));
        RET(encode_slot_vectors(c, lo, 1, log_scale_m, (u64*)lo_dev + b * Ln, (char*)ws + 2 * zb, ws_bytes - (size_t)(2 * zb)));
        RET(encode_slot_vectors(c, hi, 1, log_scale_m, (u64*)hi_dev + b * Ln, (char*)ws + 2 * zb, ws_bytes - (size_t)(2 * zb)));
    }
    return HANN_OK;
}

// words of workspace hann_project_baby needs: the two batches of rotated ciphertexts and one hoisted rotation round
static int64_t project_baby_words(const hann_ctx* c) {
    const int64_t L = c->L, N = c->N, nb = std::max(c->B - 1, 1);
    return 2 * nb * 2 * L * N + prepare_words(c);
}

extern "C" int hann_project_baby(hann_ctx* c, const void* ct_dev, const void* lo_dev, const void* hi_dev, void* cyc_dev, void* ws,
                                 size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (!ct_dev || !lo_dev || !hi_dev || !cyc_dev) return fail(c, HANN_EINVAL, "hann_project_baby: null pointer");
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_project_baby: workspace missing or not 256-byte aligned");
    const int B = c->B;
    const int64_t ctw = 2 * (int64_t)c->L * c->N;
    DeviceGuard dg(c->device);
    Timer tm(c, 0);
    Arena ar{(char*)ws, 0, (int64_t)ws_bytes, c};
    u64* rot_a = ar.take<u64>(std::max(B - 1, 1) * ctw);
    u64* rot_h = ar.take<u64>(std::max(B - 1, 1) * ctw);
    if (!rot_a || !rot_h) return fail(c, HANN_EWORKSPACE, "hann_project_baby: workspace too small");
    char* sub = (char*)ws + ar.off;
    const size_t sub_bytes = ws_bytes - (size_t)ar.off;
    // rot_b(ct) and rot_{b-R}(ct) (the latter as the slot rotation by n - R + b), b = 1 .. B-1, each batch hoisted
    RET(rotate_hoisted(c, "hann_project_baby", (const u64*)ct_dev, 1, B - 1, rot_a, sub, sub_bytes));
    RET(rotate_hoisted(c, "hann_project_baby", (const u64*)ct_dev, c->n - c->R + 1, B - 1, rot_h, sub, sub_bytes));
    return launch_mask_combine(c, (const u64*)ct_dev, rot_a, rot_h, (const u64*)lo_dev, (const u64*)hi_dev, (u64*)cyc_dev);
}

extern "C" int hann_rescale(hann_ctx* c, const void* ct_dev, int64_t count, void* out_dev, void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (c->L < 2) return fail(c, HANN_ESHAPE, "hann_rescale: the chain has a single prime left");
    return hann_compact_scores(c, ct_dev, count, c->L - 1, 1, out_dev, ws, ws_bytes);
}

extern "C" int hann_fold(hann_ctx* c, void* ct_dev, int stride, int steps, void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (!ct_dev || stride < 1 || steps < 0) return fail(c, HANN_EINVAL, "hann_fold: bad argument");
    if (steps == 0) return HANN_OK;
    if (((int64_t)stride << (steps - 1)) >= c->n) return fail(c, HANN_ESHAPE, "hann_fold: rotation out of range");
    for (int t = 0; t < steps; t++)
        if (!c->keytab_host[stride << t]) return fail(c, HANN_ENOKEY, "hann_fold: the keys of rotations stride * 2^t must be loaded");
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_fold: workspace missing or not 256-byte aligned");
    const int L = c->L, N = c->N;
    const int64_t LN = (int64_t)L * N, L1N = (int64_t)(L + 1) * N, ctw = 2 * LN;
    DeviceGuard dg(c->device);
    Timer tm(c, 3);
    Arena ar{(char*)ws, 0, (int64_t)ws_bytes, c};
    KsBuffers kb;
    u64* tmp = ar.take<u64>(ctw);
    if (!tmp || !carve_keyswitch(c, ar, kb)) return fail(c, HANN_EWORKSPACE, "hann_fold: workspace too small");
    u64* cur = (u64*)ct_dev;
    u64* nxt = tmp;
    for (int t = 0; t < steps; t++) {
        const int r = stride << t;
        // nxt = cur + rot_r(cur): the Horner step of the rotate-and-sum with the ciphertext itself as the addend
        RET(ks_digits_to_lifted(c, kb.c1c, 1, kb.digits, (int64_t)L * L1N, r, 0, 1, kb.u, kb.lifted, cur + LN, ctw));
        RET(launch_moddown_combine(c, kb.u, kb.lifted, 1, r, 0, cur, ctw, cur, ctw, nxt, nxt + LN, ctw));
        std::swap(cur, nxt);
    }
    if (cur != (u64*)ct_dev) RET(launch_copy2d(c, (u64*)ct_dev, ctw, cur, ctw, ctw, 1));
    return HANN_OK;
}

extern "C" int64_t hann_project_bytes(const hann_ctx* top, const hann_ctx* mid) {
    if (!top || !mid) return HANN_EINVAL;
    const int64_t B = top->B, G = mid->G;
    const int64_t cyc_top = align256(B * hann_sizeof(top, HANN_SIZE_CT)), cyc_mid = align256(B * hann_sizeof(mid, HANN_SIZE_CT));
    const int64_t inner = align256(G * hann_sizeof(mid, HANN_SIZE_CT)), acc = align256(hann_sizeof(mid, HANN_SIZE_CT));
    const int64_t sub = std::max<int64_t>(std::max<int64_t>(project_baby_words(top) * 8 + kSlack, hann_workspace_bytes(top, B)),
                                          hann_workspace_bytes(mid, 1));
    return cyc_top + cyc_mid + inner + acc + align256(sub) + kSlack;
}

extern "C" int hann_project_query(hann_ctx* top, hann_ctx* mid, const void* ct_dev, const void* lo_dev, const void* hi_dev,
                                  const void* wpt_dev, int D, void* out_dev, void* ws, size_t ws_bytes) {
    if (!top || !mid) return HANN_EINVAL;
    hann_ctx* c = top;
    if (!ct_dev || !lo_dev || !hi_dev || !wpt_dev || !out_dev) return fail(c, HANN_EINVAL, "hann_project_query: null pointer");
    if (mid->L != top->L - 1 || mid->L < 2 || mid->N != top->N || mid->R != top->R || mid->B != top->B || mid->device != top->device ||
        mid->stream != top->stream)
        return fail(c, HANN_ESHAPE, "hann_project_query: the second context must be the same ring, R, B, device and stream with one prime less");
    for (int i = 0; i < mid->L; i++)
        if (mid->mod[i] != top->mod[i]) return fail(c, HANN_ESHAPE, "hann_project_query: the second context's primes must be the first L-1 of the first's");
    if (mid->mod[mid->L] != top->mod[top->L]) return fail(c, HANN_ESHAPE, "hann_project_query: the contexts must share the special prime");
    const int R = top->R;
    if (D < R || D % R || top->n % D || ((D / R) & (D / R - 1))) return fail(c, HANN_ESHAPE, "hann_project_query: D / R must be a power of two, D must divide n");
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_project_query: workspace missing or not 256-byte aligned");
    if ((int64_t)ws_bytes < hann_project_bytes(top, mid)) return fail(c, HANN_EWORKSPACE, "hann_project_query: workspace too small");
    const int64_t B = top->B, G = mid->G;
    Arena ar{(char*)ws, 0, (int64_t)ws_bytes, c};
    u64* cyc_top = ar.take<u64>(B * hann_sizeof(top, HANN_SIZE_CT) / 8);
    u64* cyc_mid = ar.take<u64>(B * hann_sizeof(mid, HANN_SIZE_CT) / 8);
    u64* inner = ar.take<u64>(G * hann_sizeof(mid, HANN_SIZE_CT) / 8);
    u64* acc = ar.take<u64>(hann_sizeof(mid, HANN_SIZE_CT) / 8);
    if (!cyc_top || !cyc_mid || !inner || !acc) return fail(c, HANN_EWORKSPACE, "hann_project_query: workspace too small");
    char* sub = (char*)ws + ar.off;
    const size_t sub_bytes = ws_bytes - (size_t)ar.off;
    auto relay = [&](int rc) {  // failures of the second context are reported through the first
        if (rc != HANN_OK && top->err.empty()) top->err = mid->err;
        return rc;
    };
    top->err.clear();
    // baby steps inside the windows (scale Delta * mask scale), first rescale: the baby set of the middle chain
    RET(hann_project_baby(top, ct_dev, lo_dev, hi_dev, cyc_top, sub, sub_bytes));
    RET(hann_rescale(top, cyc_top, B, cyc_mid, sub, sub_bytes));
    // packed matrix x in-window rotations, giant steps, the single fold over the windows, second rescale
    RET(relay(hann_score_level(mid, cyc_mid, wpt_dev, 1, inner, sub, sub_bytes)));
    RET(relay(hann_rotate_sum(mid, inner, 1, acc, sub, sub_bytes)));
    int steps = 0;
    while ((R << steps) < D) steps++;
    RET(relay(hann_fold(mid, acc, R, steps, sub, sub_bytes)));
    RET(relay(hann_rescale(mid, acc, 1, out_dev, sub, sub_bytes)));
    return HANN_OK;
}

extern "C" int hann_keyswitch(hann_ctx* c, int rot, const void* poly_dev, void* ks0_dev, void* ks1_dev, void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (!poly_dev || !ks0_dev || !ks1_dev) return fail(c, HANN_EINVAL, "hann_keyswitch: null pointer");
    if (rot < 1 || rot >= c->n) return fail(c, HANN_ESHAPE, "hann_keyswitch: rotation out of range");
    if (!c->keytab_host[rot]) return fail(c, HANN_ENOKEY, "hann_keyswitch: key not loaded");
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_keyswitch: workspace missing or not 256-byte aligned");
    const int L = c->L;
    DeviceGuard dg(c->device);
    Timer tm(c, 4);
    Arena ar{(char*)ws, 0, (int64_t)ws_bytes, c};
    KsBuffers kb;
    if (!carve_keyswitch(c, ar, kb)) return fail(c, HANN_EWORKSPACE, "hann_keyswitch: workspace too small");
    u64 *c1c = kb.c1c, *digits = kb.digits, *u = kb.u, *lifted = kb.lifted;
    // the stored key is phi_k^{-1}(evk): switch phi_k^{-1}(d) and apply phi_k to the result
    const unsigned kinv = c->h_galois[(c->n - rot) % c->n];
    RET(launch_permute(c, (const u64*)poly_dev, c1c, L, kinv));
    RET(ks_digits_to_lifted(c, c1c, 1, digits, 0, rot, 0, 1, u, lifted));
    RET(launch_moddown_combine(c, u, lifted, 1, rot, 0, nullptr, 0, nullptr, 0, (u64*)ks0_dev, (u64*)ks1_dev, 0));
    return HANN_OK;
}

extern "C" int hann_query_level(hann_ctx* c, const void* ct_dev, const float* rows_dev, int64_t n_rows, int dim, void* baby_dev,
                                void* pt_dev, void* inner_dev, void* score_ct_dev, void* ws, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (!ct_dev || !rows_dev || !baby_dev || !pt_dev || !inner_dev || !score_ct_dev || n_rows < 1)
        return fail(c, HANN_EINVAL, "hann_query_level: bad argument");
    if (!ws || ((uintptr_t)ws & 255)) return fail(c, HANN_EWORKSPACE, "hann_query_level: workspace missing or not 256-byte aligned");
    if (dim < 1 || dim > c->R) return fail(c, HANN_ESHAPE, "hann_query_level: dim must be in 1..R");
    const int64_t prep = c->B > 1 ? align256(prepare_words(c) * 8 + kSlack) : 0;
    if ((int64_t)ws_bytes < prep + encode_ws_bytes(c)) return fail(c, HANN_EWORKSPACE, "hann_query_level: workspace too small");
    DeviceGuard dg(c->device);
    const int64_t nblk = (n_rows + c->n - 1) / c->n;
    // fork: the baby rotations of the query on the helper stream, the candidate encoding on the context's stream
    cudaStream_t main_stream = c->stream;
    // (measured on the face level: two groups gain 1.5 %, three and more lose, the device being limited by its FP64 pipe
    // and its power cap in every stage: the groups are used only when asked for)
    int ng = 1;
    int64_t ws_score = 0;
    if (c->host_groups > 1) level_groups(c, nblk, &ng, &ws_score);
    const int64_t enc_bytes = align256(encode_ws_bytes(c));
    // the groups need a workspace layout of their own; a smaller workspace, the per-launch profile (whose kernel times must
    // not overlap) or a context that already runs on a helper stream take the plain order
    if (ng > 1 && ((int64_t)ws_bytes < prep + enc_bytes + 2 * ws_score || c->kprof || main_stream == c->aux_stream)) ng = 1;
    CK(cudaEventRecord(c->ev_fork, main_stream));
    CK(cudaStreamWaitEvent(c->aux_stream, c->ev_fork, 0));
    c->stream = c->aux_stream;
    int rc = hann_query_prepare(c, ct_dev, baby_dev, ws, (size_t)prep);
    c->stream = main_stream;
    if (ng == 1) {
        cudaError_t e = cudaEventRecord(c->ev_join, c->aux_stream);
        if (rc == HANN_OK) rc = hann_encode_candidates(c, rows_dev, n_rows, dim, pt_dev, (char*)ws + prep, ws_bytes - (size_t)prep);
        // join before anything else is reported, so that the helper stream never runs past this call's buffers unobserved
        cudaError_t e2 = cudaStreamWaitEvent(main_stream, c->ev_join, 0);
        RET(rc);
        CK(e);
        CK(e2);
        RET(hann_score_level(c, baby_dev, pt_dev, nblk, inner_dev, ws, ws_bytes));
        RET(hann_rotate_sum(c, inner_dev, nblk, score_ct_dev, ws, ws_bytes));
        return HANN_OK;
    }
    // Groups of blocks: the context's stream encodes group after group; a group is scored (multiply-accumulate,
    // rotate-and-sum) on one of two scoring streams as soon as it is encoded, beside the encoding of the next groups: the
    // latency chains of a group's key switches fill the gaps of the encoding kernels.  Only the last group's scoring follows
    // the last encoding.  Same operations on the same data as the plain order, hence the same bits.
    cudaError_t ce = cudaEventRecord(c->prep_done, c->aux_stream);
    for (int i = 0; i < 2 && ce == cudaSuccess; i++) ce = cudaStreamWaitEvent(c->score_stream[i], c->ev_fork, 0);
    while ((int)c->enc_ev.size() < ng && ce == cudaSuccess) {
        cudaEvent_t e;
        ce = cudaEventCreateWithFlags(&e, cudaEventDisableTiming);
        if (ce == cudaSuccess) c->enc_ev.push_back(e);
    }
    const int64_t ptw = hann_sizeof(c, HANN_SIZE_PT_BLOCK) / 8, ctw = hann_sizeof(c, HANN_SIZE_CT) / 8;
    const int64_t innerw = hann_sizeof(c, HANN_SIZE_INNER) / 8;
    char* ws_enc = (char*)ws + prep;
    char* wss[2] = {ws_enc + enc_bytes, ws_enc + enc_bytes + ws_score};
    const int saved_lanes = c->max_lanes;
    for (int gi = 0; gi < ng && rc == HANN_OK && ce == cudaSuccess; gi++) {
        const int64_t b0 = nblk - nblk * (ng - gi) / ng, b1 = nblk - nblk * (ng - gi - 1) / ng, nb = b1 - b0;
        const int64_t r0 = b0 * c->n, rn = std::min<int64_t>(nb * c->n, n_rows - r0);
        rc = hann_encode_candidates(c, rows_dev + r0 * dim, rn, dim, (u64*)pt_dev + b0 * ptw, ws_enc, (size_t)enc_bytes);
        if (rc != HANN_OK) break;
        cudaStream_t ss = c->score_stream[gi & 1];
        ce = cudaEventRecord(c->enc_ev[gi], main_stream);
        if (ce == cudaSuccess) ce = cudaStreamWaitEvent(ss, c->enc_ev[gi], 0);
        if (ce == cudaSuccess && gi < 2) ce = cudaStreamWaitEvent(ss, c->prep_done, 0);  // the baby rotations are ready
        if (ce != cudaSuccess) break;
        c->stream = ss;
        c->max_lanes = 1;  // the groups run side by side instead of the lanes
        rc = hann_score_level(c, baby_dev, (const u64*)pt_dev + b0 * ptw, nb, (u64*)inner_dev + b0 * innerw, wss[gi & 1], (size_t)ws_score);
        if (rc == HANN_OK)
            rc = hann_rotate_sum(c, (const u64*)inner_dev + b0 * innerw, nb, (u64*)score_ct_dev + b0 * ctw, wss[gi & 1], (size_t)ws_score);
        c->stream = main_stream;
        c->max_lanes = saved_lanes;
    }
    // join every helper stream before reporting anything
    cudaError_t ej[3];
    ej[0] = cudaStreamWaitEvent(main_stream, c->prep_done, 0);
    for (int i = 0; i < 2; i++) {
        ej[1 + i] = cudaEventRecord(c->score_join[i], c->score_stream[i]);
        if (ej[1 + i] == cudaSuccess) ej[1 + i] = cudaStreamWaitEvent(main_stream, c->score_join[i], 0);
    }
    RET(rc);
    CK(ce);
    for (int i = 0; i < 3; i++) CK(ej[i]);
    return HANN_OK;
}

// ================================================================================================ host-buffer level

namespace {
struct LevelPlan {
    int64_t nblk, ct, baby, rows, pt, inner, score, stage, ws, ws_score, total;
    int ng;  // block groups; group gi covers blocks [nblk - nblk (ng - gi) / ng, nblk - nblk (ng - gi - 1) / ng)
};
LevelPlan plan_level(const hann_ctx* c, int64_t n_rows, int dim) {
    LevelPlan p;
    const int64_t ctb = hann_sizeof(c, HANN_SIZE_CT);
    p.nblk = (n_rows + c->n - 1) / c->n;
    p.ct = align256(ctb);
    p.baby = align256(hann_sizeof(c, HANN_SIZE_BABY));
    p.rows = align256(n_rows * (int64_t)dim * 4);
    p.pt = align256(p.nblk * hann_sizeof(c, HANN_SIZE_PT_BLOCK));
    p.inner = align256(p.nblk * hann_sizeof(c, HANN_SIZE_INNER));
    p.score = align256(p.nblk * ctb);
    p.stage = align256(p.nblk * ctb);
    p.ws = align256(hann_workspace_bytes(c, p.nblk));
    // with more than one group: a rotate-and-sum workspace for each of the two scoring streams
    level_groups(c, p.nblk, &p.ng, &p.ws_score);
    p.total = p.ct + p.baby + p.rows + p.pt + p.inner + p.score + p.stage + p.ws + 2 * p.ws_score;
    return p;
}
}  // namespace

extern "C" int64_t hann_level_host_bytes(const hann_ctx* c, int64_t n_rows) {
    if (!c || n_rows < 0) return HANN_EINVAL;
    return plan_level(c, n_rows, c->R).total;
}

extern "C" int hann_score_level_host(hann_ctx* c, const uint64_t* ct_host, const float* rows_host, int64_t n_rows, int dim,
                                     uint64_t* score_ct_host, void* ws_dev, size_t ws_bytes) {
    if (!c) return HANN_EINVAL;
    if (!ct_host || !rows_host || !score_ct_host || n_rows < 1) return fail(c, HANN_EINVAL, "hann_score_level_host: bad argument");
    if (dim < 1 || dim > c->R) return fail(c, HANN_ESHAPE, "hann_score_level_host: dim must be in 1..R");
    if (!ws_dev || ((uintptr_t)ws_dev & 255)) return fail(c, HANN_EWORKSPACE, "hann_score_level_host: workspace missing or not 256-byte aligned");
    const LevelPlan p = plan_level(c, n_rows, dim);
    if ((int64_t)ws_bytes < p.total) return fail(c, HANN_EWORKSPACE, "hann_score_level_host: workspace too small");
    DeviceGuard dg(c->device);
    char* b = (char*)ws_dev;
    u64* ct = (u64*)b; b += p.ct;
    u64* baby = (u64*)b; b += p.baby;
    float* rows = (float*)b; b += p.rows;
    u64* pt = (u64*)b; b += p.pt;
    u64* inner = (u64*)b; b += p.inner;
    u64* score = (u64*)b; b += p.score;
    u64* stage = (u64*)b; b += p.stage;
    void* ws = b; b += p.ws;
    char* ws_score[2] = {b, b + p.ws_score};
    // The query goes up first, then the rows block by block on the upload stream; the helper stream prepares the baby
    // rotations; the context's stream encodes each block as soon as its rows have arrived.  The level is cut into groups
    // of blocks: a group is scored (multiply-accumulate, rotate-and-sum, inverse transform of its score ciphertexts) on
    // one of two scoring streams while the following groups are still uploaded and encoded, and its scores go home on
    // the download stream beside all that.  Only the last group's scoring and download follow the last upload.  (One
    // group: everything on the context's stream, the rotate-and-sum on its four lanes.)
    const int ng = p.ng;
    while ((int64_t)c->blk_ev.size() < p.nblk) {
        cudaEvent_t e;
        CK(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        c->blk_ev.push_back(e);
    }
    while ((int)c->grp_ev.size() < ng || (int)c->enc_ev.size() < ng) {
        cudaEvent_t e, e2;
        CK(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        c->grp_ev.push_back(e);
        CK(cudaEventCreateWithFlags(&e2, cudaEventDisableTiming));
        c->enc_ev.push_back(e2);
    }
    const int64_t prep = c->B > 1 ? align256(prepare_words(c) * 8 + kSlack) : 0;
    cudaStream_t main_stream = c->stream;
    CK(cudaEventRecord(c->ev_fork, main_stream));
    for (cudaStream_t st : {c->up_stream, c->down_stream, c->aux_stream, c->score_stream[0], c->score_stream[1]})
        CK(cudaStreamWaitEvent(st, c->ev_fork, 0));
    // host-to-device copies are served in the order they were queued, whatever their stream: the query must not wait
    // behind the rows
    c->stream = c->aux_stream;
    int rc = import_polys(c, ct_host, 2, ct);
    c->stream = main_stream;
    for (int64_t blk = 0; blk < p.nblk; blk++) {
        const int64_t r0 = blk * c->n, rn = std::min<int64_t>(c->n, n_rows - r0);
        CK(cudaMemcpyAsync(rows + r0 * dim, rows_host + r0 * dim, (size_t)rn * dim * 4, cudaMemcpyHostToDevice, c->up_stream));
        CK(cudaEventRecord(c->blk_ev[blk], c->up_stream));
    }
    c->stream = c->aux_stream;
    if (rc == HANN_OK) rc = hann_query_prepare(c, ct, baby, ws, (size_t)prep);
    c->stream = main_stream;
    cudaError_t ce = cudaEventRecord(c->prep_done, c->aux_stream);
    const int64_t ptw = hann_sizeof(c, HANN_SIZE_PT_BLOCK) / 8, ctw = hann_sizeof(c, HANN_SIZE_CT) / 8;
    const int64_t innerw = hann_sizeof(c, HANN_SIZE_INNER) / 8;
    const int keep = c->host_limbs >= c->L ? c->L : c->host_limbs;  // limbs of every score polynomial that go home
    const int64_t kw = (int64_t)keep * c->N;
    const int saved_lanes = c->max_lanes;
    for (int gi = 0; gi < ng && rc == HANN_OK; gi++) {
        const int64_t b0 = p.nblk - p.nblk * (ng - gi) / ng, b1 = p.nblk - p.nblk * (ng - gi - 1) / ng, nb = b1 - b0;
        for (int64_t blk = b0; blk < b1 && rc == HANN_OK; blk++) {
            const int64_t r0 = blk * c->n, rn = std::min<int64_t>(c->n, n_rows - r0);
            if (cudaStreamWaitEvent(main_stream, c->blk_ev[blk], 0) != cudaSuccess) rc = fail(c, HANN_ECUDA, "cudaStreamWaitEvent failed");
            if (rc == HANN_OK)
                rc = hann_encode_candidates(c, rows + r0 * dim, rn, dim, pt + blk * ptw, (char*)ws + prep, (size_t)(p.ws - prep));
        }
        if (rc != HANN_OK) break;
        // the scoring stream of this group: the context's own when there is one group
        cudaStream_t ss = ng > 1 ? c->score_stream[gi & 1] : main_stream;
        cudaError_t e = cudaSuccess;
        if (ng > 1) {
            e = cudaEventRecord(c->enc_ev[gi], main_stream);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(ss, c->enc_ev[gi], 0);
            c->max_lanes = 1;  // the groups run side by side instead of the lanes
        }
        if (e == cudaSuccess && gi < 2) e = cudaStreamWaitEvent(ss, c->prep_done, 0);  // the baby rotations are ready
        c->stream = ss;
        void* wsg = ng > 1 ? (void*)ws_score[gi & 1] : ws;
        const size_t wsg_bytes = ng > 1 ? (size_t)p.ws_score : (size_t)p.ws;
        if (e == cudaSuccess) rc = hann_score_level(c, baby, pt + b0 * ptw, nb, inner + b0 * innerw, wsg, wsg_bytes);
        if (e == cudaSuccess && rc == HANN_OK) rc = hann_rotate_sum(c, inner + b0 * innerw, nb, score + b0 * ctw, wsg, wsg_bytes);
        // canonical form of the group's scores in the staging buffer (first `keep` limbs of every polynomial: with
        // keep < L the exact compaction of hann_compact_scores), then home on the download stream
        const int64_t npoly = nb * 2;
        u64* st = stage + b0 * 2 * kw;
        if (e == cudaSuccess && rc == HANN_OK) rc = launch_copy2d(c, st, kw, score + b0 * ctw, (int64_t)c->L * c->N, kw, npoly);
        if (e == cudaSuccess && rc == HANN_OK) rc = launch_ntt_inv(c, st, npoly * keep, c->N, limbmap_first(keep));
        c->stream = main_stream;
        c->max_lanes = saved_lanes;
        if (e == cudaSuccess && rc == HANN_OK) e = cudaEventRecord(c->grp_ev[gi], ss);
        if (e == cudaSuccess && rc == HANN_OK) e = cudaStreamWaitEvent(c->down_stream, c->grp_ev[gi], 0);
        if (e == cudaSuccess && rc == HANN_OK)
            e = cudaMemcpyAsync(score_ct_host + b0 * 2 * kw, st, (size_t)(npoly * kw) * 8, cudaMemcpyDeviceToHost, c->down_stream);
        if (ce == cudaSuccess) ce = e;
    }
    // join every helper stream before reporting anything
    cudaError_t ej[6];
    ej[0] = cudaStreamWaitEvent(main_stream, c->prep_done, 0);
    ej[1] = cudaStreamWaitEvent(main_stream, c->blk_ev[p.nblk - 1], 0);
    ej[2] = cudaEventRecord(c->down_done, c->down_stream);
    if (ej[2] == cudaSuccess) ej[2] = cudaStreamWaitEvent(main_stream, c->down_done, 0);
    for (int i = 0; i < 2; i++) {
        ej[3 + i] = cudaEventRecord(c->score_join[i], c->score_stream[i]);
        if (ej[3 + i] == cudaSuccess) ej[3 + i] = cudaStreamWaitEvent(main_stream, c->score_join[i], 0);
    }
    ej[5] = cudaSuccess;
    RET(rc);
    CK(ce);
    for (int i = 0; i < 6; i++) CK(ej[i]);
    RET(sync_and_check(c));
    return HANN_OK;
}
