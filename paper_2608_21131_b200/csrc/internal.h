// Private declarations shared by the translation units of the library.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>
#include <string>
#include <vector>

#include "../../include/hann.h"
#include "modarith.cuh"

#define HANN_NKINDS 5  // timed call kinds: query_prepare, encode, score_level, rotate_sum, keyswitch

// kernel classes of the per-launch profile (hann_kernel_profile / hann_kernel_times)
enum {
    KC_NTT_FWD_A = 0, KC_NTT_FWD_B, KC_NTT_INV_B, KC_NTT_INV_A, KC_FFT_A, KC_FFT_B, KC_MAC, KC_LIFT_DIGITS, KC_KS_INNER,
    KC_MODDOWN_LIFT, KC_MODDOWN_COMBINE, KC_PERMUTE, KC_OTHER, KC_KS_INNER_KEYS, KC_COUNT
};

struct hann_ctx {
    hann_params prm;
    int logN = 0, N = 0, n = 0, L = 0, R = 0, B = 0, G = 0;
    int ntt_tau = 0;  // 1 when the transform-domain layout swaps the low nibbles of positions (rings of 2^10 and more)
    int device = 0;
    cudaStream_t stream = nullptr;
    // helper stream and events of hann_query_level, which runs the query preparation beside the candidate encoding
    cudaStream_t aux_stream = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    // further helper streams: hann_rotate_sum runs independent block ranges side by side (aux_stream is lane 1)
    cudaStream_t lane_stream[2] = {nullptr, nullptr};
    cudaEvent_t lane_join[2] = {nullptr, nullptr};
    std::vector<cudaEvent_t> blk_ev;  // one event per block: hann_score_level_host encodes a block as soon as its rows arrived
    // hann_score_level_host: rows travel on up_stream, score ciphertexts on down_stream (both copy engines busy at once);
    // grp_ev[i] marks group i's scores ready in the staging buffer, down_done the end of the downloads
    cudaStream_t up_stream = nullptr, down_stream = nullptr;
    cudaEvent_t down_done = nullptr;
    std::vector<cudaEvent_t> grp_ev;
    int host_groups = 0;  // block groups of hann_score_level_host (0: chosen from the level's size)
    // hann_score_level_host scores its groups on two streams of their own (alternating), beside the encoding of the
    // following groups on the context's stream; enc_ev[i]: group i is encoded; prep_done: the baby rotations are ready
    cudaStream_t score_stream[2] = {nullptr, nullptr};
    cudaEvent_t score_join[2] = {nullptr, nullptr};
    cudaEvent_t prep_done = nullptr;
    std::vector<cudaEvent_t> enc_ev;
    int max_lanes = 4;  // block ranges hann_rotate_sum runs side by side
    u64 mod[HANN_MAXL1] = {};  // q_0..q_{L-1}, p
    LimbTable lt = {};
    LimbConst* lt_dev = nullptr;  // device copy of lt.c (the transform kernels read it from memory)
    // word raised by a kernel that gave up a bounded wait: mapped page-locked host memory (kflag is its device address), read
    // and cleared after the synchronisation that ends every host-pointer call and hann_sync
    int* kflag = nullptr;
    int* kflag_host = nullptr;
    // transform tables on the device, [L+1][N][2]: (w, floor(w*2^64/q)) for w = psi^brev(k) and psi^-brev(k)
    u64 *tw_fwd = nullptr, *tw_inv = nullptr;
    // the same twiddles for the binary64 transform path, [L+1][N][2] doubles: (balanced w, fl(w / q))
    double *tw_fwd_f64 = nullptr, *tw_inv_f64 = nullptr;
    // encode tables on the device
    double2* fft_T = nullptr;  // [n/2] exp(-2 pi i t / n)
    double2* fft_U = nullptr;  // [n]   exp(-i pi k / N)
    int32_t* jinv = nullptr;   // [n]   slot j feeding FFT input position pos: jinv[pos] = j with u_j = brev(pos), u_j = (5^j mod 2N - 1)/4
    unsigned* galois_dev = nullptr;  // [n] 5^r mod 2N
    std::vector<unsigned> h_galois;
    // host copies used by decode
    std::vector<double> hU_re, hU_im;
    std::vector<int32_t> h_uidx;
    // evaluation keys by rotation: device buffers [L][2][L+1][N], transformed and permuted by the inverse
    // automorphism so that the key-switch inner product reads keys and digits contiguously
    std::vector<u64*> keytab_host;
    u64** keytab_dev = nullptr;  // [n] device copy of keytab_host
    // growable device scratch of the exchange and client calls (never used by the server-side scoring calls)
    void* scratch = nullptr;
    int64_t scratch_bytes = 0;
    // plaintexts encoded and transformed per launch group: small enough that the group's intermediates stay in L2
    int encode_group = 1 << 20;
    int host_limbs = 0;  // limbs of every score polynomial that hann_score_level_host downloads (L: all)
    // key-switch lift launches of at most this many CTAs (after the split) are cut along their targets: 160 keeps it to the
    // ModDown lifts of a single item; hann_rotate_sum raises it to 320 for levels of one or two blocks, whose launches
    // otherwise leave most of the machine idle
    int lift_split_ctas = 160;
    // debugging aid: guards behind every workspace sub-buffer (see Arena in api.cu), filled when carved, checked on request
    int canaries = 0;
    std::vector<u64*> guards;
    int pair_b32 = 0;    // hann_score_level_batch pairs queries at B = 32 too (eight warps of four baby steps, FP64 form)
    int mac_f64 = 4;     // how many of a thread's four sums the single-query multiply-accumulate keeps on the FP64 pipe
    int lazy_lanes = 2;  // block ranges hann_rotate_sum_lazy runs side by side
    int giant_lazy = 0;  // hann_rotate_sum (and the calls built on it) evaluates the giant steps in the lazy order
    int encode_sym = 1;  // encode_candidates computes half of every transform and mirrors it (real slot vectors)
    // statistics
    hann_stats stats = {};
    int timing = 0;
    cudaEvent_t ev[HANN_NKINDS][2] = {};
    int ev_pending[HANN_NKINDS] = {};
    // per-launch profile: one event pair per launch while enabled
    int kprof = 0;
    struct KRec { int cls; cudaEvent_t a, b; };
    std::vector<KRec> krec;
    size_t krec_used = 0;
    std::string err;
};

// brackets one kernel launch with events when the per-launch profile is on
struct KProf {
    hann_ctx* c;
    cudaEvent_t b = nullptr;
    KProf(hann_ctx* c_, int cls) : c(c_) {
        c->stats.launches++;
        if (!c->kprof) return;
        if (c->krec_used == c->krec.size()) {
            hann_ctx::KRec r{cls, nullptr, nullptr};
            if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) return;
            c->krec.push_back(r);
        }
        hann_ctx::KRec& r = c->krec[c->krec_used++];
        r.cls = cls;
        cudaEventRecord(r.a, c->stream);
        b = r.b;
    }
    ~KProf() {
        if (b) cudaEventRecord(b, c->stream);
    }
};

// ---- host mathematics (hostmath.cpp)
namespace hm {
u64 mulmod(u64 a, u64 b, u64 q);
u64 powmod(u64 a, u64 e, u64 q);
u64 invmod(u64 a, u64 q);
bool is_prime(u64 n);
u64 find_psi(u64 q, int N);
u64 shoup(u64 w, u64 q);  // floor(w * 2^64 / q)
int bitrev(int x, int bits);
void unit_root(long t, long den, double* c, double* s);  // exp(2 pi i t/den), correctly rounded
// residues [L][N] -> centred integers in (-Q/2, Q/2] as long double
void crt_to_real(const u64* res, int L, int N, const u64* q, long double* out);
void fft_inplace(double* re, double* im, int n, int logn, int sign);
u64 hash64(u64 seed, u64 stream, u64 ctr);  // the 64-bit counter hash of the seeded calls (see hann_expand_uniform)
void seeded_ternary(u64 seed, u64 stream, int N, int8_t* s);                       // uniform on {-1, 0, 1}
void seeded_gaussian(u64 seed, u64 stream, u64 ctr0, long count, double sigma, int8_t* e);  // rounded Gaussian (Box-Muller)
}  // namespace hm

// bytes of workspace one hann_keyswitch carves (api.cu); device address of the built-in scratch (static_scratch.cu)
int64_t keyswitch_ws_bytes(const hann_ctx* c);
int static_scratch_resolve(hann_ctx* c, void** out);

// out = ma * a + mb * b + k on npoly polynomials of c->L limbs (k on the first polynomial of every pair); b may be null
int launch_linear(hann_ctx* c, const u64* a, long long ma, const u64* b, long long mb, long long k, int64_t npoly, u64* out,
                  int64_t b_period = 0);
// d[i] = (a0 b0, a0 b1 + a1 b0, a1 b1) for `count` ciphertext pairs
int launch_mul_ct(hann_ctx* c, const u64* a, const u64* b, int64_t count, u64* d);
int launch_guard_fill(hann_ctx* c, u64* guard);                                             // 32 words of pattern
int launch_guard_verify(hann_ctx* c, u64* const* guards, int64_t count, unsigned long long* damaged);  // counts damaged guards
// debug build: point each translation unit's range-check word at the context's error word (no-ops in a release build)
int debug_bind_keyswitch(int* word);
int debug_bind_project(int* word);
int debug_bind_encode(int* word);

// ---- launchers: each enqueues on ctx->stream, counts its launches and returns HANN_OK or HANN_ECUDA
int check_launch(hann_ctx* c, const char* what);

// transforms of npoly polynomials; polynomial p starts at data + p*stride and uses modulus lm.limb[p % lm.period]
int launch_ntt_fwd(hann_ctx* c, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm);
int launch_ntt_inv(hann_ctx* c, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm);
int launch_ntt_fwd_pass_b(hann_ctx* c, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm);
bool ntt_fwd_half_available(const hann_ctx* c, const void* data, int64_t stride);
int launch_ntt_fwd_pass_b_half(hann_ctx* c, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm);
int launch_copy2d(hann_ctx* c, u64* dst, int64_t dst_pitch, const u64* src, int64_t src_pitch, int64_t width, int64_t rows);
int launch_unpack_half(hann_ctx* c, const u64* half, int64_t npoly, u64* full);
int launch_ntt_inv_pass_b(hann_ctx* c, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm);
bool ntt_inv_pass_b_gathers(const hann_ctx* c, const void* src, const void* dst);
int launch_ntt_inv_pass_b_from(hann_ctx* c, const u64* src, int64_t src_gstride, u64* data, int64_t npoly, int64_t stride, const LimbMap& lm);
bool ks_lift_available(const hann_ctx* c);
int launch_wait_selftest(hann_ctx* c, unsigned long long limit_ns, unsigned long long* waited_ns_dev);
int launch_ks_lift(hann_ctx* c, u64* src, int64_t src_stride, int64_t nsrc, const LimbMap& src_lm, u64* dst, int n_tgt, int tgt_limb0);
// encode a block and run pass A of the transforms in one kernel when the parameters allow it (returns false if not)
bool encode_fused_available(const hann_ctx* c);
int launch_encode_rows_fused(hann_ctx* c, const float* rows, int64_t rows_in_block, int dim, int p_first, int count, u64* out,
                             int64_t out_stride, void* ws, bool sym);
LimbMap limbmap_q(const hann_ctx* c);   // period L: limbs 0..L-1
LimbMap limbmap_qp(const hann_ctx* c);  // period L+1: limbs 0..L
LimbMap limbmap_single(int limb);

// encode (coefficient-domain residues out; the caller transforms)
int launch_encode_rows(hann_ctx* c, const float* rows, int64_t rows_in_block, int dim, int p_first, int count, u64* pt_block,
                       void* ws);
int launch_encode_slots(hann_ctx* c, const double* z_dev, u64* poly_out, void* ws, int log_scale = -1);
// packed projection (project.cu): slot vectors of a packed matrix diagonal and of the window masks; the mask combine
int launch_packed_diagonal(hann_ctx* c, const float* W, int D, int g, int b, double* z);
int launch_window_masks(hann_ctx* c, int b, double* lo, double* hi);
int launch_mask_combine(hann_ctx* c, const u64* ct, const u64* rot_a, const u64* rot_h, const u64* lo, const u64* hi, u64* cyc);
int64_t encode_ws_bytes(const hann_ctx* c);
int64_t encode_fft_bytes(const hann_ctx* c);
int encode_stage_group(const hann_ctx* c);

// scoring
int launch_mac(hann_ctx* c, const u64* baby, const u64* pt, int64_t n_blocks, u64* inner);
// n_queries baby sets against the same blocks: inner [q][n_blocks][G] ciphertexts
int launch_mac_batch(hann_ctx* c, const u64* baby, int n_queries, const u64* pt, int64_t n_blocks, u64* inner);

// key switching pieces
int launch_lift_digits(hann_ctx* c, const u64* src, int64_t src_stride, int64_t nitems, u64* digits);
int launch_ks_inner(hann_ctx* c, const u64* digits, int64_t digit_stride, int rot0, int rot_inc, int64_t nitems, u64* u);
int launch_moddown_lift(hann_ctx* c, const u64* u, int64_t npoly, u64* lifted);
// lazy giant steps (items laid out giant step after giant step, see keyswitch.cu)
int launch_ks_inner_batches(hann_ctx* c, const u64* digits, int64_t digit_stride, int rot0, int rot_zinc, int nz, int64_t per_z, u64* u);
int launch_giant_sum_p(hann_ctx* c, const u64* u, int64_t nblk, u64* up);
int launch_lift_p(hann_ctx* c, const u64* up, int64_t npoly, u64* lifted);
int launch_giant_combine(hann_ctx* c, const u64* u, const u64* lifted, const u64* inner, int64_t nblk, u64* score);
int launch_moddown_combine(hann_ctx* c, const u64* u, const u64* lifted, int64_t nitems, int rot0, int rot_inc, const u64* c0,
                           int64_t c0_stride, const u64* addend, int64_t addend_stride, u64* out0, u64* out1,
                           int64_t out_stride);
int launch_permute(hann_ctx* c, const u64* src, u64* dst, int64_t npoly, unsigned k);
// output compaction: centred lift of coefficient-domain residues mod q_{L-1} into limbs 0..keep-1; (src - lifted) / q_{L-1}
int launch_rescale_lift(hann_ctx* c, const u64* t, int64_t npoly, int keep, u64* lifted);
int launch_rescale_combine(hann_ctx* c, const u64* src, const u64* lifted, int64_t npoly, int keep, u64* out);
LimbMap limbmap_first(int nlimbs);  // period nlimbs: limbs 0..nlimbs-1

// helpers of the client half
int launch_lift_i8(hann_ctx* c, const int8_t* v, int nlimbs, u64* out);
int launch_mul(hann_ctx* c, const u64* a, const u64* b, int bperiod, u64* out, int64_t npoly, const LimbMap& lm);
int launch_add(hann_ctx* c, const u64* a, const u64* b, u64* out, int64_t npoly, const LimbMap& lm);
int launch_evk_finish(hann_ctx* c, const u64* as_coeff, const int8_t* e, const int8_t* sprime, u64* b_out);
int launch_encrypt_finish(hann_ctx* c, const u64* as_coeff, const int8_t* e, const u64* m, u64* c0_out);
// a[L][N] = counter hash of (seed, stream, l*N + x) mod q_l (coefficient domain, canonical)
int launch_expand_uniform(hann_ctx* c, u64 seed, u64 stream, u64* a);
// a[L][L+1][N] = counter hash of (seed, stream, ctr0 + index) reduced into the modulus of each of the L+1 limbs
int launch_expand_uniform_qp(hann_ctx* c, u64 seed, u64 stream, u64 ctr0, u64* a);
// encrypted database: relinearisation key finish, block encryption finish, ct x ct multiply-accumulate
int launch_rlk_finish(hann_ctx* c, const u64* as_coeff, const int8_t* e, const u64* s2, u64* b_out);
int launch_encrypt_block_finish(hann_ctx* c, const u64* pt, const u64* as, const u64* ehat, u64* ct, int64_t npt);
int launch_mac_ct(hann_ctx* c, const u64* baby, const u64* ctdb, int64_t n_bg, u64* inner3);
