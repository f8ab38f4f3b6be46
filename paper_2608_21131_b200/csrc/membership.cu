// The membership (threshold) circuit of the face task as a sequence of the library's own calls (Sec. 3.1, "The norm
// problem", membership bullet; Sec. 2, "Security parameters": depth 11 on a chain of 12 primes).  The server compares the raw
// score <x, q_R> with tau |q_R| = sqrt(tau^2 |q_R|^2) under encryption and returns a ciphertext whose SIGN is the decision:
//   1. t = |q_R|^2 in every slot: the tiled query times itself (ciphertext x ciphertext, relinearised, rescaled), folded over
//      the R slots of a period;
//   2. u = a t + b in [-1, 1] (the factor a is absorbed by the client's encoding: it sends lam q_R, lam^2 = a q_{L-1} / Delta);
//   3. r = sum_k c_k T_k(u), the low-degree Chebyshev interpolant of kappa tau sqrt(t): T_k by the product identity
//      T_{m+n} = 2 T_m T_n - T_{m-n}, m = ceil(k/2); one integer-constant multiply per term brings all terms to one scale;
//   4. s = kappa <x, q_R>: the ordinary scorer (candidates enrolled times kappa / lam) on the level that ends where r ends;
//   5. sign(s - r) ~ f(f(f(.))), f(x) = x (3 - x^2) / 2, the halving done by a rescale over a prime of twice the scale.
// Every ciphertext carries (level, scale); the scale arithmetic below is written operation by operation in IEEE binary64 so
// that any evaluation of the same circuit in the same order gets the same integer constants.
#include <cmath>
#include <algorithm>
#include <string>
#include <utility>
#include <vector>

#include "internal.h"

namespace {

inline int64_t align256(int64_t x) { return (x + 255) & ~(int64_t)255; }

// n ciphertexts of one level and scale, stored one after the other: the circuit's operations act on all of them at once
struct MCt {
    u64* p = nullptr;
    int level = 0;
    double scale = 0;
    int64_t n = 1;
};

struct Circuit {
    hann_ctx* const* arith;   // arith[l - 1]: the first l primes, R = B = 1
    int L;
    hann_ctx* top;            // arith[L - 1]: errors are reported through it
    int N;
    char* base;               // bump area for the circuit's ciphertexts
    int64_t off = 0, cap = 0;
    void* sub;                // workspace lent to the library calls
    size_t sub_bytes;
    int rc = HANN_OK;

    hann_ctx* at(int level) const { return arith[level - 1]; }
    double prime(int i) const { return (double)top->mod[i]; }
    bool fail(int code, const std::string& msg) {
        if (rc == HANN_OK) {
            rc = code;
            top->err = msg;
        }
        return false;
    }
    bool ok(int r, hann_ctx* from) {
        if (r != HANN_OK && rc == HANN_OK) {
            rc = r;
            if (from != top) top->err = from->err;
        }
        return rc == HANN_OK;
    }
    u64* take(int level, int64_t cts = 1) {
        const int64_t bytes = align256(cts * 2 * (int64_t)level * N * 8);
        if (rc != HANN_OK) return nullptr;
        if (off + bytes > cap) {
            fail(HANN_EWORKSPACE, "hann_membership_decide: workspace too small");
            return nullptr;
        }
        u64* r = (u64*)(base + off);
        off += bytes;
        return r;
    }

    // the first `level` primes of a: exact while the ciphertext's content is small against the shorter product
    MCt drop(const MCt& a, int level) {
        if (a.level == level || rc != HANN_OK) return a;
        MCt o{take(level, a.n), level, a.scale, a.n};
        if (o.p) ok(launch_copy2d(at(level), o.p, (int64_t)level * N, a.p, (int64_t)a.level * N, (int64_t)level * N, 2 * a.n), at(level));
        return o;
    }
    // ma a + mb b + k; b is either as many ciphertexts as a or a single one that goes with every ciphertext of a
    MCt linear(const MCt& a, long long ma, const MCt* b, long long mb, long long k, double scale) {
        MCt o{take(a.level, a.n), a.level, scale, a.n};
        if (b && b->n != a.n && b->n != 1) fail(HANN_EINVAL, "hann_membership_decide: internal operand count mismatch");
        const int64_t period = b && b->n == 1 && a.n > 1 ? 2LL * a.level * N : 0;
        if (o.p && rc == HANN_OK) ok(launch_linear(at(a.level), a.p, ma, b ? b->p : nullptr, mb, k, 2 * a.n, o.p, period), at(a.level));
        return o;
    }
    MCt add(const MCt& a0, const MCt& b0, int sign) {
        const int l = a0.level < b0.level ? a0.level : b0.level;
        const MCt a = drop(a0, l), b = drop(b0, l);
        return linear(a, 1, &b, sign, 0, a.scale);
    }
    // c - a
    MCt const_minus(const MCt& a, double c) { return linear(a, -1, nullptr, 0, (long long)std::nearbyint(c * a.scale), a.scale); }
    MCt add_const(const MCt& a, double c) { return linear(a, 1, nullptr, 0, (long long)std::nearbyint(c * a.scale), a.scale); }
    MCt mul_int(const MCt& a, long long m) { return linear(a, m, nullptr, 0, 0, a.scale); }
    MCt rescale(const MCt& a) {
        MCt o{take(a.level - 1, a.n), a.level - 1, a.scale / prime(a.level - 1), a.n};
        if (o.p) ok(hann_rescale(at(a.level), a.p, a.n, o.p, sub, sub_bytes), at(a.level));
        return o;
    }
    // ciphertext x ciphertext, pair by pair: the degree-2 product with one relinearisation, then the rescale
    MCt mul(const MCt& a0, const MCt& b0) {
        const int l = a0.level < b0.level ? a0.level : b0.level;
        const MCt a = drop(a0, l), b = drop(b0, l);
        if (a.n != b.n) fail(HANN_EINVAL, "hann_membership_decide: internal operand count mismatch");
        MCt prod{take(l, a.n), l, a.scale * b.scale, a.n};
        if (prod.p && rc == HANN_OK) ok(hann_multiply(at(l), a.p, b.p, a.n, prod.p, sub, sub_bytes), at(l));
        return rescale(prod);
    }
    // several independent products on one level in ONE multiply and ONE rescale call: pairs[i] = (a_i, b_i), every pair with
    // the same lower level; the operands are gathered into two rows of ciphertexts first.  Item i comes back with its own scale
    // (a_i.scale b_i.scale / q_last), as mul() would have given it; the bits are mul()'s too (the items do not interact).
    std::vector<MCt> mul_many(const std::vector<std::pair<MCt, MCt>>& pairs) {
        const int64_t k = (int64_t)pairs.size();
        std::vector<MCt> out((size_t)k);
        if (k == 0 || rc != HANN_OK) return out;
        int l = pairs[0].first.level < pairs[0].second.level ? pairs[0].first.level : pairs[0].second.level;
        for (const auto& pr : pairs) {
            const int li = pr.first.level < pr.second.level ? pr.first.level : pr.second.level;
            if (li != l || pr.first.n != 1 || pr.second.n != 1) fail(HANN_EINVAL, "hann_membership_decide: internal level mismatch in a batch of products");
        }
        const int64_t ctw = 2LL * l * N;
        MCt a{take(l, k), l, 0, k}, b{take(l, k), l, 0, k}, prod{take(l, k), l, 0, k};
        if (!a.p || !b.p || !prod.p || rc != HANN_OK) return out;
        for (int64_t i = 0; i < k && rc == HANN_OK; i++) {
            const MCt &x = pairs[(size_t)i].first, &y = pairs[(size_t)i].second;
            ok(launch_copy2d(at(l), a.p + i * ctw, (int64_t)l * N, x.p, (int64_t)x.level * N, (int64_t)l * N, 2), at(l));
            ok(launch_copy2d(at(l), b.p + i * ctw, (int64_t)l * N, y.p, (int64_t)y.level * N, (int64_t)l * N, 2), at(l));
        }
        if (rc == HANN_OK) ok(hann_multiply(at(l), a.p, b.p, k, prod.p, sub, sub_bytes), at(l));
        const MCt low = rescale(prod);
        if (!low.p || rc != HANN_OK) return out;
        const int64_t ctw_low = 2LL * (l - 1) * N;
        for (int64_t i = 0; i < k; i++)
            out[(size_t)i] = MCt{low.p + i * ctw_low, l - 1, (pairs[(size_t)i].first.scale * pairs[(size_t)i].second.scale) / prime(l - 1), 1};
        return out;
    }
    MCt rotate(const MCt& a, int r) {
        MCt o{take(a.level), a.level, a.scale};
        if (o.p) ok(hann_rotate_hoisted(at(a.level), a.p, r, 1, o.p, sub, sub_bytes), at(a.level));
        return o;
    }
};

int threshold_depth(int deg) {
    int lg = 0;
    while ((1 << lg) < deg) lg++;
    return 1 + lg + 1;
}

}  // namespace

extern "C" int hann_membership_levels(int deg, int sign_iters, int* chain_primes, int* score_level) {
    if (deg < 1 || deg > 15 || sign_iters < 0 || !chain_primes || !score_level) return HANN_EINVAL;
    *chain_primes = threshold_depth(deg) + 2 * sign_iters + 1;
    *score_level = *chain_primes - threshold_depth(deg) + 1;
    return HANN_OK;
}

extern "C" int64_t hann_membership_bytes(hann_ctx* const* arith, int L, const hann_ctx* scorer, const hann_membership_params* prm,
                                         int64_t n_blocks) {
    if (!arith || !scorer || !prm || L < 2 || n_blocks < 0) return HANN_EINVAL;
    for (int l = 1; l <= L; l++)
        if (!arith[l - 1]) return HANN_EINVAL;
    const int64_t N = arith[L - 1]->N, ct_top = align256(2 * (int64_t)L * N * 8);
    // The circuit's ciphertexts never share storage.  Counted at the size of a ciphertext of the full chain (most live on
    // shorter ones): at most 12 per Chebyshev term (two level drops, product, rescale, doubling, the difference, and drop /
    // multiple / rescale / sum in the combination), 2 per fold step, 3 per block plus 8 per sign iteration, 16 spare.
    int folds = 0;
    while ((1 << folds) < prm->R) folds++;
    const int64_t cts = 16 + 12 * (int64_t)prm->deg + 2 * folds + n_blocks * (3 + 8 * (int64_t)prm->sign_iters);
    int64_t sub = 0;
    for (int l = 1; l <= L; l++) sub = std::max<int64_t>(sub, hann_workspace_bytes(arith[l - 1], l < scorer->L ? std::max<int64_t>(n_blocks, 4) : 4));
    sub = std::max<int64_t>(sub, hann_workspace_bytes(scorer, 8));
    const int64_t scoring = align256(hann_sizeof(scorer, HANN_SIZE_BABY)) + n_blocks * (align256(hann_sizeof(scorer, HANN_SIZE_INNER)) +
                                                                                      align256(hann_sizeof(scorer, HANN_SIZE_CT)));
    return cts * ct_top + scoring + align256(sub) + 4096;
}

extern "C" int hann_membership_decide(hann_ctx* const* arith, int L, hann_ctx* scorer, const hann_membership_params* prm,
                                      const void* ct_dev, const void* pt_dev, int64_t n_blocks, void* out_dev, double* out_scale,
                                      void* thr_dev, int* thr_level, double* thr_scale, void* ws, size_t ws_bytes) {
    if (!arith || L < 2 || !arith[L - 1]) return HANN_EINVAL;
    hann_ctx* top = arith[L - 1];
    auto bad = [&](int code, const char* msg) {
        top->err = msg;
        return code;
    };
    if (!scorer || !prm || !prm->coef || !ct_dev || !out_dev || !out_scale || n_blocks < 0 || (n_blocks > 0 && !pt_dev))
        return bad(HANN_EINVAL, "hann_membership_decide: bad argument");
    int want_L = 0, score_level = 0;
    if (hann_membership_levels(prm->deg, prm->sign_iters, &want_L, &score_level) != HANN_OK || want_L != L)
        return bad(HANN_ESHAPE, "hann_membership_decide: the chain must have depth(threshold) + 2 * sign iterations + 1 primes");
    for (int l = 1; l <= L; l++) {
        const hann_ctx* a = arith[l - 1];
        if (!a || a->L != l || a->N != top->N || a->R != 1 || a->B != 1 || a->device != top->device || a->stream != top->stream)
            return bad(HANN_ESHAPE, "hann_membership_decide: arith[l-1] must be the context of the first l primes with R = B = 1");
        for (int i = 0; i < l; i++)
            if (a->mod[i] != top->mod[i]) return bad(HANN_ESHAPE, "hann_membership_decide: the contexts must share one chain of primes");
        if (a->mod[l] != top->mod[L]) return bad(HANN_ESHAPE, "hann_membership_decide: the contexts must share the special prime");
    }
    if (scorer->L != score_level || scorer->N != top->N || scorer->R != prm->R || scorer->device != top->device || scorer->stream != top->stream)
        return bad(HANN_ESHAPE, "hann_membership_decide: the scorer must be the context of the first (L - depth(threshold) + 1) primes with rank R");
    for (int i = 0; i < score_level; i++)
        if (scorer->mod[i] != top->mod[i]) return bad(HANN_ESHAPE, "hann_membership_decide: the scorer must use the chain's primes");
    if (prm->R < 1 || (prm->R & (prm->R - 1)) || prm->t_hi <= prm->t_lo || prm->log_scale < 1 || prm->log_scale > 60)
        return bad(HANN_EINVAL, "hann_membership_decide: R must be a power of two, t_lo < t_hi");
    if (!ws || ((uintptr_t)ws & 255)) return bad(HANN_EWORKSPACE, "hann_membership_decide: workspace missing or not 256-byte aligned");
    if ((int64_t)ws_bytes < hann_membership_bytes(arith, L, scorer, prm, n_blocks)) return bad(HANN_EWORKSPACE, "hann_membership_decide: workspace too small");

    const int N = top->N;
    int64_t sub = 0;
    // below the scorer's level the operations run over all blocks at once, above it over the up to four products of one depth of
    // the Chebyshev basis: room for several key switches side by side
    for (int l = 1; l <= L; l++) sub = std::max<int64_t>(sub, hann_workspace_bytes(arith[l - 1], l < score_level ? std::max<int64_t>(n_blocks, 4) : 4));
    sub = align256(std::max<int64_t>(sub, hann_workspace_bytes(scorer, 8)));
    Circuit C;
    C.arith = arith; C.L = L; C.top = top; C.N = N;
    C.sub = ws; C.sub_bytes = (size_t)sub;
    C.base = (char*)ws + sub; C.cap = (int64_t)ws_bytes - sub;
    top->err.clear();

    const double delta = std::ldexp(1.0, prm->log_scale), a = 2.0 / (prm->t_hi - prm->t_lo);
    const double lam = std::sqrt(a * C.prime(L - 1) / delta);
    const MCt q{(u64*)ct_dev, L, delta};

    // 1, 2: |q_R|^2 (times lam^2) in every slot, read as a t at scale Delta; u = a t - (t_hi + t_lo) / (t_hi - t_lo)
    MCt t = C.mul(q, q);
    for (int r = 1; r < prm->R; r <<= 1) t = C.add(t, C.rotate(t, r), 1);
    t.scale = t.scale / (lam * lam) * a;
    const MCt u = C.add_const(t, -(prm->t_hi + prm->t_lo) / (prm->t_hi - prm->t_lo));
    // 3: Chebyshev basis by the product identity, then the combination at one common scale
    // (the products of one depth do not depend on each other: T_3, T_4 need T_1, T_2 only, T_5 .. T_7 need T_2 .. T_4; each depth
    // is one batched multiply and rescale)
    std::vector<MCt> T(prm->deg + 1);
    T[1] = u;
    for (int k0 = 2; k0 <= prm->deg;) {
        // the run of k whose operands T_ceil(k/2), T_floor(k/2) exist already: k0 .. min(deg, 2 (k0 - 1))
        const int k1 = std::min(prm->deg, 2 * (k0 - 1));
        std::vector<std::pair<MCt, MCt>> pairs;
        for (int k = k0; k <= k1; k++) pairs.emplace_back(T[(k + 1) / 2], T[k - (k + 1) / 2]);
        // a batch needs one common level; it has one whenever the run starts at a power of two plus one .. (checked by mul_many:
        // the lower operand of every pair of a run lies on the run's deepest level); single products go through mul()
        bool same = true;
        for (const auto& pr : pairs) same = same && std::min(pr.first.level, pr.second.level) == std::min(pairs[0].first.level, pairs[0].second.level);
        std::vector<MCt> prods;
        if (same && pairs.size() > 1) prods = C.mul_many(pairs);
        else for (const auto& pr : pairs) prods.push_back(C.mul(pr.first, pr.second));
        if (C.rc != HANN_OK) return C.rc;
        for (int k = k0; k <= k1; k++) {
            const int m = (k + 1) / 2, nn = k - m;
            const MCt prod2 = C.mul_int(prods[(size_t)(k - k0)], 2);
            T[k] = m == nn ? C.add_const(prod2, -1.0) : C.add(prod2, T[m - nn], -1);
        }
        k0 = k1 + 1;
    }
    int level = T[1].level;
    for (int k = 1; k <= prm->deg; k++) level = T[k].level < level ? T[k].level : level;
    level -= 1;
    // every term's integer multiple (to_scale) lands in one row of ciphertexts, which takes ONE rescale call
    std::vector<int> ks;
    for (int k = 1; k <= prm->deg; k++)
        if (std::fabs(prm->coef[k]) >= 1e-15) ks.push_back(k);
    MCt acc;
    if (!ks.empty() && C.rc == HANN_OK) {
        const int lv = level + 1;
        const int64_t nt = (int64_t)ks.size(), ctw = 2LL * lv * N, ctw_low = 2LL * level * N;
        const double ql = C.prime(lv - 1);
        MCt row{C.take(lv, nt), lv, 0, nt};
        std::vector<double> scales((size_t)nt);
        for (int64_t i = 0; i < nt && row.p && C.rc == HANN_OK; i++) {
            const MCt a = C.drop(T[ks[(size_t)i]], lv);
            const double factor = prm->coef[ks[(size_t)i]];
            const double m = std::nearbyint(((factor * delta) * ql) / a.scale);   // as to_scale()
            if (a.p) C.ok(launch_linear(C.at(lv), a.p, (long long)m, nullptr, 0, 0, 2, row.p + i * ctw), C.at(lv));
            scales[(size_t)i] = ((a.scale * m) / ql) / factor;
        }
        const MCt low = C.rescale(row);
        for (int64_t i = 0; i < nt && low.p && C.rc == HANN_OK; i++) {
            const MCt term{low.p + i * ctw_low, level, scales[(size_t)i], 1};
            acc = acc.p ? C.add(acc, term, 1) : term;
        }
    }
    if (C.rc == HANN_OK && !acc.p) return bad(HANN_EINVAL, "hann_membership_decide: all polynomial coefficients vanish");
    const MCt thr = C.add_const(acc, prm->coef[0]);
    if (C.rc != HANN_OK) return C.rc;
    if (thr.level + 1 != score_level) return bad(HANN_ESHAPE, "hann_membership_decide: internal level mismatch");
    if (thr_dev) {
        C.ok(launch_copy2d(C.at(thr.level), (u64*)thr_dev, 2LL * thr.level * N, thr.p, 2LL * thr.level * N, 2LL * thr.level * N, 1), C.at(thr.level));
        if (thr_level) *thr_level = thr.level;
        if (thr_scale) *thr_scale = thr.scale;
    }
    // 4: the scores of every block on the scorer's level, rescaled onto the threshold's level; 5: sign iterations
    if (n_blocks > 0) {
        const MCt qs = C.drop(q, score_level);
        const int64_t babyb = align256(hann_sizeof(scorer, HANN_SIZE_BABY)), innerb = align256(hann_sizeof(scorer, HANN_SIZE_INNER));
        u64* baby = nullptr;
        u64* inner = nullptr;
        if (C.rc == HANN_OK) {
            if (C.off + babyb + n_blocks * innerb > C.cap) return bad(HANN_EWORKSPACE, "hann_membership_decide: workspace too small");
            baby = (u64*)(C.base + C.off); C.off += babyb;
            inner = (u64*)(C.base + C.off); C.off += n_blocks * innerb;
        }
        u64* score = C.take(score_level, n_blocks);
        if (C.rc == HANN_OK) {
            C.ok(hann_query_prepare(scorer, qs.p, baby, C.sub, C.sub_bytes), scorer);
            C.ok(hann_score_level(scorer, baby, pt_dev, n_blocks, inner, C.sub, C.sub_bytes), scorer);
            C.ok(hann_rotate_sum(scorer, inner, n_blocks, score, C.sub, C.sub_bytes), scorer);
        }
        // all blocks advance together: every operation below is one (chunked) call over n_blocks ciphertexts
        if (C.rc == HANN_OK) {
            const MCt s = C.rescale(MCt{score, score_level, qs.scale * delta, n_blocks});
            MCt x = C.add(s, thr, -1);
            for (int it = 0; it < prm->sign_iters; it++) {
                const MCt w = C.const_minus(C.mul(x, x), 3.0);         // 3 - x^2 over a prime ~Delta
                x = C.mul(x, w);                                      // x (3 - x^2) over a prime ~2 Delta ...
                x.scale *= 2.0;                                       // ... read at the same scale it is x (3 - x^2) / 2
            }
            if (C.rc != HANN_OK) return C.rc;
            if (x.level != 1) return bad(HANN_ESHAPE, "hann_membership_decide: internal level mismatch at the output");
            C.ok(launch_copy2d(C.at(1), (u64*)out_dev, 2LL * N, x.p, 2LL * N, 2LL * N, n_blocks), C.at(1));
            *out_scale = x.scale;
        }
    }
    return C.rc;
}
