"""Pins of the CPU oracle against what the scheme and the mathematics fix, none of them the oracle itself:
python-integer schoolbook products, direct polynomial evaluation, multi-precision cosine sums, explicit slot
permutations, the known error arrays, the analytic key-switch noise bound, plain float64 matrix-vector products.
"""
import math

import mpmath
import numpy as np
import pytest
import sympy

from oracle.oracle import Oracle, PackedProjection, find_primes, is_prime, restrict_keys
from paper_2608_21131_b200 import synth
from tests.helpers import rescale_error_bound, rescale_error_sigma


def make(ps):
    return Oracle(ps.logN, ps.q, ps.p, ps.log_scale, ps.R, ps.B)


def schoolbook_negacyclic(a, b, q):
    N = len(a)
    out = [0] * N
    for i in range(N):
        for j in range(N):
            k = i + j
            v = int(a[i]) * int(b[j])
            if k < N:
                out[k] = (out[k] + v) % q
            else:
                out[k - N] = (out[k - N] - v) % q
    return out


def rand_poly(rng, N, q):
    return np.array([int(rng.integers(0, q)) for _ in range(N)], dtype=np.uint64)


# ------------------------------------------------------------------ primes


def test_primes_are_the_largest_below_the_bound():
    for bits, logstep, want in ((50, 17, synth.Q50), (60, 17, (synth.P60,)), (30, 13, synth.Q30), (31, 13, (synth.P31,))):
        got = find_primes(bits, logstep, len(want))
        assert tuple(got) == tuple(want)
        step = 1 << logstep
        # brute recomputation with an independent primality test: every skipped candidate is composite
        c = (1 << bits) - step + 1
        found = []
        while len(found) < len(want):
            if sympy.isprime(c):
                found.append(c)
            c -= step
        assert tuple(found) == tuple(want)


def test_miller_rabin_agrees_with_sympy():
    rng = np.random.default_rng(0)
    for x in [0, 1, 2, 3, 4, 561, 2147377153, 2147377155, 3215031751, 2 ** 61 - 1, 2 ** 61 + 1]:
        assert is_prime(x) == sympy.isprime(x)
    for x in rng.integers(2, 2 ** 62, size=300):
        assert is_prime(int(x) | 1) == sympy.isprime(int(x) | 1)


# ------------------------------------------------------------------ NTT


@pytest.mark.parametrize("logN,big", [(4, False), (6, False), (8, False), (8, True)])
def test_ntt_roundtrip_definition_and_schoolbook(logN, big):
    ps = synth.small_params(logN, 4, 2, big=big)
    o = make(ps)
    rng = np.random.default_rng(logN)
    N = ps.N
    for limb in range(ps.L + 1):
        q = o.mods[limb]
        a, b = rand_poly(rng, N, q), rand_poly(rng, N, q)
        assert np.array_equal(o.intt(limb, o.ntt(limb, a)), a)
        # definition: a_hat[t] = a(psi^(2t+1))
        psi = o.psi(limb)
        assert pow(psi, N, q) == q - 1
        ah = o.ntt(limb, a)
        for t in (0, 1, N // 2, N - 1):
            x = pow(psi, 2 * t + 1, q)
            assert int(ah[t]) == sum(int(a[i]) * pow(x, i, q) for i in range(N)) % q
        # product through the transform == schoolbook product in Z_q[X]/(X^N+1)
        got = o.negacyclic_mul(limb, a, b)
        assert [int(v) for v in got] == schoolbook_negacyclic(a, b, q)


def test_crt_roundtrip():
    o = make(synth.small_params(4, 4, 2, L=4, big=True))
    rng = np.random.default_rng(1)
    vals = [int(rng.integers(-2 ** 62, 2 ** 62)) * int(rng.integers(1, 2 ** 62)) * int(rng.integers(1, 2 ** 62)) for _ in range(14)]
    vals += [o.Q // 2, -(o.Q // 2)]
    assert all(abs(v) <= o.Q // 2 for v in vals)
    res = o.reduce(vals)
    back = o.crt_centred(res)
    assert [int(v) for v in back] == vals


# ------------------------------------------------------------------ encode / decode


def exact_encode(z, N, log_scale):
    """m_k = rint((Delta/n) sum_j z_j cos(pi g_j k / N)) in 200-bit arithmetic; also returns the distance of the
    exact value from the nearest half-integer (a near-tie may legitimately round either way in binary64)."""
    mpmath.mp.prec = 200
    n = N // 2
    g = [pow(5, j, 2 * N) for j in range(n)]
    zs = [mpmath.mpf(float(v)) for v in z]
    cos_tab = [mpmath.cos(mpmath.pi * t / N) for t in range(2 * N)]   # cos(pi t / N), t mod 2N
    out, margin = [], []
    for k in range(N):
        acc = mpmath.mpf(0)
        for j in range(n):
            acc += zs[j] * cos_tab[(g[j] * k) % (2 * N)]
        val = acc * mpmath.mpf(2) ** log_scale / n
        out.append(int(mpmath.nint(val)))
        margin.append(float(abs(abs(val - mpmath.floor(val)) - mpmath.mpf(0.5))))
    return out, margin


@pytest.mark.parametrize("logN", [3, 4, 6, 8])
def test_encode_equals_exact_cosine_sum(logN):
    ps = synth.small_params(logN, 1, 1)
    o = make(ps)
    z = synth.gaussian(9, logN, np.arange(ps.n))
    m = o.encode(z, 25)
    want, margin = exact_encode(z, ps.N, 25)
    for k in range(ps.N):
        assert int(m[k]) == want[k] or (abs(int(m[k]) - want[k]) == 1 and margin[k] < 1e-6)
    assert sum(int(m[k]) != want[k] for k in range(ps.N)) == 0


def test_encode_equals_exact_cosine_sum_at_the_production_scale():
    """the same pin at N = 1024 and scale 2^40, the scale of every configuration but the toy: coefficients of ~2^35
    (Delta |z| / sqrt(n)) need 35 of the 53 mantissa bits, so a sloppier evaluation order than the pinned one, or a
    table that is not correctly rounded, would show here first"""
    ps = synth.small_params(10, 1, 1)
    o = make(ps)
    z = synth.gaussian(11, 40, np.arange(ps.n))
    m = o.encode(z, 40)
    want, margin = exact_encode(z, ps.N, 40)
    assert max(abs(int(v)) for v in want) > 2 ** 34
    bad = [k for k in range(ps.N) if int(m[k]) != want[k]]
    # the binary64 evaluation carries a relative error of a few 2^-53 per operation into values of ~2^35, i.e. ~2^-15 of
    # a unit: only an exact value within that distance of a half-integer may round the other way
    assert all(abs(int(m[k]) - want[k]) == 1 and margin[k] < 2.0 ** -10 for k in bad), bad
    assert len(bad) <= 1


@pytest.mark.parametrize("logN,big", [(4, False), (8, False), (10, True)])
def test_encoding_of_real_slots_is_fixed_by_conjugation(logN, big):
    """cos(pi g (N - k) / N) = -cos(pi g k / N) for odd g, so the cosine sum gives m_{N-k} = -m_k (and m_n = 0): the
    encoding is fixed by X -> 1/X = -X^(N-1).  The pinned binary64 evaluation keeps this to the last bit, and the
    transform therefore takes the same value at psi^(2t+1) and at its inverse psi^(2(N-1-t)+1)."""
    ps = synth.small_params(logN, 1, 1, big=big)
    o = make(ps)
    z = synth.gaussian(3, logN, np.arange(ps.n)) * 3.0
    m = o.encode(z, 25)
    assert m[ps.n] == 0
    assert np.array_equal(m[1:][::-1], -m[1:])
    for limb in range(ps.L):
        q = o.mods[limb]
        res = np.array([int(v) % q for v in m], dtype=np.uint64)
        ah = o.ntt(limb, res)
        assert np.array_equal(ah, ah[::-1])


def test_encode_known_answer_n8():
    # N = 8, Delta = 2^10, z = (1/4, 1/2, 3/4, 1): m_0 = (Delta/n) * sum z = 256 * 2.5 = 640; the other
    # coefficients are (Delta/n) sum_j z_j cos(pi g_j k/8) with g = (1, 5, 9, 13), e.g.
    # m_4 = 256 * (cos(pi/2))*(...) = 0 and m_k = -m_{8-k} for odd symmetry of the cosine sum.
    o = Oracle(3, synth.Q30, synth.P31, 10, 1, 1)
    m = o.encode(np.array([0.25, 0.5, 0.75, 1.0]), 10)
    assert m.tolist() == [640, -69, -91, -167, 0, 167, 91, 69]
    # rotation by one slot is X -> X^5 on the coefficients
    res = o.reduce(m, 1)[0]
    rot = o.automorphism(0, 5, res)
    cent = [int(v) if int(v) < o.mods[0] // 2 else int(v) - o.mods[0] for v in rot]
    assert cent == [640, -167, 91, 69, 0, -69, -91, 167]
    assert cent == o.encode(np.array([0.5, 0.75, 1.0, 0.25]), 10).tolist()


def test_index_tables():
    t = Oracle(3, synth.Q30, synth.P31, 10, 1, 1).tables()
    assert t["g5"].tolist() == [1, 5, 9, 13] and t["uidx"].tolist() == [0, 1, 2, 3]
    t = Oracle(5, synth.Q30, synth.P31, 10, 1, 1).tables()
    assert t["uidx"].tolist() == [0, 1, 6, 15, 12, 13, 2, 11, 8, 9, 14, 7, 4, 5, 10, 3]
    assert t["g5"].tolist() == [pow(5, j, 64) for j in range(16)]
    assert sorted(t["uidx"].tolist()) == list(range(16))


@pytest.mark.parametrize("logN,stride", [(10, 1), (12, 1), (16, 37)])
def test_unit_root_tables_are_correctly_rounded(logN, stride):
    mpmath.mp.prec = 200
    o = Oracle(logN, synth.Q50[:1], synth.P60, 40, 1, 1)
    t = o.tables()
    n, N = o.n, o.N
    assert t["T_re"][0] == 1.0 and t["T_im"][0] == 0.0
    assert t["T_re"][n // 4] == 0.0 and t["T_im"][n // 4] == -1.0
    assert t["U_re"][0] == 1.0 and t["U_im"][0] == 0.0
    assert t["U_re"][n // 2] == -t["U_im"][n // 2]
    for k in list(range(0, n // 2, stride)) + [n // 2 - 1]:
        x = mpmath.mpf(2 * k) / n  # angle / pi, exact
        assert t["T_re"][k] == float(mpmath.cospi(x)) and t["T_im"][k] == float(-mpmath.sinpi(x))
    for k in list(range(0, n, stride)) + [n - 1]:
        x = mpmath.mpf(k) / N
        assert t["U_re"][k] == float(mpmath.cospi(x)) and t["U_im"][k] == float(-mpmath.sinpi(x))


def test_encode_special_cases_and_decode_roundtrip():
    ps = synth.small_params(10, 1, 1)
    o = make(ps)
    assert not o.encode(np.zeros(ps.n)).any()
    m = o.encode(np.full(ps.n, 0.3125))
    assert m[0] == round(0.3125 * 2 ** 25) and not m[1:].any()
    z = synth.uniform(4, 0, np.arange(ps.n)) * 2 - 1
    m = o.encode(z)
    back = o.decode(m.astype(np.float64), 2.0 ** 25)
    err = np.abs(back - z)
    # coefficient rounding error is uniform(-1/2,1/2) per coefficient: slot error std sqrt(N/12)/Delta
    std = math.sqrt(ps.N / 12) / 2 ** 25
    assert err.max() < 6 * std and err.max() > 0.2 * std


@pytest.mark.parametrize("r", [1, 3, 7])
def test_automorphism_is_slot_rotation_and_ntt_gather(r):
    ps = synth.small_params(8, 1, 1)
    o = make(ps)
    z = synth.uniform(5, r, np.arange(ps.n))
    m = o.encode(z)
    k = o.galois(r)
    assert k == pow(5, r, 2 * ps.N)
    res = o.reduce(m, 1)[0]
    rot = o.automorphism(0, k, res)
    q = o.mods[0]
    cent = np.array([int(v) if int(v) <= q // 2 else int(v) - q for v in rot], dtype=np.float64)
    back = o.decode(cent, 2.0 ** 25).real
    assert np.abs(back - np.roll(z, -r)).max() < 1e-5  # left rotation: out[i] = z[i + r]
    # bit-exact form of the same statement: phi_k(encode(z)) == encode(roll(z)) up to rounding ties only
    assert np.abs(cent - o.encode(np.roll(z, -r))).max() <= 1
    # transform-domain gather == transform of the coefficient-domain map
    assert np.array_equal(o.automorphism_ntt(k, o.ntt(0, res)), o.ntt(0, rot))


# ------------------------------------------------------------------ encryption


def test_decrypt_of_encrypt_returns_message_plus_the_error_array():
    ps = synth.small_params(8, 4, 2, L=2)
    o = make(ps)
    km = synth.key_material(ps, 11)
    m = (synth.gaussian(1, 0, np.arange(ps.N)) * 1e6).astype(np.int64)
    ct = o.encrypt(km.s, m, km.ct_a, km.ct_e)
    assert np.array_equal(ct[1], km.ct_a)
    mu = o.decrypt_int(km.s, ct)
    assert [int(v) for v in mu] == [int(a) + int(b) for a, b in zip(m, km.ct_e)]


# ------------------------------------------------------------------ key switching


def centred_product_mod_Q(o, d_res, s2):
    """d * s2 mod Q as centred python integers, by schoolbook over the integers (N small)."""
    d = o.crt_centred(d_res)
    N = o.N
    out = [0] * N
    for i in range(N):
        if s2[i] == 0:
            continue
        for j in range(N):
            k = i + j
            v = int(s2[i]) * int(d[j])
            if k < N:
                out[k] += v
            else:
                out[k - N] -= v
    Q = o.Q
    return [((v + Q // 2) % Q) - Q // 2 for v in out]


def signed_automorphism(s, k, N):
    out = np.zeros(N, dtype=np.int64)
    for i in range(N):
        e = (i * k) % (2 * N)
        if e < N:
            out[e] = s[i]
        else:
            out[e - N] = -s[i]
    return out


@pytest.mark.parametrize("big", [False, True])
def test_keyswitch_error_within_analytic_bound(big):
    ps = synth.small_params(8, 8, 4, L=2, big=big)
    o = make(ps)
    km = synth.key_material(ps, 21)
    rng = np.random.default_rng(2)
    r = 3
    evk = o.evk_gen(km.s, r, km.evk_a[r - 1], km.evk_e[r - 1])
    d = np.stack([rand_poly(rng, ps.N, q) for q in ps.q])
    ks0, ks1 = o.keyswitch(d, evk)
    s2 = signed_automorphism(km.s, o.galois(r), ps.N)
    want = centred_product_mod_Q(o, d, s2)
    # ks0 + ks1*s as centred integers
    ct = np.stack([ks0, ks1])
    got = o.decrypt_int(km.s, ct)
    Q = o.Q
    err = np.array([float(((int(g) - int(w) + Q // 2) % Q) - Q // 2) for g, w in zip(got, want)])
    qmean = float(np.mean([float(x) for x in ps.q]))
    std = math.sqrt(ps.L * ps.N * 3.2 ** 2 * qmean ** 2 / (12 * float(ps.p) ** 2) + ps.N / 18.0)
    assert abs(err.mean()) < 0.5 * std
    assert 0.7 * std < err.std() < 1.3 * std
    assert np.abs(err).max() < 6 * std


def test_moddown_of_multiple_of_p_is_exact():
    ps = synth.small_params(6, 4, 2, L=2, big=True)
    o = make(ps)
    rng = np.random.default_rng(3)
    x = [int(rng.integers(-2 ** 40, 2 ** 40)) for _ in range(ps.N)]
    px = [v * ps.p for v in x]
    u = o.reduce(px, ps.L + 1)
    out = o.moddown(u)
    assert [int(v) for v in o.crt_centred(out)] == x
    # and rounds to nearest otherwise
    px1 = [v * ps.p + ps.p // 2 - 3 for v in x]
    assert [int(v) for v in o.crt_centred(o.moddown(o.reduce(px1, ps.L + 1)))] == x


def test_rotate_decrypts_to_left_rotation_and_hoisting_is_bit_identical():
    ps = synth.small_params(8, 8, 4, L=2)
    o = make(ps)
    km = synth.key_material(ps, 31)
    z = synth.uniform(6, 0, np.arange(ps.n)) - 0.5
    ct = o.encrypt(km.s, o.encode(z), km.ct_a, km.ct_e)
    for r in (1, 4):
        evk = o.evk_gen(km.s, r, km.evk_a[r - 1], km.evk_e[r - 1])
        rot = o.rotate(ct, r, evk)
        back = o.decrypt_slots(km.s, rot, ps.log_scale).real
        assert np.abs(back - np.roll(z, -r)).max() < 2e-4
        assert np.array_equal(rot, o.rotate(ct, r, evk, hoisted=True))


# ------------------------------------------------------------------ diagonal / BSGS scoring


def all_keys(o, km):
    return np.stack([o.evk_gen(km.s, r, km.evk_a[i], km.evk_e[i]) for i, r in enumerate(km.rots)])


@pytest.mark.parametrize("logN,R,B", [(4, 4, 2), (5, 4, 2), (6, 8, 2), (6, 4, 4), (6, 4, 1)])
def test_bsgs_without_noise_equals_plain_matvec(logN, R, B):
    ps = synth.small_params(logN, R, B, L=2)
    o = make(ps)
    km = synth.key_material(ps, 41, zero_noise=True)
    rows = synth.toy_corpus(3, rows=ps.n - 3, dim=R)  # ragged block: last 3 rows missing
    qv = synth.toy_query(4, dim=R)
    ct = o.encrypt_query(km.s, qv, km.ct_a, km.ct_e)
    evk = all_keys(o, km)
    baby = o.baby_set(ct, evk)
    score, pt, inner = o.score_block(rows, baby, evk[B - 1], True, True)
    got = o.decrypt_slots(km.s, score, 2 * ps.log_scale)
    want = np.zeros(ps.n)
    want[: ps.n - 3] = rows.astype(np.float64) @ qv.astype(np.float64)
    # only encode rounding and key-switch rounding remain
    assert np.abs(got.real - want).max() < 2e-5 and np.abs(got.imag).max() < 2e-5
    # each plaintext decodes to the pre-rotated diagonal it was built from
    M = np.zeros((ps.n, R))
    M[: ps.n - 3] = rows
    for g in range(ps.G):
        for b in range(B):
            cent = [int(v) if int(v) <= ps.q[0] // 2 else int(v) - ps.q[0] for v in pt[g, b, 0]]
            z = o.decode(np.array(cent, dtype=np.float64), 2.0 ** ps.log_scale).real
            i = np.arange(ps.n)
            assert np.abs(z - M[(i - g * B) % ps.n, (i + b) % R]).max() < 1e-5
    # Horner equals the sum of separately rotated partial sums (after decryption)
    total = np.zeros(ps.n, dtype=complex)
    for g in range(ps.G):
        total += np.roll(o.decrypt_slots(km.s, inner[g], 2 * ps.log_scale), -g * B)
    assert np.abs(total - got).max() < 2e-5


# ------------------------------------------------------------------ giant steps, second order of evaluation (lazy)


def test_key_product_then_moddown_is_the_key_switch():
    """orc_ks_accumulate repeats the inner product of orc_keyswitch: followed by ModDown it must give the same bits"""
    ps = synth.small_params(7, 8, 4, L=3, big=True)
    o = make(ps)
    km = synth.key_material(ps, 23)
    rng = np.random.default_rng(4)
    evk = o.evk_gen(km.s, 2, km.evk_a[1], km.evk_e[1])
    d = np.stack([rand_poly(rng, ps.N, q) for q in ps.q])
    u0, u1 = o.ks_accumulate(d, evk)
    ks0, ks1 = o.keyswitch(d, evk)
    assert np.array_equal(o.moddown(u0), ks0) and np.array_equal(o.moddown(u1), ks1)
    # and it accumulates: a second product lands on top of the first
    d2 = np.stack([rand_poly(rng, ps.N, q) for q in ps.q])
    v0, v1 = o.ks_accumulate(d2, evk)
    w0, w1 = o.ks_accumulate(d2, evk, u0.copy(), u1.copy())
    mods = np.array(list(ps.q) + [ps.p], dtype=object)[:, None]
    assert np.array_equal(w0.astype(object), (u0.astype(object) + v0.astype(object)) % mods)
    assert np.array_equal(w1.astype(object), (u1.astype(object) + v1.astype(object)) % mods)


@pytest.mark.parametrize("big", [False, True])
def test_lazy_giant_steps_error_within_analytic_bound(big):
    """sum_g rot_{gB}(inner[g]) with distinct keys and one ModDown: the decryption of the result minus the exactly rotated
    decryptions of the terms (python integers, explicit coefficient map) is the key-switch error of G-1 key products and
    ONE rounding: variance (G-1) L N sigma^2 q^2 / (12 p^2) + N/18.  Horner on the same terms rounds G-1 times: its
    error is measurably larger where the rounding term dominates (50-bit primes under a 60-bit special prime)."""
    ps = synth.small_params(8, 16, 4, L=2, big=big)
    o = make(ps)
    G, B, N, Q = ps.G, ps.B, ps.N, 1
    for q in ps.q:
        Q *= q
    km = synth.key_material(ps, 27, rots=[g * B for g in range(1, G)])
    evk = all_keys(o, km)
    rng = np.random.default_rng(8)
    inner = np.stack([np.stack([np.stack([rand_poly(rng, N, q) for q in ps.q]) for _ in range(2)]) for _ in range(G)])
    want = np.zeros(N, dtype=object)
    for g in range(G):
        dg = o.decrypt_int(km.s, inner[g])
        k = o.galois(g * B)
        rot = np.zeros(N, dtype=object)
        for i in range(N):
            e = (i * k) % (2 * N)
            if e < N:
                rot[e] = int(dg[i])
            else:
                rot[e - N] = -int(dg[i])
        want = want + rot

    def error_of(ct):
        got = o.decrypt_int(km.s, ct)
        return np.array([float(((int(a) - int(b) + Q // 2) % Q) - Q // 2) for a, b in zip(got, want)])

    err = error_of(o.rotate_sum_lazy(inner, evk))
    qmean = float(np.mean([float(x) for x in ps.q]))
    key_var = ps.L * N * 3.2 ** 2 * qmean ** 2 / (12 * float(ps.p) ** 2)
    std = math.sqrt((G - 1) * key_var + N / 18.0)
    assert abs(err.mean()) < 0.5 * std and 0.7 * std < err.std() < 1.3 * std and np.abs(err).max() < 6 * std
    # Horner with the single key of rotation B on the same terms: G-1 roundings
    err_h = error_of(o.rotate_sum(inner, evk[0]))
    std_h = math.sqrt((G - 1) * (key_var + N / 18.0))
    assert 0.7 * std_h < err_h.std() < 1.3 * std_h
    if big:
        assert err_h.std() > 1.3 * err.std()


@pytest.mark.parametrize("logN,R,B", [(5, 4, 2), (6, 8, 2), (6, 4, 1), (6, 4, 4)])
def test_lazy_giant_steps_without_noise_equal_plain_matvec(logN, R, B):
    ps = synth.small_params(logN, R, B, L=2)
    o = make(ps)
    rots = sorted(set(range(1, B)) | {g * B for g in range(1, ps.G)})
    km = synth.key_material(ps, 41, rots=rots, zero_noise=True)
    evk = dict(zip(rots, all_keys(o, km)))
    rows = synth.toy_corpus(3, rows=ps.n - 3, dim=R)
    qv = synth.toy_query(4, dim=R)
    ct = o.encrypt_query(km.s, qv, km.ct_a, km.ct_e)
    baby = o.baby_set(ct, np.stack([evk[r] for r in range(1, B)]) if B > 1 else np.zeros((0, ps.L, 2, ps.L + 1, ps.N), dtype=np.uint64))
    inner = o.mac(o.encode_block(rows), baby)
    giant = np.stack([evk[g * B] for g in range(1, ps.G)]) if ps.G > 1 else np.zeros((0, ps.L, 2, ps.L + 1, ps.N), dtype=np.uint64)
    score = o.rotate_sum_lazy(inner, giant)
    got = o.decrypt_slots(km.s, score, 2 * ps.log_scale)
    want = np.zeros(ps.n)
    want[: ps.n - 3] = rows.astype(np.float64) @ qv.astype(np.float64)
    assert np.abs(got.real - want).max() < 2e-5 and np.abs(got.imag).max() < 2e-5
    if ps.G == 1:
        assert np.array_equal(score, inner[0])


# ------------------------------------------------------------------ packed projection (Sec. 3.1 Detail)


@pytest.mark.parametrize("D,R,B", [(16, 16, 4), (32, 16, 4), (64, 16, 2), (64, 16, 16), (64, 8, 1), (128, 32, 8)])
def test_packed_projection_on_plain_slots_is_the_matrix_product(D, R, B):
    """the index formulas alone, no encryption: packed diagonals, in-window rotations from two slot rotations and 0/1
    masks, giant steps by plain slot rotations, ONE final fold -> every slot i holds (W^T q)[i mod R]"""
    pp = PackedProjection(9, synth.Q50, synth.P60, 40, D, R, B, 50, 50)
    rng = np.random.default_rng(D + R + B)
    W, qv = rng.standard_normal((D, R)), rng.standard_normal(D)
    got, unfolded = pp.plain(W, qv)
    want = np.tile(W.T @ qv, pp.n // R)
    assert np.abs(got - want).max() < 1e-12
    lo, hi = pp.masks()
    assert np.array_equal(lo + hi, np.ones_like(lo)) and set(np.unique(lo)) <= {0.0, 1.0}
    # masks + two slot rotations = rotation inside every window of R slots
    x = pp.query_slots(qv)
    for b in range(B):
        inwin = np.roll(x.reshape(-1, R), -b, axis=1).reshape(-1)
        assert np.array_equal(lo[b] * np.roll(x, -b) + hi[b] * np.roll(x, -(b - R)), inwin)
    if D > R and B < R:
        # before the fold a window holds a mix of chunk products, not the answer: the fold is what makes it right, and it
        # is needed once only (folding commutes with the slot rotations of the giant steps)
        assert np.abs(unfolded - want).max() > 1e-3
        assert np.abs(sum(np.roll(unfolded, -k * R) for k in range(D // R)) - want).max() < 1e-12


def test_keys_of_a_shorter_chain_are_a_restriction_of_the_longer_chain_keys():
    ps = synth.small_params(7, 8, 4, L=4, big=True)
    km = synth.key_material(ps, 12, rots=[3])
    full = make(ps).evk_gen(km.s, 3, km.evk_a[0], km.evk_e[0])
    for Lt in (3, 2):
        short = Oracle(ps.logN, ps.q[:Lt], ps.p, ps.log_scale, ps.R, ps.B)
        limbs = list(range(Lt)) + [ps.L]
        want = short.evk_gen(km.s, 3, km.evk_a[0][:Lt][:, limbs], km.evk_e[0][:Lt])
        assert np.array_equal(restrict_keys(full, ps.L, Lt), want)


@pytest.mark.parametrize("logN,D,R,B,lazy", [(9, 64, 16, 4, False), (10, 128, 32, 4, True), (9, 32, 32, 8, False)])
def test_packed_projection_under_encryption(logN, D, R, B, lazy):
    """the encrypted pipeline at production primes (4 x 50 bits + 60, scale 2^40, masks and matrix at 2^50): the result
    decrypts, at its exact scale Delta 2^50/q_3 2^50/q_2, to the float64 W^T q tiled over the slots within 2^-20, on the
    chain of L - 2 primes; it equals the UNPACKED projection (one D-diagonal block through the ordinary scorer) within
    the same tolerance."""
    pp = PackedProjection(logN, synth.Q50, synth.P60, 40, D, R, B, 50, 50)
    top = pp.top
    rots = sorted(set(pp.baby_rotations()) | {g * B for g in range(1, pp.G)} | set(pp.fold_rotations()))
    ps = synth.ParamSet("pp", logN, synth.Q50, synth.P60, 40, R, B, -18)
    km = synth.key_material(ps, 61, rots=rots)
    evk = dict(zip(rots, all_keys(top, km)))
    rng = np.random.default_rng(5)
    W = np.linalg.qr(rng.standard_normal((D, R)))[0]
    qv = rng.standard_normal(D)
    qv = (qv / np.linalg.norm(qv)).astype(np.float32)
    ct = top.encrypt(km.s, top.encode(pp.query_slots(qv)), km.ct_a, km.ct_e)
    out = pp.project(ct, evk, pp.enrol(W), lazy=lazy)
    assert out.shape == (2, 2, pp.N)
    mu = pp.low.decrypt_int(km.s, out)
    slots = pp.low.decode(np.array([float(v) for v in mu]), pp.scale_out)
    want = np.tile(W.T.astype(np.float64) @ qv.astype(np.float64), pp.n // R)
    assert np.abs(slots.real - want).max() < 2.0 ** -20 and np.abs(slots.imag).max() < 2.0 ** -20
    assert abs(pp.scale_out / 2.0 ** 40 - 1.0) < 2.0 ** -20          # the two rescales bring the scale back to ~Delta
    # the unpacked projection: W^T tiled down the slots as one block of D diagonals, ordinary scorer (R = D)
    ub = min(B, D)
    un = Oracle(logN, synth.Q50, synth.P60, 40, D, ub)
    kmu = synth.key_material(synth.ParamSet("un", logN, synth.Q50, synth.P60, 40, D, ub, -18), 61)
    evu = all_keys(un, kmu)
    block = np.tile(W.T.astype(np.float32), (pp.n // R, 1))
    ctu = un.encrypt_query(kmu.s, qv, kmu.ct_a, kmu.ct_e)
    sc, _, _ = un.score_block(block, un.baby_set(ctu, evu), evu[ub - 1])
    plain = un.decrypt_slots(kmu.s, sc, 80).real
    assert np.abs(plain - slots.real).max() < 2.0 ** -19


def test_zero_padding_96_to_128_is_exact():
    # Sec. 4 (datasets): zero-padding 96 -> 128 dimensions changes no dot product
    x = synth.toy_corpus(8, rows=50, dim=96).astype(np.float64)
    qv = synth.toy_query(9, dim=96).astype(np.float64)
    xp = np.zeros((50, 128)); xp[:, :96] = x
    qp = np.zeros(128); qp[:96] = qv
    a = np.array([sum(x[i, d] * qv[d] for d in range(96)) for i in range(50)])
    b = np.array([sum(xp[i, d] * qp[d] for d in range(128)) for i in range(50)])
    assert np.array_equal(a, b)
    # the padded coordinates occupy exact zeros in the slot vectors that get encoded: a block whose rows are all
    # zero beyond dimension 96 has, on diagonal b, zero slots wherever (i + b) mod 128 >= 96
    ps = synth.small_params(9, 128, 32, L=2)
    o = make(ps)
    pt = o.encode_block(synth.project_rows(x.astype(np.float32), None, 128))
    q0 = ps.q[0]
    for b in (0, 31):
        cent = np.array([int(v) if int(v) <= q0 // 2 else int(v) - q0 for v in pt[0, b, 0]], dtype=np.float64)
        z = o.decode(cent, 2.0 ** ps.log_scale).real
        i = np.arange(ps.n)
        assert np.abs(z[(i + b) % 128 >= 96]).max() < 1e-5


def test_toy_configuration_scores_within_tolerance():
    """Toy configuration: N = 2^12, two ~30-bit primes + one ~31-bit special prime, scale 2^25, 4,096 unit-norm
    rows of dimension 64 -> two blocks; decrypted scores within 2^-10 of the float64 dot products."""
    ps = synth.TOY
    o = make(ps)
    km = synth.key_material(ps, 3)
    rows = synth.toy_corpus(1)
    qv = synth.toy_query(2)
    ct = o.encrypt_query(km.s, qv, km.ct_a, km.ct_e)
    evk = all_keys(o, km)
    baby = o.baby_set(ct, evk)
    worst = 0.0
    for blk in range(2):
        sc, _, _ = o.score_block(rows[blk * ps.n:(blk + 1) * ps.n], baby, evk[ps.B - 1])
        got = o.decrypt_slots(km.s, sc, 2 * ps.log_scale)
        want = rows[blk * ps.n:(blk + 1) * ps.n].astype(np.float64) @ qv.astype(np.float64)
        worst = max(worst, np.abs(got.real - want).max())
        assert np.abs(got.imag).max() < 2.0 ** ps.tol_log2
    assert worst < 2.0 ** ps.tol_log2
    assert worst < 4 * 2.0 ** -12.2  # regression alarm: observed error level of this parameter set
    # baby rotations taken directly from the query: each decrypts to the rotated tiled query
    z = np.tile(np.pad(qv, (0, ps.R - len(qv))).astype(np.float64), ps.n // ps.R)
    for r in (1, ps.B - 1):
        back = o.decrypt_slots(km.s, baby[r], ps.log_scale).real
        assert np.abs(back - np.roll(z, -r)).max() < 1e-3


def test_full_size_primes_scores_within_tolerance_small_ring():
    """The production primes (4 x ~50 bit + ~60 bit, scale 2^40) on a reduced ring: tolerance 2^-18."""
    ps = synth.ParamSet("n11", 11, synth.Q50, synth.P60, 40, 128, 32, -18)
    o = make(ps)
    km = synth.key_material(ps, 5)
    rows = synth.project_rows(synth.toy_corpus(1, rows=ps.n - 100, dim=96).astype(np.float64), None, 128)
    qv = np.zeros(128, dtype=np.float32); qv[:96] = synth.toy_query(2, dim=96)
    ct = o.encrypt_query(km.s, qv, km.ct_a, km.ct_e)
    evk = all_keys(o, km)
    baby = o.baby_set(ct, evk)
    sc, _, _ = o.score_block(rows, baby, evk[ps.B - 1])
    got = o.decrypt_slots(km.s, sc, 2 * ps.log_scale)
    want = np.zeros(ps.n); want[: ps.n - 100] = rows.astype(np.float64) @ qv.astype(np.float64)
    assert np.abs(got.real - want).max() < 2.0 ** -18
    assert np.abs(got.real - want).max() < 2.0 ** -24
    assert np.abs(got.imag).max() < 2.0 ** -18


# ------------------------------------------------------------------ output compaction (rescale + limb drop)


def test_compaction_is_exact_division_of_the_crt_integer():
    """Big-integer pin: with C the centred CRT integer of a polynomial over q_0..q_{L-1} and r the centred residue
    mod q_{L-1}, the kept limbs must hold (C - r) / q_{L-1} (an exact division), i.e. C / q_{L-1} rounded to nearest."""
    ps = synth.small_params(5, 4, 2, L=3, big=True)
    o = make(ps)
    rng = np.random.default_rng(11)
    ct = np.stack([np.stack([rand_poly(rng, ps.N, q) for q in ps.q]) for _ in range(2)])
    ql = ps.q[-1]
    for keep in (1, 2):
        out = o.compact(ct, keep)
        assert np.array_equal(o.compact(ct, keep, rescale=False), ct[:, :keep])
        for poly in range(2):
            C = [int(v) for v in o.crt_centred(ct[poly])]
            for x in range(ps.N):
                r = C[x] % ql
                if r > ql // 2:
                    r -= ql
                assert (C[x] - r) % ql == 0
                want = (C[x] - r) // ql
                assert abs(want * ql - C[x]) <= ql // 2            # nearest multiple
                for i in range(keep):
                    assert int(out[poly, i, x]) == want % ps.q[i]


def test_compacted_scores_decrypt_to_the_same_scores():
    """Production primes on a reduced ring.  Dropping to two limbs is exact (identical centred integers); a rescale to
    one limb (scale 2^80 / q_3 ~ 2^30) adds the rounding error of the division: inside the Laplace-tail bound of its analytic size (see helpers) and,
    on this ring, still inside 2^-18."""
    ps = synth.ParamSet("n11", 11, synth.Q50, synth.P60, 40, 128, 32, -18)
    o = make(ps)
    km = synth.key_material(ps, 5)
    rows = synth.project_rows(synth.toy_corpus(1, rows=ps.n - 100, dim=96).astype(np.float64), None, 128)
    qv = np.zeros(128, dtype=np.float32); qv[:96] = synth.toy_query(2, dim=96)
    ct = o.encrypt_query(km.s, qv, km.ct_a, km.ct_e)
    evk = all_keys(o, km)
    sc, _, _ = o.score_block(rows, o.baby_set(ct, evk), evk[ps.B - 1])
    want = np.zeros(ps.n); want[: ps.n - 100] = rows.astype(np.float64) @ qv.astype(np.float64)
    full_int = o.decrypt_int(km.s, sc)
    full = o.decrypt_slots(km.s, sc, 2 * ps.log_scale)
    two = o.compact(sc, 2, rescale=False)
    assert np.array_equal(two, sc[:, :2])
    assert list(o.decrypt_compact_int(km.s, two)) == list(full_int)          # the same integers from half the limbs
    sigma = rescale_error_sigma(ps.N, 2.0 ** 80 / ps.q[-1])
    for keep in (1, 3):
        small = o.compact(sc, keep)
        assert small.shape == (2, keep, ps.N)
        got = o.decrypt_compact_slots(km.s, small, 2 * ps.log_scale)
        assert np.abs(got.real - full.real).max() < rescale_error_bound(ps.N, 2.0 ** 80 / ps.q[-1], ps.n)
        assert np.abs(got.real - full.real).std() > sigma / 3                # and the error really is of that size
        assert np.abs(got.real - want).max() < 2.0 ** -18
        assert np.abs(got.imag).max() < 2.0 ** -18
    # toy primes: only 2^50 / q_1 ~ 2^20 of scale is left on the one ~30-bit limb, so the rounding error of the
    # division (sigma ~ 2^-10.5) exceeds the scoring tolerance: the toy set has no room for a rescale
    ps = synth.TOY
    o = make(ps)
    km = synth.key_material(ps, 3)
    rows = synth.toy_corpus(1, rows=ps.n)
    qv = synth.toy_query(2)
    ct = o.encrypt_query(km.s, qv, km.ct_a, km.ct_e)
    evk = all_keys(o, km)
    sc, _, _ = o.score_block(rows, o.baby_set(ct, evk), evk[ps.B - 1])
    got = o.decrypt_compact_slots(km.s, o.compact(sc, 1), 2 * ps.log_scale)
    sigma = rescale_error_sigma(ps.N, 2.0 ** 50 / ps.q[-1])
    err = np.abs(got.real - o.decrypt_slots(km.s, sc, 2 * ps.log_scale).real)
    assert sigma / 3 < err.std() and err.max() < rescale_error_bound(ps.N, 2.0 ** 50 / ps.q[-1], ps.n)


# ------------------------------------------------------------------ encrypted database: ct x ct, relinearisation


def db_material(ps, seed):
    """uniform a [R][L][N] and small e [R][N] for the symmetric encryption of one block's diagonals"""
    a = synth.uniform_residues(seed, 40, list(ps.q), ps.N, lead=(ps.R,))
    e = synth.rounded_gaussian(seed, 41, (ps.R, ps.N))
    return a, e


def test_ct_times_ct_decrypts_to_the_product_and_relinearises():
    """Degree-2 decryption d0 + d1 s + d2 s^2 of the ct x ct multiply-accumulate, computed here with schoolbook python
    integers, equals sum_b (x0 + x1 s)(y0 + y1 s) limb by limb; relinearisation changes that value by no more than the
    key-switch noise; noise-free everything reproduces the plain matrix-vector product."""
    ps = synth.small_params(5, 4, 2, L=2)
    o = make(ps)
    km = synth.key_material(ps, 9)
    rng = np.random.default_rng(5)
    ctdb = np.stack([np.stack([np.stack([rand_poly(rng, ps.N, q) for q in ps.q]) for _ in range(2)]) for _ in range(ps.R)])
    baby = np.stack([np.stack([np.stack([rand_poly(rng, ps.N, q) for q in ps.q]) for _ in range(2)]) for _ in range(ps.B)])
    d = o.mac_ct(ctdb, baby)
    assert d.shape == (ps.G, 3, ps.L, ps.N)
    s_int = [int(v) for v in km.s]
    for l, q in enumerate(ps.q):
        sq = [v % q for v in s_int]
        s2 = schoolbook_negacyclic(sq, sq, q)
        for g in range(ps.G):
            want = [0] * ps.N
            for b in range(ps.B):
                x = ctdb[g * ps.B + b, :, l]
                y = baby[b, :, l]
                xs = [(int(u) + int(v)) % q for u, v in zip(x[0], schoolbook_negacyclic(x[1], sq, q))]
                ys = [(int(u) + int(v)) % q for u, v in zip(y[0], schoolbook_negacyclic(y[1], sq, q))]
                want = [(u + v) % q for u, v in zip(want, schoolbook_negacyclic(xs, ys, q))]
            got = [(int(a0) + int(a1) + int(a2)) % q for a0, a1, a2 in
                   zip(d[g, 0, l], schoolbook_negacyclic(d[g, 1, l], sq, q), schoolbook_negacyclic(d[g, 2, l], s2, q))]
            assert got == want
    # relinearisation: c0 + c1 s = d0 + d1 s + d2 s^2 + (key-switch error), error within the analytic bound of the key switch
    ka = synth.uniform_residues(77, 50, list(ps.q) + [ps.p], ps.N, lead=(ps.L,))
    ke = synth.rounded_gaussian(77, 51, (ps.L, ps.N))
    rlk = o.rlk_gen(km.s, ka, ke)
    Q = 1
    for q in ps.q:
        Q *= q
    for g in range(ps.G):
        ct = o.relin(d[g], rlk)
        lhs = o.decrypt_int(km.s, ct)
        deg2 = []
        for l, q in enumerate(ps.q):
            sq = [v % q for v in s_int]
            s2 = schoolbook_negacyclic(sq, sq, q)
            deg2.append(np.array([(int(a0) + int(a1) + int(a2)) % q for a0, a1, a2 in
                                  zip(d[g, 0, l], schoolbook_negacyclic(d[g, 1, l], sq, q), schoolbook_negacyclic(d[g, 2, l], s2, q))],
                                 dtype=np.uint64))
        rhs = o.crt_centred(np.stack(deg2))
        err = np.array([float((int(a) - int(b) + Q // 2) % Q - Q // 2) for a, b in zip(lhs, rhs)])
        sigma = math.sqrt(ps.L * ps.N * 3.2 ** 2 * (max(ps.q) / ps.p) ** 2 / 12 + ps.N / 18)
        assert np.abs(err).max() < 8 * sigma and err.std() > sigma / 4


def test_encrypted_database_scores_within_tolerance():
    """toy primes, N = 2^10: diagonals encrypted under the same key, ct x ct multiply-accumulate, relinearisation, the
    unchanged rotate-and-sum: decrypted scores within 2^-10 of the float64 dot products; without noise the result is
    bit-identical to the plaintext-database path"""
    ps = synth.small_params(10, 16, 4, L=2)
    o = make(ps)
    rows = synth.toy_corpus(4, rows=ps.n - 7, dim=16)
    qv = synth.toy_query(5, dim=16)
    for zero in (False, True):
        km = synth.key_material(ps, 3, zero_noise=zero)
        evk = all_keys(o, km)
        ka = synth.uniform_residues(78, 50, list(ps.q) + [ps.p], ps.N, lead=(ps.L,))
        ke = np.zeros((ps.L, ps.N), dtype=np.int8) if zero else synth.rounded_gaussian(78, 51, (ps.L, ps.N))
        rlk = o.rlk_gen(km.s, ka, ke)
        ct = o.encrypt_query(km.s, qv, km.ct_a, km.ct_e)
        baby = o.baby_set(ct, evk)
        pt = o.encode_block(rows)
        a, e = db_material(ps, 21)
        if zero:
            e = np.zeros_like(e)
        ctdb = o.encrypt_block(km.s, pt, a, e)
        # each database ciphertext decrypts to its diagonal plus its error array
        for r in (0, ps.R - 1):
            mu = o.decrypt_residues(km.s, ctdb[r])
            want = (pt.reshape(ps.R, ps.L, ps.N)[r, 0].astype(object) + e[r].astype(object)) % ps.q[0]
            assert [int(v) for v in mu[0]] == [int(v) for v in want]
        d = o.mac_ct(ctdb, baby)
        inner = np.stack([o.relin(d[g], rlk) for g in range(ps.G)])
        score = o.rotate_sum(inner, evk[ps.B - 1])
        got = o.decrypt_slots(km.s, score, 2 * ps.log_scale).real
        want = np.zeros(ps.n); want[: ps.n - 7] = rows.astype(np.float64) @ qv.astype(np.float64)
        assert np.abs(got - want).max() < 2.0 ** ps.tol_log2
        if zero:
            plain = o.rotate_sum(o.mac(pt, baby), evk[ps.B - 1])
            # (c0 + c1 s) agree exactly although the ciphertexts differ: same message, no noise anywhere but the roundings
            # of ModDown, which differ -> compare decrypted integers up to those roundings
            a_int, b_int = o.decrypt_int(km.s, score), o.decrypt_int(km.s, plain)
            assert max(abs(int(x) - int(y)) for x, y in zip(a_int, b_int)) < 64 * ps.N


# ------------------------------------------------------------------ seed-compressed ciphertexts


def test_seed_expansion_matches_the_published_check_values():
    """the counter hash against its four check values h(1, 0, 0..3) and, through them, against the harness generator;
    the expanded polynomial is the harness's uniform residue array"""
    from oracle.oracle import lib

    want = [0xCE6D52A9E69DA903, 0x3C904E4F0D0C01AF, 0x6E6AE58702F2C840, 0xD254BD0790389C63]
    assert [int(lib().orc_hash64(1, 0, i)) for i in range(4)] == want
    assert [int(v) for v in synth.hash64(1, 0, np.arange(4))] == want
    ps = synth.small_params(8, 8, 4, L=2)
    o = make(ps)
    a = o.expand_uniform(123456789, 19)
    assert np.array_equal(a, synth.uniform_residues(123456789, 19, list(ps.q), ps.N))
    assert all(int(a[l].max()) < ps.q[l] for l in range(ps.L))
    # roughly uniform: mean near q/2
    assert abs(float(a[0].astype(np.float64).mean()) / ps.q[0] - 0.5) < 0.1
