"""Pins of the membership (threshold) circuit of the CPU oracle (oracle/membership.py; Sec. 3.1 "The norm problem",
membership bullet, and Sec. 2 "Security parameters": depth 11): the Chebyshev coefficients against numpy's interpolation
routine and against the function itself, the product-identity basis against cos(k arccos u), the sign iteration's
monotonicity, the plain-number circuit against the direct decision score >= tau |q_R|, and the encrypted circuit (12
primes, depth 11) against the plain-number circuit and the direct decision."""
import math

import numpy as np
import pytest

from oracle import membership as mb
from paper_2608_21131_b200 import synth


def test_chebyshev_coefficients_are_the_library_interpolant_and_approximate_the_root():
    tau, lo, hi, deg = 0.4, 0.05, 1.0, 7
    f = lambda t: 0.5 * tau * np.sqrt(t)
    c = mb.chebyshev_coefficients(f, deg, lo, hi)
    ref = np.polynomial.chebyshev.chebinterpolate(lambda u: f(0.5 * (hi - lo) * u + 0.5 * (hi + lo)), deg)
    assert np.abs(c - ref).max() < 1e-13
    t = np.linspace(lo, hi, 2001)
    u = (2 * t - (hi + lo)) / (hi - lo)
    err = np.abs(np.polynomial.chebyshev.chebval(u, c) - f(t)).max()
    assert err < 2e-3 * tau            # a low degree suffices: the root is smooth away from zero
    assert np.abs(np.polynomial.chebyshev.chebval(u, c[:4]) - f(t)).max() > 4 * err   # and the degree matters


@pytest.mark.parametrize("deg", [2, 3, 5, 7, 12])
def test_product_identity_basis_is_the_chebyshev_basis(deg):
    u = np.linspace(-1, 1, 101)
    T = mb.chebyshev_basis(lambda a, b: a * b, lambda a, b: a - b, lambda a: 2.0 * a, lambda a, c: a + c, u, deg)
    for k in range(1, deg + 1):
        assert np.abs(T[k] - np.cos(k * np.arccos(u))).max() < 1e-12
    # depth of T_k under the identity: ceil(log2 k) products
    depth = {1: 0}
    for k in range(2, deg + 1):
        m = (k + 1) // 2
        depth[k] = max(depth[m], depth[k - m]) + 1
        assert depth[k] == math.ceil(math.log2(k))


def test_sign_iteration_keeps_the_sign_and_amplifies():
    x = np.linspace(-1, 1, 4001)
    y = x.copy()
    for _ in range(3):
        y = y * (3 - y * y) / 2
    assert np.all(np.sign(y) == np.sign(x)) and np.all(np.abs(y) <= 1 + 1e-12)
    assert np.all(np.diff(y) >= -1e-15)                         # monotone on [-1, 1]
    assert np.all(np.abs(y[np.abs(x) >= 0.05]) >= 3.3 * 0.05)   # slope 27/8 at the origin
    assert np.all(np.abs(y[np.abs(x) >= 0.5]) > 0.97)            # f(f(f(0.5))) = 0.975


def unit_rows(seed, rows, R):
    return synth.toy_corpus(seed, rows=rows, dim=R)


def test_plain_circuit_decides_like_the_direct_comparison():
    R, tau = 16, 0.45
    m = mb.Membership(9, R, tau)
    assert m.depth == 11 and m.L == 12
    rows = unit_rows(3, 256, R)
    rng = np.random.default_rng(1)
    for norm in (0.3, 0.6, 0.95):
        qR = rows[7] + 0.2 * rng.standard_normal(R)
        qR = (norm * qR / np.linalg.norm(qR)).astype(np.float32)
        out = m.plain(rows, qR)
        direct = rows.astype(np.float64) @ qR.astype(np.float64) - tau * np.linalg.norm(qR.astype(np.float64))
        assert abs(out["r"] - 0.5 * tau * np.linalg.norm(qR)) < 1e-3 * tau
        clear = np.abs(direct) > 4e-3 * tau                     # outside the polynomial's approximation error
        assert np.array_equal(np.sign(out["out"][clear]), np.sign(direct[clear]))
        assert out["out"][7] > 0                                 # the planted row matches


def test_encrypted_circuit_depth_eleven_matches_the_plain_circuit():
    logN, R, tau = 10, 16, 0.45
    m = mb.Membership(logN, R, tau)
    ev = m.ev
    q, p, L = ev.q, ev.p, ev.L
    ps = synth.ParamSet("mem", logN, tuple(q), p, 45, R, 1, -10)
    rots = sorted(set(m.score_rotations()) | set(m.fold_rotations()))
    km = synth.key_material(ps, 31, rots=rots)
    top = ev.o[L]
    rot_keys = {r: top.evk_gen(km.s, r, km.evk_a[i], km.evk_e[i]) for i, r in enumerate(rots)}
    ka = synth.uniform_residues(31, 50, list(q) + [p], ps.N, lead=(L,))
    ke = synth.rounded_gaussian(31, 51, (L, ps.N))
    ev.set_keys(top.rlk_gen(km.s, ka, ke), rot_keys)
    rows = unit_rows(3, ps.n - 40, R)
    rng = np.random.default_rng(2)
    qR = rows[11] + 0.25 * rng.standard_normal(R)
    qR = (0.7 * qR / np.linalg.norm(qR)).astype(np.float32)
    ct = mb.Ct(top.encrypt(km.s, top.encode(m.query_slots(qR), 45), km.ct_a, km.ct_e), 2.0 ** 45)
    want = m.plain(rows, qR)
    # the threshold alone: tau kappa |q_R| in every slot, five levels down
    thr = m.threshold(ct)
    assert thr.level == L - 5
    got_thr = ev.decrypt(km.s, thr).real
    assert np.abs(got_thr - want["r"]).max() < 1e-5
    out = m.decide(ct, rows)
    assert m.levels == {"threshold": L - 5, "score": L - 5, "out": 1}          # depth 11 on 12 primes
    assert abs(math.log2(out.scale) - 45) < 0.01 and ev.worst_scale_mismatch < 2.0 ** -15
    got = ev.decrypt(km.s, out).real[: rows.shape[0]]
    assert np.abs(got - want["out"]).max() < 1e-4
    direct = rows.astype(np.float64) @ qR.astype(np.float64) - tau * np.linalg.norm(qR.astype(np.float64))
    clear = np.abs(direct) > 4e-3 * tau
    assert np.array_equal(np.sign(got[clear]), np.sign(direct[clear])) and got[11] > 0.2
    assert clear.mean() > 0.9
