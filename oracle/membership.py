"""Membership (threshold) path of the face task, as a plain leveled CKKS circuit over the CPU oracle's primitives.

TEST INFRASTRUCTURE ONLY (see oracle.py).  Sec. 3.1, "The norm problem", membership bullet: the server must return a
match / no-match decision under encryption, so it cannot let the client divide by |q_R|.  It compares the raw score
<x, q_R> with the threshold scaled into the query's units, tau |q_R| = sqrt(tau^2 |q_R|^2), the square root taken by a
LOW-DEGREE Chebyshev polynomial evaluated directly (no Paterson-Stockmeyer), everything pre-scaled into [-1, 1] by
plaintext constants, then evaluates sign(score - tau |q_R|).  Sec. 2, "Security parameters": this path runs at
multiplicative depth 11 (the ranked path at 4).

Reading taken (the paper names the ingredients, not the circuit):
  1. t = |q_R|^2 in every slot: one ciphertext x ciphertext product of the tiled query with itself, relinearised and
     rescaled, then a fold over the R slots of a period (log2 R slot rotations).                               depth 1
  2. u = (2 t - (t_hi + t_lo)) / (t_hi - t_lo) in [-1, 1] for t in [t_lo, t_hi]: an affine map; its factor is absorbed by
     the client (it encodes lam q_R, lam^2 = a q_{L-1} / Delta, so that the rescaled product read at scale Delta holds
     a t), its offset is a constant added to the first coefficient limb-wise.                                   depth 0
  3. r = (kappa tau) sqrt(t) ~ sum_k c_k T_k(u), degree DEG: T_k by the product identity T_{m+n} = 2 T_m T_n - T_{m-n} with
     m = ceil(k/2) (depth ceil(log2 k)), then one integer-constant multiply per term that also brings all terms to one
     common scale (depth 1).                                                                                    depth 4 at degree 7
  4. s = kappa <x, q_R> for every candidate: the ordinary diagonal scorer on the same chain, entered at the level that
     makes it end where r ends (dropping primes of a fresh ciphertext is exact); kappa = 1/2 keeps d = s - r in [-1, 1]
     and is folded into the candidates' plaintexts and the c_k ("pre-scale into [-1,1] with a plaintext constant, which
     also saves one multiplication").                                                                           depth 1, in parallel
  5. sign(d) ~ f(f(f(d))), f(x) = x (3 - x^2) / 2: x^2 costs a level, x (3 - x^2) another; the division by two is the
     rescale of that second product by a prime of TWICE the scale, so every ciphertext stays at ~2^45.          depth 6
Total depth 5 + 6 = 11: the norm recovery and the sign check share one budget, as the paper says.  The client decrypts a
value whose SIGN is the decision; for |d| above the noise it is amplified towards +-1.

Chain: q_0 a ~58-bit prime (the last level must hold a value of magnitude ~1 at scale 2^45), then primes just below 2^45
(the paper's 45-bit scale: a rescale by such a prime returns the scale to ~2^45) and, for the three halvings of the sign
stage, just below 2^46; one ~60-bit special prime; L = 12 ("L ~ 12").
"""
from __future__ import annotations

import math

import numpy as np

from .oracle import Oracle, find_primes, restrict_keys


def membership_chain(logN, deg=7, sign_iters=3, log_scale=45):
    """(q, p) for the circuit below.  Levels are consumed from the last prime down: |q_R|^2 (one prime ~2^log_scale), the
    Chebyshev basis (ceil(log2 deg) primes), the combination (one), then per sign iteration one prime ~2^log_scale (for x^2)
    and one ~2^(log_scale + 1) (for x w: the rescale by TWICE the scale is the division by two of f(x) = x (3 - x^2) / 2,
    so the scale stays put); q_0 is the largest prime below 2^58, the special prime the largest below 2^60; all 1 mod 2N."""
    step = logN + 1
    n_thr = 1 + math.ceil(math.log2(deg)) + 1
    p45, p46 = find_primes(log_scale, step, n_thr + sign_iters), find_primes(log_scale + 1, step, sign_iters)
    consumed = p45[:n_thr]                                    # in the order the circuit consumes them
    for i in range(sign_iters):
        consumed += [p45[n_thr + i], p46[i]]                  # x^2 over a prime ~Delta, x (3 - x^2) over one ~2 Delta
    q = find_primes(58, step, 1) + consumed[::-1]            # a rescale always removes the LAST prime of the chain
    return q, find_primes(60, step, 1)[0]


class Ct:
    """a ciphertext on the first `level` primes, read at `scale`"""

    def __init__(self, res, scale):
        self.res, self.scale = np.ascontiguousarray(res, dtype=np.uint64), float(scale)

    @property
    def level(self):
        return self.res.shape[1]


class Evaluator:
    """leveled arithmetic on Ct over one chain; every level has its own oracle context (R = B = 1)"""

    def __init__(self, logN, q, p, log_scale):
        self.logN, self.q, self.p, self.L, self.log_scale = logN, [int(x) for x in q], int(p), len(q), log_scale
        self.o = {l: Oracle(logN, self.q[:l], p, log_scale, 1, 1) for l in range(1, self.L + 1)}
        self.N, self.n = 1 << logN, 1 << (logN - 1)
        self.worst_scale_mismatch = 0.0

    # ---- keys: generated once on the full chain, restricted per level
    def set_keys(self, rlk, rot_keys):
        self.rlk, self.rot_keys = rlk, dict(rot_keys)

    def _key(self, key, level):
        return restrict_keys(key, self.L, level)

    # ---- level and scale management
    def drop(self, a, level):
        """exact: c0 + c1 s is the same integer modulo the shorter product while it is small against it"""
        assert level <= a.level
        return Ct(a.res[:, :level], a.scale)

    def _align(self, a, b):
        l = min(a.level, b.level)
        a, b = self.drop(a, l), self.drop(b, l)
        self.worst_scale_mismatch = max(self.worst_scale_mismatch, abs(a.scale / b.scale - 1.0))
        return a, b

    def _mods(self, level):
        return np.array(self.q[:level], dtype=object).reshape(1, level, 1)

    def add(self, a, b, sign=1):
        a, b = self._align(a, b)
        r = (a.res.astype(object) + sign * b.res.astype(object)) % self._mods(a.level)
        return Ct(r.astype(np.uint64), a.scale)

    def sub(self, a, b):
        return self.add(a, b, -1)

    def neg(self, a):
        return Ct(((-a.res.astype(object)) % self._mods(a.level)).astype(np.uint64), a.scale)

    def add_const(self, a, c):
        """value + c in every slot: the constant polynomial rint(c scale) added to c0"""
        m = int(round(c * a.scale))
        r = a.res.astype(object)
        r[0, :, 0] = (r[0, :, 0] + m) % np.array(self.q[:a.level], dtype=object)
        return Ct(r.astype(np.uint64), a.scale)

    def rescale(self, a):
        o = self.o[a.level]
        return Ct(o.compact(a.res, a.level - 1, rescale=True), a.scale / self.q[a.level - 1])

    def mul(self, a, b):
        """ciphertext x ciphertext: degree-2 product, relinearisation, rescale"""
        a, b = self._align(a, b)
        o = self.o[a.level]
        d = o.mac_ct(a.res[None], b.res[None])[0]
        return self.rescale(Ct(o.relin(d, self._key(self.rlk, a.level)), a.scale * b.scale))

    def mul_int(self, a, m):
        """times the integer m (every residue times m), no rescale"""
        r = (a.res.astype(object) * int(m)) % self._mods(a.level)
        return Ct(r.astype(np.uint64), a.scale)

    def to_scale(self, a, factor, target_scale):
        """factor * value at exactly `target_scale` one level down: integer-constant multiply, then rescale"""
        m = int(round(factor * target_scale * self.q[a.level - 1] / a.scale))
        out = self.rescale(self.mul_int(a, m))
        return Ct(out.res, a.scale * m / self.q[a.level - 1] / factor) if factor != 0 else out

    def mul_plain(self, a, z, log_scale):
        o = self.o[a.level]
        return self.rescale(Ct(o.mul_plain_acc(a.res, o.encode_plain(z, log_scale)), a.scale * 2.0 ** log_scale))

    def rotate(self, a, r):
        return Ct(self.o[a.level].rotate(a.res, r, self._key(self.rot_keys[r], a.level)), a.scale)

    def decrypt(self, s, a):
        o = self.o[a.level]
        return o.decode(np.array([float(v) for v in o.decrypt_int(s, a.res)]), a.scale)


def chebyshev_coefficients(f, deg, lo, hi):
    """coefficients c_0..c_deg of the degree-deg Chebyshev interpolant of f on [lo, hi] at the Chebyshev nodes"""
    k = np.arange(deg + 1)
    nodes = np.cos(np.pi * (k + 0.5) / (deg + 1))
    vals = f(0.5 * (hi - lo) * nodes + 0.5 * (hi + lo))
    c = np.array([2.0 / (deg + 1) * np.sum(vals * np.cos(np.pi * j * (k + 0.5) / (deg + 1))) for j in range(deg + 1)])
    c[0] *= 0.5
    return c


def chebyshev_basis(mul, sub_, twice, add_const, u, deg):
    """T_1..T_deg of u by the product identity T_{m+n} = 2 T_m T_n - T_{m-n}, m = ceil(k/2): depth ceil(log2 k).  The four
    callables are the arithmetic (ciphertexts or plain numbers), so the same code serves the pin on plain floats."""
    T = {1: u}
    for k in range(2, deg + 1):
        m = (k + 1) // 2
        nn = k - m
        prod2 = twice(mul(T[m], T[nn]))
        T[k] = add_const(prod2, -1.0) if m == nn else sub_(prod2, T[m - nn])
    return T


class Membership:
    """one parameter set of the membership path: ring, chain, rank R, threshold tau, range of |q_R|^2, polynomial degree"""

    def __init__(self, logN, R, tau, t_lo=0.05, t_hi=1.0, deg=7, sign_iters=3, log_scale=45, B=None):
        q, p = membership_chain(logN, deg, sign_iters, log_scale)
        self.ev = Evaluator(logN, q, p, log_scale)
        self.R, self.tau, self.t_lo, self.t_hi, self.deg, self.sign_iters = R, tau, t_lo, t_hi, deg, sign_iters
        self.B = B if B else max(1, 1 << ((R.bit_length() - 1) // 2))       # baby steps of the scorer
        self.kappa = 0.5
        self.n, self.N, self.L, self.log_scale = self.ev.n, self.ev.N, len(q), log_scale
        self.coef = chebyshev_coefficients(lambda t: self.kappa * tau * np.sqrt(t), deg, t_lo, t_hi)
        self.depth_threshold = 1 + math.ceil(math.log2(deg)) + 1
        self.depth = self.depth_threshold + 2 * sign_iters
        assert self.L == self.depth + 1
        # The affine map u = a t + b, a = 2 / (t_hi - t_lo), costs nothing if the CLIENT encodes lam * q_R with
        # lam^2 = a q_{L-1} / Delta: the product of that ciphertext with itself, rescaled by q_{L-1}, read at scale Delta,
        # holds a t.  The scorer's plaintexts carry the factor kappa / lam in exchange.
        self.a = 2.0 / (t_hi - t_lo)
        self.lam = math.sqrt(self.a * q[-1] / 2.0 ** log_scale)

    def query_slots(self, qR):
        """what the client encodes (at scale 2^log_scale): lam * q_R, tiled with period R"""
        v = np.zeros(self.R)
        v[: len(qR)] = np.asarray(qR, dtype=np.float64)
        return np.tile(self.lam * v, self.n // self.R)

    def fold_rotations(self):
        return [1 << t for t in range(self.R.bit_length() - 1)]

    # ---- the same circuit on plain numbers (what the encrypted one must reproduce)
    def plain(self, rows, qR):
        t = float(np.dot(qR, qR))
        u = (2.0 * t - (self.t_hi + self.t_lo)) / (self.t_hi - self.t_lo)
        T = chebyshev_basis(lambda a, b: a * b, lambda a, b: a - b, lambda a: 2.0 * a, lambda a, c: a + c, u, self.deg)
        r = self.coef[0] + sum(self.coef[k] * T[k] for k in range(1, self.deg + 1))
        d = self.lam * (self.scaled_rows(rows).astype(np.float64) @ qR.astype(np.float64)) - r
        x = d
        for _ in range(self.sign_iters):
            x = x * (1.5 - 0.5 * x * x)
        return {"t": t, "u": u, "r": r, "d": d, "out": x}

    # ---- under encryption
    def threshold(self, ct_q):
        """Ct of r = kappa tau sqrt(|q_R|^2) (approximately) in every slot; ct_q: the tiled query on the full chain"""
        ev = self.ev
        t = ev.mul(ct_q, ct_q)                                   # lam^2 q_d^2 in slot d
        for r in self.fold_rotations():
            t = ev.add(t, ev.rotate(t, r))                       # lam^2 |q_R|^2 in every slot
        # read at scale Delta it is a t (see __init__); the rescale left it at Delta^2 / q_{L-1} = Delta lam^2 / a ... exactly
        t = Ct(t.res, t.scale / (self.lam * self.lam) * self.a)
        u = ev.add_const(t, -(self.t_hi + self.t_lo) / (self.t_hi - self.t_lo))
        T = chebyshev_basis(ev.mul, ev.sub, lambda x: ev.mul_int(x, 2), ev.add_const, u, self.deg)
        level = min(T[k].level for k in T) - 1
        target = 2.0 ** self.log_scale
        acc = None
        for k in range(1, self.deg + 1):
            if abs(self.coef[k]) < 1e-15:
                continue
            term = ev.to_scale(ev.drop(T[k], level + 1), float(self.coef[k]), target)
            acc = term if acc is None else ev.add(acc, term)
        return ev.add_const(acc, float(self.coef[0]))

    def score_rotations(self):
        """slot rotations the scorer needs: the baby steps and the Horner rotation"""
        return list(range(1, self.B + 1))

    def scorer(self, level):
        return Oracle(self.ev.logN, self.ev.q[:level], self.ev.p, self.log_scale, self.R, self.B)

    def scaled_rows(self, rows):
        """what is enrolled: the candidates times kappa / lam (float32, as every candidate row of the scoring path)"""
        return (rows.astype(np.float64) * (self.kappa / self.lam)).astype(np.float32)

    def scores(self, ct_q, rows, level):
        """kappa <x_i, q_R> in slot i for up to n rows: the ordinary diagonal scorer (baby set, multiply-accumulate, Horner)
        on the first `level` primes, against candidates enrolled as scaled_rows(); ends one level below"""
        ev = self.ev
        assert rows.shape[0] <= self.n and rows.shape[1] == self.R
        o = self.scorer(level)
        q = ev.drop(ct_q, level)
        keys = np.stack([ev._key(ev.rot_keys[r], level) for r in self.score_rotations()])
        sc, _, _ = o.score_block(self.scaled_rows(rows), o.baby_set(q.res, keys), keys[self.B - 1])
        return ev.rescale(Ct(sc, q.scale * 2.0 ** self.log_scale))

    def decide(self, ct_q, rows):
        """Ct whose slot i is ~ sign(<x_i, q_R> - tau |q_R|), amplified towards +-1"""
        ev = self.ev
        r = self.threshold(ct_q)
        s = self.scores(ct_q, rows, r.level + 1)
        self.levels = {"threshold": r.level, "score": s.level}
        x = ev.sub(s, r)
        for _ in range(self.sign_iters):
            w = ev.add_const(ev.neg(ev.mul(x, x)), 3.0)          # 3 - x^2, one prime ~Delta
            x = ev.mul(x, w)                                      # x (3 - x^2) over a prime ~2 Delta: read at the same scale
            x = Ct(x.res, x.scale * 2.0)                          # ... it is x (3 - x^2) / 2
        self.levels["out"] = x.level
        return x
