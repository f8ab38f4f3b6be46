"""ctypes front end of the CPU oracle (``hann_oracle.c``).

TEST INFRASTRUCTURE ONLY: the plain, slow RNS-CKKS reference that the CUDA library is checked
against.  Nothing here is imported by the product package; it imports nothing from it either.

Every polynomial crossing this interface is in the canonical exchange layout: coefficient
domain, natural order, residues in [0, q_i), ``uint64``, index order ``[poly][limb][coeff]``.
CRT reconstruction (Sec. 2, "The round trip": the client decrypts the scores) is done here with
python integers, the most obviously exact arithmetic available.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hann_oracle.c")
_LIB = os.path.join(_HERE, "libhann_oracle.so")

u64p = C.POINTER(C.c_uint64)
i64p = C.POINTER(C.c_int64)
i8p = C.POINTER(C.c_int8)
f32p = C.POINTER(C.c_float)
f64p = C.POINTER(C.c_double)
i32p = C.POINTER(C.c_int)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no FMA contraction: the encode order of operations is pinned)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lquadmath", "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_create.restype = C.c_void_p
        _lib.orc_create.argtypes = [C.c_int, C.c_int, u64p, C.c_int, C.c_int, C.c_int]
        _lib.orc_destroy.argtypes = [C.c_void_p]
        _lib.orc_get_psi.restype = C.c_uint64
        _lib.orc_get_psi.argtypes = [C.c_void_p, C.c_int]
        _lib.orc_galois.restype = C.c_long
        _lib.orc_galois.argtypes = [C.c_void_p, C.c_int]
        _lib.orc_is_prime.argtypes = [C.c_uint64]
        _lib.orc_find_primes.argtypes = [C.c_int, C.c_int, C.c_int, u64p]
        _lib.orc_automorphism.argtypes = [C.c_void_p, C.c_int, C.c_long, u64p, u64p]
        _lib.orc_automorphism_ntt.argtypes = [C.c_void_p, C.c_long, u64p, u64p]
        _lib.orc_decode.argtypes = [C.c_void_p, f64p, C.c_double, f64p, f64p]
        _lib.orc_hash64.restype = C.c_uint64
        _lib.orc_hash64.argtypes = [C.c_uint64, C.c_uint64, C.c_uint64]
    return _lib


def _p(a, typ):
    return a.ctypes.data_as(typ)


def _u64(a):
    a = np.ascontiguousarray(a, dtype=np.uint64)
    return a


def find_primes(bits: int, logstep: int, count: int):
    out = np.zeros(count, dtype=np.uint64)
    k = lib().orc_find_primes(bits, logstep, count, _p(out, u64p))
    return [int(x) for x in out[:k]]


def is_prime(x: int) -> bool:
    return bool(lib().orc_is_prime(C.c_uint64(x)))


class Oracle:
    """One parameter set: ring 2^logN, ciphertext primes q (list), special prime p, scale 2^log_scale,
    padded dimension R, baby-step count B (G = R/B giant steps)."""

    def __init__(self, logN, q, p, log_scale, R, B):
        self.logN, self.N, self.n = logN, 1 << logN, 1 << (logN - 1)
        self.L = len(q)
        self.q = [int(x) for x in q]
        self.p = int(p)
        self.mods = self.q + [self.p]
        self.log_scale, self.R, self.B, self.G = log_scale, R, B, R // B
        m = np.array(self.mods, dtype=np.uint64)
        self._h = lib().orc_create(logN, self.L, _p(m, u64p), log_scale, R, B)
        if not self._h:
            raise ValueError("invalid oracle parameters")
        self.Q = 1
        for x in self.q:
            self.Q *= x

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_destroy(C.c_void_p(self._h))
            self._h = None

    @property
    def h(self):
        return C.c_void_p(self._h)

    # ---- tables and index maps
    def tables(self):
        n = self.n
        nh = max(n // 2, 1)
        Tr, Ti = np.zeros(nh), np.zeros(nh)
        Ur, Ui = np.zeros(n), np.zeros(n)
        g5, u = np.zeros(n, dtype=np.int32), np.zeros(n, dtype=np.int32)
        lib().orc_get_tables(self.h, _p(Tr, f64p), _p(Ti, f64p), _p(Ur, f64p), _p(Ui, f64p), _p(g5, i32p), _p(u, i32p))
        return dict(T_re=Tr, T_im=Ti, U_re=Ur, U_im=Ui, g5=g5, uidx=u)

    def psi(self, limb):
        return int(lib().orc_get_psi(self.h, limb))

    def galois(self, r):
        return int(lib().orc_galois(self.h, r))

    # ---- transforms (one limb)
    def ntt(self, limb, a):
        a = _u64(a).copy()
        lib().orc_ntt(self.h, C.c_int(limb), _p(a, u64p))
        return a

    def intt(self, limb, a):
        a = _u64(a).copy()
        lib().orc_intt(self.h, C.c_int(limb), _p(a, u64p))
        return a

    def negacyclic_mul(self, limb, a, b):
        a, b = _u64(a), _u64(b)
        out = np.zeros(self.N, dtype=np.uint64)
        lib().orc_negacyclic_mul(self.h, C.c_int(limb), _p(a, u64p), _p(b, u64p), _p(out, u64p))
        return out

    def automorphism(self, limb, k, a):
        a = _u64(a)
        out = np.zeros(self.N, dtype=np.uint64)
        lib().orc_automorphism(self.h, limb, C.c_long(k), _p(a, u64p), _p(out, u64p))
        return out

    def automorphism_ntt(self, k, a):
        a = _u64(a)
        out = np.zeros(self.N, dtype=np.uint64)
        lib().orc_automorphism_ntt(self.h, C.c_long(k), _p(a, u64p), _p(out, u64p))
        return out

    # ---- encode / decode
    def encode(self, z, log_scale=None):
        z = np.ascontiguousarray(z, dtype=np.float64)
        assert z.shape == (self.n,)
        m = np.zeros(self.N, dtype=np.int64)
        lib().orc_encode(self.h, _p(z, f64p), C.c_int(self.log_scale if log_scale is None else log_scale), _p(m, i64p))
        return m

    def decode(self, mu, scale):
        """mu: float64[N] real coefficients -> complex slots[n] (z_j = mu(omega^{g_j}) / scale)."""
        mu = np.ascontiguousarray(mu, dtype=np.float64)
        zr, zi = np.zeros(self.n), np.zeros(self.n)
        lib().orc_decode(self.h, _p(mu, f64p), C.c_double(scale), _p(zr, f64p), _p(zi, f64p))
        return zr + 1j * zi

    def reduce(self, m, nlimbs=None):
        """integer polynomial (python ints / int64) -> residues [nlimbs][N]"""
        nl = self.L if nlimbs is None else nlimbs
        mo = np.array([int(x) for x in m], dtype=object)
        return np.stack([np.array([int(v) for v in (mo % self.mods[l])], dtype=np.uint64) for l in range(nl)])

    def crt_centred(self, res):
        """residues [L][N] -> list-like object array of centred python integers in (-Q/2, Q/2]."""
        res = np.asarray(res)
        L, Q = self.L, self.Q
        acc = np.zeros(res.shape[1], dtype=object)
        for l in range(L):
            Qh = Q // self.q[l]
            w = Qh * pow(Qh % self.q[l], -1, self.q[l])
            acc = acc + res[l].astype(object) * w
        acc = acc % Q
        half = Q // 2
        return np.array([int(v) - Q if int(v) > half else int(v) for v in acc], dtype=object)

    # ---- encryption
    def encrypt(self, s, m, a, e):
        s = np.ascontiguousarray(s, dtype=np.int8)
        m = np.ascontiguousarray(m, dtype=np.int64)
        a = _u64(a)
        e = np.ascontiguousarray(e, dtype=np.int8)
        assert a.shape == (self.L, self.N)
        ct = np.zeros((2, self.L, self.N), dtype=np.uint64)
        lib().orc_encrypt(self.h, _p(s, i8p), _p(m, i64p), _p(a, u64p), _p(e, i8p), _p(ct, u64p))
        return ct

    def encrypt_query(self, s, qvec, a, e):
        """E3: slot vector z[i] = q[i mod R] (query tiled n/R times), encoded at Delta, encrypted."""
        qv = np.zeros(self.R, dtype=np.float32)
        qv[: len(qvec)] = np.asarray(qvec, dtype=np.float32)
        z = np.tile(qv.astype(np.float64), self.n // self.R)
        return self.encrypt(s, self.encode(z), a, e)

    def expand_uniform(self, seed, stream):
        """the uniform half a [L][N] of a seed-compressed ciphertext"""
        a = np.zeros((self.L, self.N), dtype=np.uint64)
        lib().orc_expand_uniform(self.h, C.c_uint64(seed), C.c_uint64(stream), _p(a, u64p))
        return a

    def decrypt_residues(self, s, ct):
        s = np.ascontiguousarray(s, dtype=np.int8)
        ct = _u64(ct)
        mu = np.zeros((self.L, self.N), dtype=np.uint64)
        lib().orc_decrypt_residues(self.h, _p(s, i8p), _p(ct, u64p), _p(mu, u64p))
        return mu

    def decrypt_int(self, s, ct):
        return self.crt_centred(self.decrypt_residues(s, ct))

    def decrypt_slots(self, s, ct, log_scale_out):
        mu = self.decrypt_int(s, ct)
        muf = np.array([float(v) for v in mu], dtype=np.float64)
        return self.decode(muf, float(2.0 ** log_scale_out))

    # ---- output compaction
    def compact(self, ct, keep=1, rescale=True):
        """keep the first `keep` limbs, after a rescale by the last prime if asked (scale / q_{L-1}):
        [2][L][N] -> [2][keep][N]"""
        ct = _u64(ct)
        assert ct.shape == (2, self.L, self.N) and 1 <= keep <= self.L - (1 if rescale else 0)
        out = np.zeros((2, keep, self.N), dtype=np.uint64)
        lib().orc_compact(self.h, _p(ct, u64p), C.c_int(keep), C.c_int(1 if rescale else 0), _p(out, u64p))
        return out

    def decrypt_compact_int(self, s, ctc):
        """centred integers of c0 + c1*s over the limbs the compact ciphertext still has"""
        s = np.ascontiguousarray(s, dtype=np.int8)
        ctc = _u64(ctc)
        nl = ctc.shape[1]
        mu = np.zeros((nl, self.N), dtype=np.uint64)
        lib().orc_decrypt_residues_limbs(self.h, _p(s, i8p), _p(ctc, u64p), C.c_int(nl), _p(mu, u64p))
        Q = 1
        for l in range(nl):
            Q *= self.q[l]
        acc = np.zeros(self.N, dtype=object)
        for l in range(nl):
            Qh = Q // self.q[l]
            acc = acc + mu[l].astype(object) * (Qh * pow(Qh % self.q[l], -1, self.q[l]))
        acc = acc % Q
        return np.array([int(v) - Q if int(v) > Q // 2 else int(v) for v in acc], dtype=object)

    def decrypt_compact_slots(self, s, ctc, log_scale_in, rescaled=True):
        """slots of a compacted ciphertext whose scale was 2^log_scale_in before compaction"""
        mu = self.decrypt_compact_int(s, ctc)
        muf = np.array([float(v) for v in mu], dtype=np.float64)
        scale = float(2.0 ** log_scale_in)
        return self.decode(muf, scale / float(self.q[self.L - 1]) if rescaled else scale)

    # ---- keys, key switching, rotation
    def evk_gen(self, s, r, a, e):
        s = np.ascontiguousarray(s, dtype=np.int8)
        a = _u64(a)
        e = np.ascontiguousarray(e, dtype=np.int8)
        L = self.L
        assert a.shape == (L, L + 1, self.N) and e.shape == (L, self.N)
        evk = np.zeros((L, 2, L + 1, self.N), dtype=np.uint64)
        lib().orc_evk_gen(self.h, _p(s, i8p), C.c_int(r), _p(a, u64p), _p(e, i8p), _p(evk, u64p))
        return evk

    def rlk_gen(self, s, a, e):
        """relinearisation key (evaluation key for s^2), same layout as evk_gen"""
        s = np.ascontiguousarray(s, dtype=np.int8)
        a = _u64(a)
        e = np.ascontiguousarray(e, dtype=np.int8)
        L = self.L
        assert a.shape == (L, L + 1, self.N) and e.shape == (L, self.N)
        evk = np.zeros((L, 2, L + 1, self.N), dtype=np.uint64)
        lib().orc_rlk_gen(self.h, _p(s, i8p), _p(a, u64p), _p(e, i8p), _p(evk, u64p))
        return evk

    def encrypt_block(self, s, pt, a, e):
        """pt [G][B][L][N] (or [R][L][N]) -> ctdb [R][2][L][N] under s with the given a [R][L][N], e [R][N]"""
        s = np.ascontiguousarray(s, dtype=np.int8)
        pt, a = _u64(pt).reshape(self.R, self.L, self.N), _u64(a)
        e = np.ascontiguousarray(e, dtype=np.int8)
        assert a.shape == (self.R, self.L, self.N) and e.shape == (self.R, self.N)
        out = np.zeros((self.R, 2, self.L, self.N), dtype=np.uint64)
        lib().orc_encrypt_block(self.h, _p(s, i8p), _p(pt, u64p), _p(a, u64p), _p(e, i8p), _p(out, u64p))
        return out

    def mac_ct(self, ctdb, baby):
        ctdb, baby = _u64(ctdb), _u64(baby)
        out = np.zeros((self.G, 3, self.L, self.N), dtype=np.uint64)
        lib().orc_mac_ct(self.h, _p(ctdb, u64p), _p(baby, u64p), _p(out, u64p))
        return out

    def relin(self, d, rlk):
        d, rlk = _u64(d), _u64(rlk)
        assert d.shape == (3, self.L, self.N)
        out = np.zeros((2, self.L, self.N), dtype=np.uint64)
        lib().orc_relin(self.h, _p(d, u64p), _p(rlk, u64p), _p(out, u64p))
        return out

    def moddown(self, u):
        u = _u64(u)
        out = np.zeros((self.L, self.N), dtype=np.uint64)
        lib().orc_moddown(self.h, _p(u, u64p), _p(out, u64p))
        return out

    def keyswitch(self, d, evk):
        d, evk = _u64(d), _u64(evk)
        ks0 = np.zeros((self.L, self.N), dtype=np.uint64)
        ks1 = np.zeros((self.L, self.N), dtype=np.uint64)
        lib().orc_keyswitch(self.h, _p(d, u64p), _p(evk, u64p), _p(ks0, u64p), _p(ks1, u64p))
        return ks0, ks1

    def rotate(self, ct, r, evk_r, hoisted=False):
        ct, evk_r = _u64(ct), _u64(evk_r)
        out = np.zeros((2, self.L, self.N), dtype=np.uint64)
        f = lib().orc_rotate_hoisted if hoisted else lib().orc_rotate
        f(self.h, _p(ct, u64p), C.c_int(r), _p(evk_r, u64p), _p(out, u64p))
        return out

    def baby_set(self, ct, evk):
        """evk[r-1] is the key of rotation r, r = 1..B-1 (more keys may follow; they are ignored)."""
        ct, evk = _u64(ct), _u64(evk)
        baby = np.zeros((self.B, 2, self.L, self.N), dtype=np.uint64)
        lib().orc_baby_set(self.h, _p(ct, u64p), _p(evk, u64p), _p(baby, u64p))
        return baby

    # ---- block scoring
    def encode_block(self, rows):
        rows = np.ascontiguousarray(rows, dtype=np.float32)
        assert rows.ndim == 2 and rows.shape[1] == self.R and rows.shape[0] <= self.n
        pt = np.zeros((self.G, self.B, self.L, self.N), dtype=np.uint64)
        lib().orc_encode_block(self.h, _p(rows, f32p), C.c_int(rows.shape[0]), _p(pt, u64p))
        return pt

    def mac(self, pt, baby):
        pt, baby = _u64(pt), _u64(baby)
        inner = np.zeros((self.G, 2, self.L, self.N), dtype=np.uint64)
        lib().orc_mac(self.h, _p(pt, u64p), _p(baby, u64p), _p(inner, u64p))
        return inner

    def rotate_sum(self, inner, evk_B):
        inner, evk_B = _u64(inner), _u64(evk_B)
        out = np.zeros((2, self.L, self.N), dtype=np.uint64)
        lib().orc_rotate_sum(self.h, _p(inner, u64p), _p(evk_B, u64p), _p(out, u64p))
        return out

    def ks_accumulate(self, d, evk, u0=None, u1=None):
        """(u0, u1) += sum_j digit_j(d) * (b_j, a_j) over the L+1 moduli (no ModDown); returns the two [L+1][N] arrays"""
        d, evk = _u64(d), _u64(evk)
        u0 = np.zeros((self.L + 1, self.N), dtype=np.uint64) if u0 is None else u0
        u1 = np.zeros((self.L + 1, self.N), dtype=np.uint64) if u1 is None else u1
        lib().orc_ks_accumulate(self.h, _p(d, u64p), _p(evk, u64p), _p(u0, u64p), _p(u1, u64p))
        return u0, u1

    def rotate_sum_lazy(self, inner, evk_giant):
        """sum_g rot_{gB}(inner[g]) with the keys of rotations B, 2B, .., (G-1)B (evk_giant[g-1]) and one ModDown"""
        inner, evk_giant = _u64(inner), _u64(evk_giant)
        assert inner.shape == (self.G, 2, self.L, self.N) and evk_giant.shape[0] == max(self.G - 1, 0)
        out = np.zeros((2, self.L, self.N), dtype=np.uint64)
        lib().orc_rotate_sum_lazy(self.h, _p(inner, u64p), _p(evk_giant, u64p), _p(out, u64p))
        return out

    def score_block(self, rows, baby, evk_B, want_pt=False, want_inner=False):
        rows = np.ascontiguousarray(rows, dtype=np.float32)
        baby, evk_B = _u64(baby), _u64(evk_B)
        out = np.zeros((2, self.L, self.N), dtype=np.uint64)
        pt = np.zeros((self.G, self.B, self.L, self.N), dtype=np.uint64) if want_pt else None
        inner = np.zeros((self.G, 2, self.L, self.N), dtype=np.uint64) if want_inner else None
        lib().orc_score_block(
            self.h, _p(rows, f32p), C.c_int(rows.shape[0]), _p(baby, u64p), _p(evk_B, u64p), _p(out, u64p),
            _p(pt, u64p) if want_pt else None, _p(inner, u64p) if want_inner else None,
        )
        return out, pt, inner

    # ---- pieces of the packed projection
    def encode_plain(self, z, log_scale=None):
        """real slot vector -> plaintext residues [L][N] at scale 2^log_scale"""
        z = np.ascontiguousarray(z, dtype=np.float64)
        assert z.shape == (self.n,)
        pt = np.zeros((self.L, self.N), dtype=np.uint64)
        lib().orc_encode_plain(self.h, _p(z, f64p), C.c_int(self.log_scale if log_scale is None else log_scale), _p(pt, u64p))
        return pt

    def mul_plain_acc(self, ct, pt, acc=None):
        """acc += ct * pt (ciphertext x plaintext); returns acc [2][L][N]"""
        ct, pt = _u64(ct), _u64(pt)
        acc = np.zeros((2, self.L, self.N), dtype=np.uint64) if acc is None else acc
        lib().orc_mul_plain_acc(self.h, _p(ct, u64p), _p(pt, u64p), _p(acc, u64p))
        return acc

    def add(self, a, b):
        """a + b for ciphertexts / polynomial stacks [..][L][N]"""
        mods = np.array(self.q, dtype=object).reshape((1,) * (np.ndim(a) - 2) + (self.L, 1))
        return ((np.asarray(a).astype(object) + np.asarray(b).astype(object)) % mods).astype(np.uint64)

    @staticmethod
    def num_threads():
        return int(lib().orc_num_threads())


def restrict_keys(evk, L_from, L_to):
    """Evaluation keys [..][L_from][2][L_from+1][N] of a chain of L_from primes, restricted to its first L_to primes:
    digits 0..L_to-1, limbs q_0..q_{L_to-1} and the special prime.  With one-prime digits the key material of digit j on
    limb i (b_j = -a_j s + e_j + F_j s', F_j = p mod q_j on limb j, 0 elsewhere) does not depend on the other primes, so
    the restriction IS the key of the shorter chain."""
    limbs = list(range(L_to)) + [L_from]
    return np.ascontiguousarray(np.asarray(evk)[..., :L_to, :, :, :][..., limbs, :])


class PackedProjection:
    """Rank reduction under encryption with the matrix packed by windows (Sec. 3.1 "How" and Detail):
    Enc(q_R) = W^T Enc(q), W of shape D x R (D = c R), by the diagonal method with baby and giant steps.

    Reading taken (the paper gives no index formulas):
      * slots are viewed with period D; window k of a period is positions kR .. kR+R-1; the query ciphertext holds
        q[i mod D]; chunk k of W is the R x R matrix W_k^T[r][col] = W[kR + col][r];
      * ONE packed object per diagonal d = gB + b of all c chunks (storage R objects, not D): slot kR + j of P[g][b]
        holds W_k^T[(j - gB) mod R][(j + b) mod R] -- the diagonal, shifted IN its window by the giant-step amount in
        plaintext (the paper's plaintext pre-rotation);
      * a baby step must rotate every chunk of the query INSIDE its window.  A slot rotation moves data across window
        boundaries, so the in-window rotation is put together from two slot rotations with 0/1 plaintext masks (a public
        constant: a ciphertext x plaintext multiply, no key switch):
            cyc_b = lo_b * rot_b(ct) + hi_b * rot_{b-R}(ct),  lo_b[i] = [(i mod R) + b < R],  hi_b = 1 - lo_b;
        the masks are encoded at scale 2^log_mask, and ONE rescale (by the last prime) follows;
      * inner[g] = sum_b P[g][b] * cyc_b, then the giant steps sum_g rot_{gB}(inner[g]) with ordinary slot rotations:
        these DO mix adjacent windows (slot kR + j receives from window k or k + 1), which is harmless because
      * a single final fold, acc += rot_{R 2^t}(acc) for t < log2 c, adds up all windows: window mixing is a fixed
        permutation of the windows, invisible to their sum.  Every slot i then holds q_R[i mod R]: the projected query,
        already tiled for the scoring levels;
      * one more rescale (by the next prime) returns the scale to about 2^log_scale: the projected query has L - 2 primes
        and scores at scale Delta^2 again.
    Three parameter sets of the same ring share the keys (restrict_keys): top (L primes: baby rotations and masks), mid
    (L - 1: matrix product, giant steps, fold), low (L - 2: what the scoring levels run on)."""

    def __init__(self, logN, q, p, log_scale, D, R, B, log_mask, log_w):
        assert D % R == 0 and R % B == 0 and len(q) >= 3
        self.D, self.R, self.B, self.G, self.c = D, R, B, R // B, D // R
        assert self.c & (self.c - 1) == 0, "the fold doubles: D / R must be a power of two"
        self.log_scale, self.log_mask, self.log_w = log_scale, log_mask, log_w
        self.top = Oracle(logN, q, p, log_scale, R, B)
        self.mid = Oracle(logN, q[:-1], p, log_scale, R, B)
        self.low = Oracle(logN, q[:-2], p, log_scale, R, B)
        self.n, self.N, self.L = self.top.n, self.top.N, len(q)
        assert self.n % D == 0
        # exact scale of the projected query: Delta * 2^log_mask / q_{L-1} * 2^log_w / q_{L-2}
        self.scale_out = 2.0 ** log_scale * (2.0 ** log_mask / q[-1]) * (2.0 ** log_w / q[-2])

    # ---- index formulas (plain slot vectors)
    def query_slots(self, qvec):
        return np.tile(np.asarray(qvec, dtype=np.float64), self.n // self.D)

    def matrix_slots(self, W):
        """z[g][b][i] = W[kR + (j + b) mod R][(j - gB) mod R] for i mod D = kR + j"""
        W = np.asarray(W, dtype=np.float64)
        assert W.shape == (self.D, self.R)
        i = np.arange(self.n) % self.D
        k, j = i // self.R, i % self.R
        z = np.zeros((self.G, self.B, self.n))
        for g in range(self.G):
            for b in range(self.B):
                z[g, b] = W[k * self.R + (j + b) % self.R, (j - g * self.B) % self.R]
        return z

    def masks(self):
        j = np.arange(self.n) % self.R
        lo = np.stack([(j + b < self.R).astype(np.float64) for b in range(self.B)])
        return lo, 1.0 - lo

    def baby_rotations(self):
        """slot rotations the baby steps need: b and b - R (taken modulo n), b = 1 .. B-1"""
        return list(range(1, self.B)) + [self.n - self.R + b for b in range(1, self.B)]

    def fold_rotations(self):
        return [self.R << t for t in range(self.c.bit_length() - 1)]

    def plain(self, W, qvec):
        """the same steps on plain slot vectors (no encryption): what every slot must hold at the end"""
        x = self.query_slots(qvec)
        z = self.matrix_slots(W)
        lo, hi = self.masks()
        cyc = [lo[b] * np.roll(x, -b) + hi[b] * np.roll(x, -(b - self.R)) for b in range(self.B)]
        acc = np.zeros(self.n)
        for g in range(self.G):
            acc += np.roll(sum(z[g, b] * cyc[b] for b in range(self.B)), -g * self.B)
        unfolded = acc.copy()
        for r in self.fold_rotations():
            acc = acc + np.roll(acc, -r)
        return acc, unfolded

    # ---- the encrypted pipeline
    def enrol(self, W):
        """packed diagonals of W as plaintexts of the middle chain: [G][B][L-1][N] at scale 2^log_w"""
        z = self.matrix_slots(W)
        return np.stack([np.stack([self.mid.encode_plain(z[g, b], self.log_w) for b in range(self.B)]) for g in range(self.G)])

    def mask_plaintexts(self):
        lo, hi = self.masks()
        return (np.stack([self.top.encode_plain(v, self.log_mask) for v in lo]),
                np.stack([self.top.encode_plain(v, self.log_mask) for v in hi]))

    def in_window_rotations(self, ct, evk):
        """cyc[b] = lo_b * rot_b(ct) + hi_b * rot_{b-R}(ct) over the L primes (scale Delta 2^log_mask), then the rescale:
        [B][2][L-1][N].  evk: {rotation: key of the top chain}."""
        lo, hi = self.mask_plaintexts()
        out = []
        for b in range(self.B):
            a = ct if b == 0 else self.top.rotate(ct, b, evk[b])
            acc = self.top.mul_plain_acc(a, lo[b])
            if b > 0:
                r = self.n - self.R + b
                acc = self.top.mul_plain_acc(self.top.rotate(ct, r, evk[r]), hi[b], acc)
            out.append(self.top.compact(acc, self.L - 1, rescale=True))
        return np.stack(out)

    def project(self, ct, evk, Wpt, lazy=False):
        """ct [2][L][N] (query tiled with period D, scale Delta) -> projected query [2][L-2][N] at scale `scale_out`.
        evk: {rotation: key of the TOP chain} for baby_rotations(), B (or B, 2B, .. when lazy) and fold_rotations()."""
        mid, L = self.mid, self.L
        low_key = lambda r: restrict_keys(evk[r], L, L - 1)
        cyc = self.in_window_rotations(ct, evk)
        inner = mid.mac(Wpt, cyc)
        if self.G == 1:
            acc = inner[0]
        elif lazy:
            acc = mid.rotate_sum_lazy(inner, np.stack([low_key(g * self.B) for g in range(1, self.G)]))
        else:
            acc = mid.rotate_sum(inner, low_key(self.B))
        self.unfolded = acc
        for r in self.fold_rotations():
            acc = mid.add(acc, mid.rotate(acc, r, low_key(r)))
        return mid.compact(acc, L - 2, rescale=True)
