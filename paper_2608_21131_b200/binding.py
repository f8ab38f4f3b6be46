"""Thin ctypes binding of the C-ABI CUDA library (``include/hann.h``): argument marshalling only.

Every function has the name of the C entry point it wraps (without the ``hann_`` prefix) and every step of
the scoring path runs in the library's CUDA kernels.  PyTorch is used for device memory and streams; host
arrays are numpy.  There is no CPU fallback: creating a `Context` raises if the library is not built or no
CUDA device is present.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhann.so")

HANN_MAX_PRIMES = 15
OK, EINVAL, ESHAPE, ENOKEY, EWORKSPACE, ECUDA, ENOMEM = 0, -1, -2, -3, -4, -5, -6
SIZE_POLY, SIZE_CT, SIZE_BABY, SIZE_PT_BLOCK, SIZE_INNER, SIZE_EVK, SIZE_ROWS_PER_BLOCK, SIZE_CTDB_BLOCK = 1, 2, 3, 4, 5, 6, 7, 8
KIND_POLY, KIND_CT, KIND_PT = 1, 2, 3
TUNE_ENCODE_GROUP = 1
TUNE_HOST_LIMBS = 2
TUNE_ENCODE_SYMMETRY = 3
TUNE_HOST_GROUPS = 4
TUNE_GIANT_LAZY = 5
TUNE_LAZY_LANES = 6
TUNE_MAC_F64 = 7
TUNE_PAIR_B32 = 8


class HannError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("hann error %d: %s" % (code, msg))
        self.code = code


class Params(C.Structure):
    _fields_ = [
        ("logN", C.c_int32), ("L", C.c_int32), ("q", C.c_uint64 * HANN_MAX_PRIMES), ("p", C.c_uint64),
        ("log_scale", C.c_int32), ("R", C.c_int32), ("B", C.c_int32), ("device", C.c_int32), ("stream", C.c_void_p),
    ]


class Stats(C.Structure):
    _fields_ = [
        ("launches", C.c_uint64), ("ms_query_prepare", C.c_float), ("ms_encode", C.c_float),
        ("ms_score_level", C.c_float), ("ms_rotate_sum", C.c_float), ("ms_keyswitch", C.c_float),
    ]


class MembershipParams(C.Structure):
    _fields_ = [
        ("R", C.c_int32), ("deg", C.c_int32), ("sign_iters", C.c_int32), ("log_scale", C.c_int32),
        ("tau", C.c_double), ("t_lo", C.c_double), ("t_hi", C.c_double), ("coef", C.POINTER(C.c_double)),
    ]


_lib = None


def load_library():
    """Load ``libhann.so``; raises (never falls back) when it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    path = os.environ.get("HANN_LIB", LIB_PATH)  # development override: an alternative build of the same library
    if not os.path.exists(path):
        raise RuntimeError(
            "the CUDA library %s is missing: build it with `python -m paper_2608_21131_b200.build`" % path
        )
    lib = C.CDLL(path)
    vp, i64, sz = C.c_void_p, C.c_int64, C.c_size_t
    sig = {
        "hann_ctx_create": (C.c_int, [C.POINTER(Params), C.POINTER(vp)]),
        "hann_ctx_destroy": (None, [vp]),
        "hann_sizeof": (i64, [vp, C.c_int]),
        "hann_workspace_bytes": (i64, [vp, i64]),
        "hann_sync": (C.c_int, [vp]),
        "hann_last_error": (C.c_char_p, [vp]),
        "hann_set_timing": (C.c_int, [vp, C.c_int]),
        "hann_get_stats": (C.c_int, [vp, C.POINTER(Stats)]),
        "hann_set_tuning": (C.c_int, [vp, C.c_int, C.c_int]),
        "hann_kernel_classes": (C.c_int, []),
        "hann_kernel_name": (C.c_char_p, [C.c_int]),
        "hann_kernel_profile": (C.c_int, [vp, C.c_int]),
        "hann_kernel_times": (C.c_int, [vp, vp, vp]),
        "hann_keygen_from_samples": (C.c_int, [vp, vp, C.c_int, vp, vp, vp, vp]),
        "hann_keygen_seeded": (C.c_int, [vp, C.c_uint64, C.c_int, vp, vp, vp]),
        "hann_probe_rates": (C.c_int, [vp, vp, vp]),
        "hann_debug_build": (C.c_int, []),
        "hann_debug_canaries": (C.c_int, [vp, C.c_int]),
        "hann_debug_verify": (C.c_int, [vp, vp, vp]),
        "hann_encrypt_query": (C.c_int, [vp, vp, vp, C.c_int, vp, vp, vp]),
        "hann_decrypt_scores": (C.c_int, [vp, vp, vp, i64, C.c_int, vp, vp]),
        "hann_load_keys": (C.c_int, [vp, vp, C.c_int, vp]),
        "hann_query_prepare": (C.c_int, [vp, vp, vp, vp, sz]),
        "hann_encode_candidates": (C.c_int, [vp, vp, i64, C.c_int, vp, vp, sz]),
        "hann_score_level": (C.c_int, [vp, vp, vp, i64, vp, vp, sz]),
        "hann_keygen_relin_from_samples": (C.c_int, [vp, vp, vp, vp, vp]),
        "hann_encrypt_block": (C.c_int, [vp, vp, vp, vp, vp, vp]),
        "hann_score_level_ctdb": (C.c_int, [vp, vp, vp, i64, vp, vp, sz]),
        "hann_selftest_bounded_wait": (C.c_int, [vp, C.c_int, vp]),
        "hann_score_level_batch": (C.c_int, [vp, vp, C.c_int, vp, i64, vp, vp, sz]),
        "hann_rotate_sum": (C.c_int, [vp, vp, i64, vp, vp, sz]),
        "hann_rotate_sum_lazy": (C.c_int, [vp, vp, i64, vp, vp, sz]),
        "hann_multiply": (C.c_int, [vp, vp, vp, i64, vp, vp, sz]),
        "hann_rotate_hoisted": (C.c_int, [vp, vp, C.c_int, C.c_int, vp, vp, sz]),
        "hann_encode_slots": (C.c_int, [vp, vp, i64, C.c_int, vp, vp, sz]),
        "hann_project_enrol": (C.c_int, [vp, vp, C.c_int, C.c_int, vp, vp, sz]),
        "hann_project_masks": (C.c_int, [vp, C.c_int, vp, vp, vp, sz]),
        "hann_project_baby": (C.c_int, [vp, vp, vp, vp, vp, vp, sz]),
        "hann_rescale": (C.c_int, [vp, vp, i64, vp, vp, sz]),
        "hann_fold": (C.c_int, [vp, vp, C.c_int, C.c_int, vp, sz]),
        "hann_project_bytes": (i64, [vp, vp]),
        "hann_project_query": (C.c_int, [vp, vp, vp, vp, vp, vp, C.c_int, vp, vp, sz]),
        "hann_membership_levels": (C.c_int, [C.c_int, C.c_int, vp, vp]),
        "hann_membership_bytes": (i64, [vp, C.c_int, vp, vp, i64]),
        "hann_membership_decide": (C.c_int, [vp, C.c_int, vp, vp, vp, vp, i64, vp, vp, vp, vp, vp, vp, sz]),
        "hann_keyswitch": (C.c_int, [vp, C.c_int, vp, vp, vp, vp, sz]),
        "hann_query_level": (C.c_int, [vp, vp, vp, i64, C.c_int, vp, vp, vp, vp, vp, sz]),
        "hann_static_scratch_bytes": (i64, []),
        "hann_keyswitch_bytes": (i64, [vp]),
        "hann_keyswitch_static": (C.c_int, [vp, C.c_int, vp, vp, vp]),
        "hann_import": (C.c_int, [vp, C.c_int, vp, i64, vp]),
        "hann_export": (C.c_int, [vp, C.c_int, vp, i64, vp]),
        "hann_expand_uniform": (C.c_int, [vp, C.c_uint64, C.c_uint64, vp]),
        "hann_import_seeded_ct": (C.c_int, [vp, vp, C.c_uint64, C.c_uint64, vp]),
        "hann_export_limbs": (C.c_int, [vp, vp, i64, C.c_int, vp]),
        "hann_compact_bytes": (i64, [vp, i64, C.c_int]),
        "hann_compact_scores": (C.c_int, [vp, vp, i64, C.c_int, C.c_int, vp, vp, sz]),
        "hann_decrypt_compact": (C.c_int, [vp, vp, vp, i64, C.c_int, C.c_int, C.c_int, vp, vp]),
        "hann_level_host_bytes": (i64, [vp, i64]),
        "hann_score_level_host": (C.c_int, [vp, vp, vp, i64, C.c_int, vp, vp, sz]),
    }
    for name, (res, args) in sig.items():
        f = getattr(lib, name)
        f.restype = res
        f.argtypes = args
    _lib = lib
    return lib


def _np(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _ptr(a):
    """address of a numpy array or a torch tensor (host or device)"""
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        return a.ctypes.data
    return a.data_ptr()


def restrict_keys(evk, L_from, L_to):
    """Evaluation keys [..][L_from][2][L_from+1][N] (canonical) restricted to the chain of the first L_to primes: digits
    0..L_to-1 and limbs q_0..q_{L_to-1} plus the special prime.  Pure slicing: with one-prime digits that IS the key of
    the shorter chain, so a client generates keys once for its longest chain."""
    limbs = list(range(L_to)) + [L_from]
    return np.ascontiguousarray(np.asarray(evk)[..., :L_to, :, :, :][..., limbs, :])


class Context:
    """One parameter set bound to one CUDA device and stream.  `ps` needs the attributes logN, q, p, log_scale,
    R, B."""

    def __init__(self, ps, device: int = 0, stream=None):
        import torch

        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the scoring path has no CPU fallback")
        self.torch = torch
        self.lib = load_library()
        self.device = torch.device("cuda", device)
        self.logN, self.N, self.n = ps.logN, 1 << ps.logN, 1 << (ps.logN - 1)
        self.L, self.R, self.B, self.G = len(ps.q), ps.R, ps.B, ps.R // ps.B
        self.log_scale = ps.log_scale
        prm = Params()
        prm.logN, prm.L, prm.p, prm.log_scale, prm.R, prm.B, prm.device = ps.logN, len(ps.q), ps.p, ps.log_scale, ps.R, ps.B, device
        for i, q in enumerate(ps.q):
            prm.q[i] = q
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        self.stream = stream
        prm.stream = stream.cuda_stream
        h = C.c_void_p()
        rc = self.lib.hann_ctx_create(C.byref(prm), C.byref(h))
        if rc != OK:
            raise HannError(rc, "hann_ctx_create failed (invalid parameters or CUDA error)")
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            self.lib.hann_ctx_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ck(self, rc):
        if rc != OK:
            raise HannError(rc, self.lib.hann_last_error(self.h).decode())

    # ---- sizes and buffers
    def sizeof(self, what):
        return int(self.lib.hann_sizeof(self.h, what))

    def workspace_bytes(self, max_blocks):
        return int(self.lib.hann_workspace_bytes(self.h, max_blocks))

    def alloc(self, nbytes):
        """uint64 device tensor of at least nbytes (torch allocations are 512-byte aligned)"""
        return self.torch.empty((int(nbytes) + 7) // 8, dtype=self.torch.int64, device=self.device)

    def workspace(self, max_blocks):
        return self.alloc(self.workspace_bytes(max_blocks))

    def selftest_bounded_wait(self, limit_ms):
        """device milliseconds the self-test warp waited before giving up; the next sync() raises"""
        w = C.c_double(0.0)
        self._ck(self.lib.hann_selftest_bounded_wait(self.h, int(limit_ms), C.byref(w)))
        return w.value

    def sync(self):
        self._ck(self.lib.hann_sync(self.h))

    def set_timing(self, on):
        self._ck(self.lib.hann_set_timing(self.h, 1 if on else 0))

    def get_stats(self):
        st = Stats()
        self._ck(self.lib.hann_get_stats(self.h, C.byref(st)))
        return {k: getattr(st, k) for k, _ in Stats._fields_}

    def set_tuning(self, what, value):
        self._ck(self.lib.hann_set_tuning(self.h, what, value))

    def kernel_profile(self, on):
        self._ck(self.lib.hann_kernel_profile(self.h, 1 if on else 0))

    def kernel_times(self):
        """{kernel class: (summed device ms, launches)} since the previous call"""
        k = self.lib.hann_kernel_classes()
        ms = np.zeros(k, dtype=np.float64)
        cnt = np.zeros(k, dtype=np.uint64)
        self._ck(self.lib.hann_kernel_times(self.h, _ptr(ms), _ptr(cnt)))
        return {self.lib.hann_kernel_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(k)}

    # ---- client side
    def keygen_from_samples(self, s, rots, a, e):
        s, a, e = _np(s, np.int8), _np(a, np.uint64), _np(e, np.int8)
        rots = _np(rots, np.int32)
        L, N = self.L, self.N
        assert a.shape == (len(rots), L, L + 1, N) and e.shape == (len(rots), L, N) and s.shape == (N,)
        evk = np.empty((len(rots), L, 2, L + 1, N), dtype=np.uint64)
        self._ck(self.lib.hann_keygen_from_samples(self.h, _ptr(s), len(rots), _ptr(rots), _ptr(a), _ptr(e), _ptr(evk)))
        return evk

    def keygen_seeded(self, seed, rots):
        """secret key [N] int8 and evaluation keys [len(rots)][L][2][L+1][N] drawn from a 64-bit seed"""
        rots = _np(rots, np.int32)
        L, N = self.L, self.N
        s = np.empty(N, dtype=np.int8)
        evk = np.empty((len(rots), L, 2, L + 1, N), dtype=np.uint64)
        self._ck(self.lib.hann_keygen_seeded(self.h, seed, len(rots), _ptr(rots), _ptr(s), _ptr(evk)))
        return s, evk

    def probe_rates(self):
        """(binary64 modular butterflies/s, int32 multiply-adds/s) measured on the context's device"""
        a, b = C.c_double(0.0), C.c_double(0.0)
        self._ck(self.lib.hann_probe_rates(self.h, C.byref(a), C.byref(b)))
        return a.value, b.value

    def debug_canaries(self, on):
        self._ck(self.lib.hann_debug_canaries(self.h, 1 if on else 0))

    def debug_verify(self):
        """(guards checked, guards damaged) since the last call; raises if any guard was overwritten"""
        a, b = C.c_int64(0), C.c_int64(0)
        self._ck(self.lib.hann_debug_verify(self.h, C.byref(a), C.byref(b)))
        return a.value, b.value

    def keygen_relin_from_samples(self, s, a, e):
        s, a, e = _np(s, np.int8), _np(a, np.uint64), _np(e, np.int8)
        L, N = self.L, self.N
        assert a.shape == (L, L + 1, N) and e.shape == (L, N) and s.shape == (N,)
        evk = np.empty((L, 2, L + 1, N), dtype=np.uint64)
        self._ck(self.lib.hann_keygen_relin_from_samples(self.h, _ptr(s), _ptr(a), _ptr(e), _ptr(evk)))
        return evk

    def encrypt_block(self, s, pt_block, a, e, out=None):
        """one encoded block (device, internal) -> its R ciphertexts (device, internal)"""
        s, a, e = _np(s, np.int8), _np(a, np.uint64), _np(e, np.int8)
        assert a.shape == (self.R, self.L, self.N) and e.shape == (self.R, self.N)
        if out is None:
            out = self.alloc(self.sizeof(SIZE_CTDB_BLOCK))
        self._ck(self.lib.hann_encrypt_block(self.h, _ptr(s), _ptr(pt_block), _ptr(a), _ptr(e), _ptr(out)))
        return out

    def encrypt_query(self, s, q, a, e):
        s, q, a, e = _np(s, np.int8), _np(q, np.float32), _np(a, np.uint64), _np(e, np.int8)
        assert a.shape == (self.L, self.N) and e.shape == (self.N,)
        ct = np.empty((2, self.L, self.N), dtype=np.uint64)
        self._ck(self.lib.hann_encrypt_query(self.h, _ptr(s), _ptr(q), len(q), _ptr(a), _ptr(e), _ptr(ct)))
        return ct

    def decrypt_scores(self, s, ct, log_scale_out=None, want_imag=False):
        s, ct = _np(s, np.int8), _np(ct, np.uint64)
        ct = ct.reshape(-1, 2, self.L, self.N)
        count = ct.shape[0]
        scores = np.empty((count, self.n), dtype=np.float64)
        imag = np.empty((count, self.n), dtype=np.float64) if want_imag else None
        ls = 2 * self.log_scale if log_scale_out is None else log_scale_out
        self._ck(self.lib.hann_decrypt_scores(self.h, _ptr(s), _ptr(ct), count, ls, _ptr(scores), _ptr(imag)))
        return (scores, imag) if want_imag else scores

    def decrypt_compact(self, s, ct, rescaled, log_scale_in=None, want_imag=False):
        """ct: [count][2][limbs][N] canonical, as produced by compact_scores + export_limbs"""
        s, ct = _np(s, np.int8), _np(ct, np.uint64)
        count, _, limbs, _ = ct.shape
        scores = np.empty((count, self.n), dtype=np.float64)
        imag = np.empty((count, self.n), dtype=np.float64) if want_imag else None
        ls = 2 * self.log_scale if log_scale_in is None else log_scale_in
        self._ck(self.lib.hann_decrypt_compact(self.h, _ptr(s), _ptr(ct), count, limbs, 1 if rescaled else 0, ls, _ptr(scores),
                                               _ptr(imag)))
        return (scores, imag) if want_imag else scores

    # ---- server side
    def load_keys(self, evk, rots):
        rots = _np(rots, np.int32)
        if isinstance(evk, np.ndarray):
            evk = _np(evk, np.uint64)
        self._ck(self.lib.hann_load_keys(self.h, _ptr(evk), len(rots), _ptr(rots)))

    def import_(self, kind, canonical, count):
        if isinstance(canonical, np.ndarray):
            canonical = _np(canonical, np.uint64)
        per = self.sizeof(SIZE_CT if kind == KIND_CT else SIZE_POLY)
        if kind == KIND_PT:
            per //= 2  # stored plaintexts keep half of every transform
        out = self.alloc(per * count)
        self._ck(self.lib.hann_import(self.h, kind, _ptr(canonical), count, _ptr(out)))
        return out

    def export(self, kind, internal, count, offset_bytes=0):
        polys = 2 if kind == KIND_CT else 1
        out = np.empty((count, polys, self.L, self.N), dtype=np.uint64)
        self._ck(self.lib.hann_export(self.h, kind, _ptr(internal) + offset_bytes, count, _ptr(out)))
        return out

    def expand_uniform(self, seed, stream):
        a = np.empty((self.L, self.N), dtype=np.uint64)
        self._ck(self.lib.hann_expand_uniform(self.h, seed, stream, _ptr(a)))
        return a

    def import_seeded_ct(self, c0, seed, stream, out=None):
        """c0 [L][N] canonical + the seed of the uniform half -> internal ciphertext on the device"""
        c0 = _np(c0, np.uint64)
        if out is None:
            out = self.alloc(self.sizeof(SIZE_CT))
        self._ck(self.lib.hann_import_seeded_ct(self.h, _ptr(c0), seed, stream, _ptr(out)))
        return out

    def export_limbs(self, internal, npoly, limbs):
        out = np.empty((npoly, limbs, self.N), dtype=np.uint64)
        self._ck(self.lib.hann_export_limbs(self.h, _ptr(internal), npoly, limbs, _ptr(out)))
        return out

    def compact_scores(self, score, n_blocks, keep, rescale, ws=None, out=None):
        if out is None:
            out = self.alloc(self.lib.hann_compact_bytes(self.h, n_blocks, keep))
        self._ck(self.lib.hann_compact_scores(self.h, _ptr(score), n_blocks, keep, 1 if rescale else 0, _ptr(out), _ptr(ws),
                                              ws.numel() * 8 if ws is not None else 0))
        return out

    def query_prepare(self, ct_dev, ws, baby=None):
        if baby is None:
            baby = self.alloc(self.sizeof(SIZE_BABY))
        self._ck(self.lib.hann_query_prepare(self.h, _ptr(ct_dev), _ptr(baby), _ptr(ws), ws.numel() * 8))
        return baby

    def n_blocks(self, n_rows):
        return (n_rows + self.n - 1) // self.n

    def encode_candidates(self, rows_dev, ws, pt=None):
        n_rows, dim = rows_dev.shape
        assert rows_dev.dtype == self.torch.float32 and rows_dev.is_contiguous()
        if pt is None:
            pt = self.alloc(self.n_blocks(n_rows) * self.sizeof(SIZE_PT_BLOCK))
        self._ck(self.lib.hann_encode_candidates(self.h, _ptr(rows_dev), n_rows, dim, _ptr(pt), _ptr(ws), ws.numel() * 8))
        return pt

    def score_level(self, baby, pt, n_blocks, ws=None, inner=None):
        if inner is None:
            inner = self.alloc(n_blocks * self.sizeof(SIZE_INNER))
        self._ck(self.lib.hann_score_level(self.h, _ptr(baby), _ptr(pt), n_blocks, _ptr(inner), _ptr(ws),
                                           ws.numel() * 8 if ws is not None else 0))
        return inner

    def score_level_ctdb(self, baby, ctdb, n_blocks, ws, inner=None):
        if inner is None:
            inner = self.alloc(n_blocks * self.sizeof(SIZE_INNER))
        self._ck(self.lib.hann_score_level_ctdb(self.h, _ptr(baby), _ptr(ctdb), n_blocks, _ptr(inner), _ptr(ws), ws.numel() * 8))
        return inner

    def score_level_batch(self, babies, n_queries, pt, n_blocks, ws=None, inner=None):
        """babies: the n_queries baby sets back to back; returns inner [query][blk][g]"""
        if inner is None:
            inner = self.alloc(n_queries * n_blocks * self.sizeof(SIZE_INNER))
        self._ck(self.lib.hann_score_level_batch(self.h, _ptr(babies), n_queries, _ptr(pt), n_blocks, _ptr(inner), _ptr(ws),
                                                 ws.numel() * 8 if ws is not None else 0))
        return inner

    def rotate_sum(self, inner, n_blocks, ws, score=None):
        if score is None:
            score = self.alloc(n_blocks * self.sizeof(SIZE_CT))
        self._ck(self.lib.hann_rotate_sum(self.h, _ptr(inner), n_blocks, _ptr(score), _ptr(ws), ws.numel() * 8))
        return score

    def multiply(self, a, b_, count, ws):
        out = self.alloc(count * self.sizeof(SIZE_CT))
        self._ck(self.lib.hann_multiply(self.h, _ptr(a), _ptr(b_), count, _ptr(out), _ptr(ws), ws.numel() * 8))
        return out

    def rotate_sum_lazy(self, inner, n_blocks, ws, score=None):
        if score is None:
            score = self.alloc(n_blocks * self.sizeof(SIZE_CT))
        self._ck(self.lib.hann_rotate_sum_lazy(self.h, _ptr(inner), n_blocks, _ptr(score), _ptr(ws), ws.numel() * 8))
        return score

    def query_level(self, ct_dev, rows_dev, ws, baby=None, pt=None, inner=None, score=None):
        n_rows, dim = rows_dev.shape
        nb = self.n_blocks(n_rows)
        baby = self.alloc(self.sizeof(SIZE_BABY)) if baby is None else baby
        pt = self.alloc(nb * self.sizeof(SIZE_PT_BLOCK)) if pt is None else pt
        inner = self.alloc(nb * self.sizeof(SIZE_INNER)) if inner is None else inner
        score = self.alloc(nb * self.sizeof(SIZE_CT)) if score is None else score
        self._ck(self.lib.hann_query_level(self.h, _ptr(ct_dev), _ptr(rows_dev), n_rows, dim, _ptr(baby), _ptr(pt), _ptr(inner),
                                           _ptr(score), _ptr(ws), ws.numel() * 8))
        return score

    # ---- packed projection
    def rotate_hoisted(self, ct_dev, rot0, count, ws, out=None):
        if out is None:
            out = self.alloc(max(count, 1) * self.sizeof(SIZE_CT))
        self._ck(self.lib.hann_rotate_hoisted(self.h, _ptr(ct_dev), rot0, count, _ptr(out), _ptr(ws), ws.numel() * 8))
        return out

    def encode_slots(self, z_dev, log_scale, ws):
        count = z_dev.shape[0]
        assert z_dev.dtype == self.torch.float64 and z_dev.is_contiguous() and z_dev.shape[1] == self.n
        pt = self.alloc(count * self.sizeof(SIZE_POLY) // 2)
        self._ck(self.lib.hann_encode_slots(self.h, _ptr(z_dev), count, log_scale, _ptr(pt), _ptr(ws), ws.numel() * 8))
        return pt

    def project_enrol(self, W_dev, log_scale_w, ws):
        D, R = W_dev.shape
        assert R == self.R and W_dev.dtype == self.torch.float32 and W_dev.is_contiguous()
        pt = self.alloc(self.sizeof(SIZE_PT_BLOCK))
        self._ck(self.lib.hann_project_enrol(self.h, _ptr(W_dev), D, log_scale_w, _ptr(pt), _ptr(ws), ws.numel() * 8))
        return pt

    def project_masks(self, log_scale_m, ws):
        lo = self.alloc(self.B * self.sizeof(SIZE_POLY) // 2)
        hi = self.alloc(self.B * self.sizeof(SIZE_POLY) // 2)
        self._ck(self.lib.hann_project_masks(self.h, log_scale_m, _ptr(lo), _ptr(hi), _ptr(ws), ws.numel() * 8))
        return lo, hi

    def project_baby(self, ct_dev, lo, hi, ws):
        cyc = self.alloc(self.sizeof(SIZE_BABY))
        self._ck(self.lib.hann_project_baby(self.h, _ptr(ct_dev), _ptr(lo), _ptr(hi), _ptr(cyc), _ptr(ws), ws.numel() * 8))
        return cyc

    def rescale(self, ct_dev, count, ws):
        out = self.alloc(self.lib.hann_compact_bytes(self.h, count, self.L - 1))
        self._ck(self.lib.hann_rescale(self.h, _ptr(ct_dev), count, _ptr(out), _ptr(ws), ws.numel() * 8))
        return out

    def fold(self, ct_dev, stride, steps, ws):
        self._ck(self.lib.hann_fold(self.h, _ptr(ct_dev), stride, steps, _ptr(ws), ws.numel() * 8))
        return ct_dev

    def project_query(self, mid, ct_dev, lo, hi, wpt, D, ws=None):
        """the projected query: one ciphertext of the chain with two primes fewer, [2][L-2][N] internal"""
        if ws is None:
            ws = self.alloc(self.lib.hann_project_bytes(self.h, mid.h))
        out = self.alloc(mid.lib.hann_compact_bytes(mid.h, 1, mid.L - 1))
        self._ck(self.lib.hann_project_query(self.h, mid.h, _ptr(ct_dev), _ptr(lo), _ptr(hi), _ptr(wpt), D, _ptr(out), _ptr(ws),
                                             ws.numel() * 8))
        return out

    def keyswitch(self, rot, poly, ws):
        ks0 = self.alloc(self.sizeof(SIZE_POLY))
        ks1 = self.alloc(self.sizeof(SIZE_POLY))
        self._ck(self.lib.hann_keyswitch(self.h, rot, _ptr(poly), _ptr(ks0), _ptr(ks1), _ptr(ws), ws.numel() * 8))
        return ks0, ks1

    def keyswitch_static(self, rot, poly, ks0=None, ks1=None):
        """hann_keyswitch_static: same result as `keyswitch`, scratch inside the library (no workspace argument).
        The two output polynomials may be passed in so that the call itself allocates nothing."""
        if ks0 is None:
            ks0 = self.alloc(self.sizeof(SIZE_POLY))
        if ks1 is None:
            ks1 = self.alloc(self.sizeof(SIZE_POLY))
        self._ck(self.lib.hann_keyswitch_static(self.h, rot, _ptr(poly), _ptr(ks0), _ptr(ks1)))
        return ks0, ks1

    def level_host_bytes(self, n_rows):
        return int(self.lib.hann_level_host_bytes(self.h, n_rows))

    def score_level_host(self, ct_host, rows_host, ws_dev, out=None):
        """ct_host: uint64 [2][L][N] (numpy or pinned torch), rows_host: float32 [n_rows][dim]; returns the score
        ciphertexts [n_blocks][2][L][N] in host memory."""
        n_rows, dim = rows_host.shape
        nb = self.n_blocks(n_rows)
        if out is None:
            out = np.empty((nb, 2, self.L, self.N), dtype=np.uint64)
        self._ck(self.lib.hann_score_level_host(self.h, _ptr(ct_host), _ptr(rows_host), n_rows, dim, _ptr(out), _ptr(ws_dev),
                                                ws_dev.numel() * 8))
        return out


def membership_decide(arith, scorer, R, deg, sign_iters, log_scale, tau, t_lo, t_hi, coef, ct_dev, pt_dev, n_blocks, want_threshold=False):
    """hann_membership_decide: arith = [context of the first l primes with R = B = 1 for l = 1..L], scorer = the context the
    candidates were encoded on.  Returns (out [n_blocks][2][1][N] device tensor, its scale) and, if asked, the threshold
    ciphertext (device tensor, level, scale)."""
    top = arith[-1]
    L = len(arith)
    handles = (C.c_void_p * L)(*[a.h for a in arith])
    coef = _np(coef, np.float64)
    prm = MembershipParams(R, deg, sign_iters, log_scale, tau, t_lo, t_hi, coef.ctypes.data_as(C.POINTER(C.c_double)))
    need = top.lib.hann_membership_bytes(handles, L, scorer.h, C.byref(prm), n_blocks)
    if need < 0:
        raise HannError(int(need), "hann_membership_bytes: bad argument")
    ws = top.alloc(need)
    out = top.alloc(max(n_blocks, 1) * 2 * top.N * 8)
    out_scale, thr_scale, thr_level = C.c_double(0.0), C.c_double(0.0), C.c_int(0)
    thr = top.alloc(2 * L * top.N * 8) if want_threshold else None
    top._ck(top.lib.hann_membership_decide(handles, L, scorer.h, C.byref(prm), _ptr(ct_dev), _ptr(pt_dev), n_blocks, _ptr(out),
                                           C.byref(out_scale), _ptr(thr), C.byref(thr_level), C.byref(thr_scale), _ptr(ws),
                                           ws.numel() * 8))
    if want_threshold:
        return (out, out_scale.value), (thr, thr_level.value, thr_scale.value)
    return out, out_scale.value
