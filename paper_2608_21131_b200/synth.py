"""Seeded synthetic inputs shared by the tests, the benchmark, the CUDA path and the CPU oracle.

This module holds no arithmetic of the scoring method itself: only a counter-based hash generator,
the samplers built on it (uniform, Gaussian, ternary, rounded Gaussian, uniform residues), the
parameter sets (literal primes) and the synthetic corpora that stand in for the paper's datasets
(Sec. 4: a 222,049-centroid face corpus, DataComp-1B, Deep1B), which are not available offline.
Corpora are *virtual*: a vector is a pure function of (seed, stream, id), so a billion-row corpus is
never materialised; only the rows a routing level fetches are generated.

The generator is non-cryptographic and meant for benchmarks and tests only.
"""
from __future__ import annotations

from dataclasses import dataclass, field
import numpy as np

_M1 = np.uint64(0x9E3779B97F4A7C15)
_M2 = np.uint64(0xBB67AE8584CAA73B)

# stream ids
S_COARSE, S_FINE, S_ROWS, S_QUERY, S_PROJ, S_ASSIGN, S_PAD, S_KEY = 0, 1, 2, 3, 4, 5, 6, 16


def _mix(x: np.ndarray) -> np.ndarray:
    x = x ^ (x >> np.uint64(32))
    x = x * _M1
    x = x ^ (x >> np.uint64(29))
    x = x * _M2
    x = x ^ (x >> np.uint64(32))
    return x


def hash64(seed: int, stream: int, ctr) -> np.ndarray:
    """h(seed, stream, ctr) for an array of 64-bit counters (arithmetic mod 2^64)."""
    with np.errstate(over="ignore"):
        ctr = np.asarray(ctr, dtype=np.uint64)
        a = _mix(np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + _M1)
        b = _mix(a ^ (np.uint64(stream) * _M2))
        return _mix(b + ctr * _M1)


def uniform(seed: int, stream: int, ctr) -> np.ndarray:
    """uniform in [0,1) with 53 random bits"""
    return (hash64(seed, stream, ctr) >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)


def gaussian(seed: int, stream: int, ctr) -> np.ndarray:
    """standard normal by Box-Muller; the two uniforms come from sub-streams 2*stream and 2*stream+1
    of a seed-derived generator, so every (seed, stream, ctr) gives one independent variate."""
    u1 = uniform(seed, 2 * stream + 1000, ctr)
    u2 = uniform(seed, 2 * stream + 1001, ctr)
    return np.sqrt(-2.0 * np.log(1.0 - u1)) * np.cos(2.0 * np.pi * u2)


def gaussian_vectors(seed: int, stream: int, ids, dim: int) -> np.ndarray:
    """float64 [len(ids)][dim]; coordinate c of vector id uses counter id*dim + c."""
    ids = np.asarray(ids, dtype=np.uint64)
    with np.errstate(over="ignore"):
        ctr = ids[:, None] * np.uint64(dim) + np.arange(dim, dtype=np.uint64)[None, :]
    return gaussian(seed, stream, ctr)


def normalise(x: np.ndarray) -> np.ndarray:
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


# ----------------------------------------------------------------------------- parameter sets


@dataclass(frozen=True)
class ParamSet:
    """Ring 2^logN; ciphertext primes q (each 1 mod 2N), one special prime p; scale 2^log_scale;
    padded dimension R; baby-step count B (giant steps G = R/B)."""

    name: str
    logN: int
    q: tuple
    p: int
    log_scale: int
    R: int
    B: int
    tol_log2: int  # decrypted-score tolerance: |score - float64 dot| <= 2^tol_log2

    @property
    def N(self):
        return 1 << self.logN

    @property
    def n(self):
        return 1 << (self.logN - 1)

    @property
    def L(self):
        return len(self.q)

    @property
    def G(self):
        return self.R // self.B

    def with_(self, **kw):
        d = dict(name=self.name, logN=self.logN, q=self.q, p=self.p, log_scale=self.log_scale, R=self.R, B=self.B,
                 tol_log2=self.tol_log2)
        d.update(kw)
        return ParamSet(**d)


# The L largest primes below 2^50 that are 1 mod 2^17 (valid for N = 2^15 and 2^16), the largest
# such prime below 2^60; the toy set likewise below 2^30 / 2^31 with 1 mod 2^13.
Q50 = (1125899903827969, 1125899902124033, 1125899887312897, 1125899886395393)
P60 = 1152921504606584833
Q30 = (1073692673, 1073668097)
P31 = 2147377153

TOY = ParamSet("toy", 12, Q30, P31, 25, 64, 8, -10)
FULL16 = ParamSet("n16", 16, Q50, P60, 40, 128, 32, -18)
FULL15 = ParamSet("n15", 15, Q50, P60, 40, 128, 32, -18)


def small_params(logN: int, R: int, B: int, L: int = 2, log_scale: int = 25, big: bool = False) -> ParamSet:
    """Small rings for fast tests.  All listed primes are 1 mod 2^17, hence valid for every logN <= 16."""
    if big:
        return ParamSet("small-big", logN, Q50[:L], P60, log_scale, R, B, -18)
    # 30/31-bit primes that are 1 mod 2^13 only reach logN <= 12
    assert logN <= 12
    return ParamSet("small", logN, Q30[:L], P31, log_scale, R, B, -10)


# ----------------------------------------------------------------------------- key / encryption material


def ternary(seed: int, stream: int, N: int) -> np.ndarray:
    return (hash64(seed, stream, np.arange(N)) % np.uint64(3)).astype(np.int8) - np.int8(1)


def rounded_gaussian(seed: int, stream: int, shape, sigma: float = 3.2) -> np.ndarray:
    cnt = int(np.prod(shape))
    g = gaussian(seed, stream, np.arange(cnt))
    return np.rint(g * sigma).astype(np.int8).reshape(shape)


def uniform_residues(seed: int, stream: int, mods, N: int, lead=()) -> np.ndarray:
    """uint64 [*lead][len(mods)][N], entry uniform in [0, mods[i]) (up to a 2^-4 relative hash bias)."""
    lead = tuple(lead)
    nl = len(mods)
    cnt = int(np.prod(lead, dtype=np.int64)) if lead else 1
    out = np.empty((cnt, nl, N), dtype=np.uint64)
    base = np.arange(N, dtype=np.uint64)
    for c in range(cnt):
        for i, q in enumerate(mods):
            with np.errstate(over="ignore"):
                ctr = np.uint64((c * nl + i) * N) + base
            out[c, i] = hash64(seed, stream, ctr) % np.uint64(q)
    return out.reshape(lead + (nl, N))


@dataclass
class KeyMaterial:
    """All random draws one client needs, as arrays: ternary secret s[N]; for each rotation r in `rots`
    the uniform a[L][L+1][N] and errors e[L][N] of its evaluation key; the query's a[L][N] and e[N]."""

    s: np.ndarray
    rots: list
    evk_a: np.ndarray  # [n_rot][L][L+1][N]
    evk_e: np.ndarray  # [n_rot][L][N]
    ct_a: np.ndarray  # [L][N]
    ct_e: np.ndarray  # [N]


def key_material(ps: ParamSet, seed: int, rots=None, zero_noise: bool = False) -> KeyMaterial:
    """rots defaults to 1..B (baby rotations 1..B-1 and the giant/Horner rotation B)."""
    if rots is None:
        rots = list(range(1, ps.B + 1))
    N, L = ps.N, ps.L
    mods = list(ps.q) + [ps.p]
    s = ternary(seed, S_KEY, N)
    nr = len(rots)
    evk_a = uniform_residues(seed, S_KEY + 1, mods, N, lead=(nr, L))
    ct_a = uniform_residues(seed, S_KEY + 3, list(ps.q), N)
    if zero_noise:
        evk_e = np.zeros((nr, L, N), dtype=np.int8)
        ct_e = np.zeros(N, dtype=np.int8)
    else:
        evk_e = rounded_gaussian(seed, S_KEY + 2, (nr, L, N))
        ct_e = rounded_gaussian(seed, S_KEY + 4, (N,))
    return KeyMaterial(s, list(rots), evk_a, evk_e, ct_a, ct_e)


# ----------------------------------------------------------------------------- corpora


def projection_matrix(seed: int, d_in: int, d_out: int) -> np.ndarray:
    """Seeded random orthonormal d_in -> d_out projection (columns orthonormal): QR of a Gaussian."""
    a = gaussian_vectors(seed, S_PROJ, np.arange(d_in), d_out)
    qm, r = np.linalg.qr(a)
    return qm * np.sign(np.diag(r))[None, :]


def project_rows(x: np.ndarray, W, R: int) -> np.ndarray:
    """client/enrolment side: project (or zero-pad) to R dims, renormalise, float32."""
    if W is not None:
        y = normalise(x @ W)
    else:
        y = x
    out = np.zeros((y.shape[0], R), dtype=np.float32)
    out[:, : y.shape[1]] = y.astype(np.float32)
    return out


def toy_corpus(seed: int, rows: int = 4096, dim: int = 64) -> np.ndarray:
    """i.i.d. Gaussian rows normalised to unit norm, float32 (toy configuration)."""
    return normalise(gaussian_vectors(seed, S_ROWS, np.arange(rows), dim)).astype(np.float32)


def toy_query(seed: int, dim: int = 64) -> np.ndarray:
    return normalise(gaussian_vectors(seed, S_QUERY, np.arange(1), dim))[0].astype(np.float32)


@dataclass
class FlatMixture:
    """Face-corpus-like flat level: `rows` vectors of dimension `dim` drawn from a mixture of `k`
    Gaussians (per-coordinate sigma around unit-norm means), renormalised."""

    seed: int = 2608
    rows: int = 222_049
    dim: int = 512
    k: int = 2048
    sigma: float = 0.15

    def means(self, ks) -> np.ndarray:
        return normalise(gaussian_vectors(self.seed, S_COARSE, ks, self.dim))

    def assignment(self, ids) -> np.ndarray:
        return (hash64(self.seed, S_ASSIGN, ids) % np.uint64(self.k)).astype(np.int64)

    def vectors(self, ids) -> np.ndarray:
        ids = np.asarray(ids, dtype=np.int64)
        k = self.assignment(ids)
        uk, inv = np.unique(k, return_inverse=True)
        mu = self.means(uk)[inv]
        return normalise(mu + self.sigma * gaussian_vectors(self.seed, S_ROWS, ids, self.dim))


@dataclass
class Hierarchy:
    """Two-level virtual Gaussian-mixture corpus: `n_coarse` unit-norm coarse means, `fan` fine means
    under each, `leaf` rows under each fine mean.  row id = (coarse*fan + fine)*leaf + j."""

    seed: int = 2608
    dim: int = 512
    n_coarse: int = 65_536
    fan: int = 64
    leaf: int = 331
    sigma_fine: float = 0.05
    sigma_row: float = 0.03

    @property
    def n_rows(self):
        return self.n_coarse * self.fan * self.leaf

    def coarse(self, cs) -> np.ndarray:
        return normalise(gaussian_vectors(self.seed, S_COARSE, cs, self.dim))

    def fine(self, fs) -> np.ndarray:
        """fine-cell ids fs = coarse*fan + f"""
        fs = np.asarray(fs, dtype=np.int64)
        c = fs // self.fan
        uc, inv = np.unique(c, return_inverse=True)
        mu = self.coarse(uc)[inv]
        return normalise(mu + self.sigma_fine * gaussian_vectors(self.seed, S_FINE, fs, self.dim))

    def rows(self, ids) -> np.ndarray:
        ids = np.asarray(ids, dtype=np.int64)
        f = ids // self.leaf
        uf, inv = np.unique(f, return_inverse=True)
        nu = self.fine(uf)[inv]
        return normalise(nu + self.sigma_row * gaussian_vectors(self.seed, S_ROWS, ids, self.dim))

    def query_near(self, row_id: int, qseed: int, eps: float = 0.01) -> np.ndarray:
        """a perturbed copy of a planted row: its true nearest neighbour is known without a full scan"""
        x = self.rows(np.array([row_id]))[0]
        return normalise(x + eps * gaussian_vectors(qseed, S_QUERY, np.arange(1), self.dim)[0])


def padding_groups(seed: int, n_cells: int, group: int) -> np.ndarray:
    """Seeded fixed anonymity groups (Sec. 5, padding defences): a seeded permutation pi of the cell
    ids; cell r belongs to the group of the `group` cells whose pi-rank shares floor(pi(r)/group).
    Returns pi (int64[n_cells]); see `padded_fetch`."""
    keys = hash64(seed, S_PAD, np.arange(n_cells))
    order = np.argsort(keys, kind="stable")  # order[rank] = cell
    pi = np.empty(n_cells, dtype=np.int64)
    pi[order] = np.arange(n_cells)
    return pi


def padded_fetch(pi: np.ndarray, wanted, group: int) -> np.ndarray:
    """O = union of g(r) over the wanted cells r, de-duplicated, ascending id."""
    order = np.argsort(pi, kind="stable")
    wanted = np.asarray(wanted, dtype=np.int64)
    gids = np.unique(pi[wanted] // group)
    ranks = (gids[:, None] * group + np.arange(group)[None, :]).ravel()
    ranks = ranks[ranks < len(pi)]
    return np.unique(order[ranks])
