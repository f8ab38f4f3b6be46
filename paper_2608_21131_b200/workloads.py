"""The five benchmark configurations as concrete synthetic inputs (stand-ins for the paper's face corpus,
DataComp-1B and Deep1B, Sec. 4, which are not available offline).  Each builder returns plain numpy arrays:
projected, renormalised, zero-padded float32 candidate rows per routing level and float32 queries.  No scoring
arithmetic lives here; the float64 "plaintext routing" helpers are the client-side ranking the paper describes
(Sec. 2, The round trip: the client decrypts, ranks and chooses the next cells).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import synth

CORPUS_SEED, PROJ_SEED, KEY_SEED, PAD_SEED = 2608, 21131, 1, 7


def query_seed(i: int) -> int:
    return 1000 + i


@dataclass
class Level:
    name: str
    ids: np.ndarray  # candidate ids in the order they are scored (row blk*n+i <-> slot i of block blk)
    rows: np.ndarray  # float32 [len(ids)][R]


# ------------------------------------------------------------------------------------------------ config 0: toy


def toy(seed_corpus=1, seed_query=2):
    return synth.TOY, synth.toy_corpus(seed_corpus), synth.toy_query(seed_query)


# ------------------------------------------------------------------------------------------------ config 1: face-like


def face_level(rows: int = 222_049, chunk: int = 16_384, ps=synth.FULL16):
    """222,049 centroids of dimension 512 from a mixture of 2,048 Gaussians (sigma 0.15), renormalised, projected
    512 -> 128 by a seeded orthonormal map, renormalised, float32.  The query is a perturbed copy of a planted row,
    projected the same way (not renormalised: the client divides by |q_R| after decryption)."""
    fm = synth.FlatMixture(seed=CORPUS_SEED, rows=rows)
    W = synth.projection_matrix(PROJ_SEED, fm.dim, ps.R)
    out = np.empty((rows, ps.R), dtype=np.float32)
    for lo in range(0, rows, chunk):
        ids = np.arange(lo, min(rows, lo + chunk))
        out[lo:lo + len(ids)] = synth.project_rows(fm.vectors(ids), W, ps.R)
    planted = rows // 3
    x = fm.vectors(np.array([planted]))[0]
    q = synth.normalise(x + 0.01 * synth.gaussian_vectors(query_seed(0), synth.S_QUERY, np.arange(1), fm.dim)[0])
    qR = (q @ W).astype(np.float32)
    return ps, Level("flat", np.arange(rows), out), qR, planted


# ------------------------------------------------------------------------------------------------ configs 2, 3: hierarchies


@dataclass
class HierConfig:
    name: str
    ps: synth.ParamSet
    h: synth.Hierarchy
    W: object  # projection matrix or None (zero-pad)
    nprobe: int  # coarse cells opened
    leaf_beam: int  # fine cells opened


def datacomp_like():
    """virtual 65,536 x 64 x 331 = 1.39e9 rows of dimension 512, projected to 128; coarse level scores all 65,536
    centroids, fine level 64 x top-16 cells, rerank the rows of the top-296 fine cells (97,976 rows, ~100k)."""
    h = synth.Hierarchy(seed=CORPUS_SEED, dim=512, n_coarse=65_536, fan=64, leaf=331)
    return HierConfig("datacomp-like", synth.FULL16, h, synth.projection_matrix(PROJ_SEED, 512, 128), 16, 296)


def deep1b_like():
    """virtual 1000 x 1000 x 1000 = 1e9 rows of dimension 96 zero-padded to 128; levels 1,000 / 16,000 / 64,000."""
    h = synth.Hierarchy(seed=CORPUS_SEED, dim=96, n_coarse=1000, fan=1000, leaf=1000)
    return HierConfig("deep1b-like", synth.FULL16, h, None, 16, 64)


def hier_project(cfg: HierConfig, x: np.ndarray) -> np.ndarray:
    return synth.project_rows(x, cfg.W, cfg.ps.R)


def hier_query(cfg: HierConfig, i: int):
    """query i: a perturbed copy of a planted row (true nearest neighbour known); returns (q_R float32, row id)"""
    h = cfg.h
    planted = int(synth.hash64(query_seed(i), synth.S_QUERY, np.arange(1))[0] % np.uint64(h.n_rows))
    q = h.query_near(planted, query_seed(i))
    if cfg.W is not None:
        qR = (q @ cfg.W).astype(np.float32)
    else:
        qR = np.zeros(cfg.ps.R, dtype=np.float32)
        qR[: h.dim] = q.astype(np.float32)
    return qR, planted


def coarse_level(cfg: HierConfig, chunk: int = 8192) -> Level:
    h = cfg.h
    out = np.empty((h.n_coarse, cfg.ps.R), dtype=np.float32)
    for lo in range(0, h.n_coarse, chunk):
        ids = np.arange(lo, min(h.n_coarse, lo + chunk))
        out[lo:lo + len(ids)] = hier_project(cfg, h.coarse(ids))
    return Level("coarse", np.arange(h.n_coarse), out)


def fine_level(cfg: HierConfig, cells) -> Level:
    """fine centroids under the given coarse cells"""
    cells = np.asarray(cells, dtype=np.int64)
    ids = (cells[:, None] * cfg.h.fan + np.arange(cfg.h.fan)[None, :]).ravel()
    return Level("fine", ids, hier_project(cfg, cfg.h.fine(ids)))


def rerank_level(cfg: HierConfig, fine_cells, chunk: int = 16_384) -> Level:
    fine_cells = np.asarray(fine_cells, dtype=np.int64)
    ids = (fine_cells[:, None] * cfg.h.leaf + np.arange(cfg.h.leaf)[None, :]).ravel()
    out = np.empty((len(ids), cfg.ps.R), dtype=np.float32)
    for lo in range(0, len(ids), chunk):
        out[lo:lo + chunk] = hier_project(cfg, cfg.h.rows(ids[lo:lo + chunk]))
    return Level("rerank", ids, out)


def topk_ids(scores: np.ndarray, ids: np.ndarray, k: int) -> np.ndarray:
    """higher score first, ties by lower id"""
    order = np.lexsort((ids, -scores))
    return ids[order[:k]]


# ------------------------------------------------------------------------------------------------ config 4: sweep


def sweep_level(base_rows: int, ps=synth.FULL16, cell: int = 256, group: int = 4):
    """dim-128 clustered rows in cells of `cell` rows; the wanted cells are inflated x`group` by seeded fixed
    anonymity groups (Sec. 5, padding defences), so base_rows wanted rows become group*base_rows scored rows."""
    n_cells_total = max(4 * group * (base_rows // cell), group)
    pi = synth.padding_groups(PAD_SEED, n_cells_total, group)
    order = np.argsort(pi, kind="stable")
    # wanted cells: one per anonymity group so that the inflation is exactly x group
    wanted = order[np.arange(base_rows // cell) * group]
    fetched = synth.padded_fetch(pi, wanted, group)
    h = synth.Hierarchy(seed=CORPUS_SEED, dim=128, n_coarse=max(n_cells_total // 64, 1), fan=64, leaf=cell)
    ids = (fetched[:, None] * cell + np.arange(cell)[None, :]).ravel()
    out = np.empty((len(ids), ps.R), dtype=np.float32)
    for lo in range(0, len(ids), 16_384):
        out[lo:lo + 16_384] = synth.project_rows(h.rows(ids[lo:lo + 16_384]), None, ps.R)
    return ps, Level("sweep", ids, out)
