"""The benchmark configurations at their full sizes, in the launch configuration bench.py times (whole levels per
call): bit-exact conformance against the CPU oracle on the first and last block of a level, the score tolerance on every
scored row, and agreement of the FHE-steered routing with plaintext routing (same top-10 ids, same planted-neighbour
hit) on the synthetic hierarchies."""
import numpy as np
import pytest

from paper_2608_21131_b200 import synth, workloads as wl
from tests.helpers import Pair, make_oracle, rescale_error_bound

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pair16():
    """the production parameter set with the keys of rotations 1..B and, for the lazy order of the giant steps, 2B..(G-1)B
    (key material of a rotation depends on its place in the list, so the first B keys are those of bench.py's key set too)"""
    ps = synth.FULL16
    p = Pair(ps, key_seed=wl.KEY_SEED)
    rots = list(range(1, ps.B + 1)) + [gg * ps.B for gg in range(2, ps.G)]
    km = synth.key_material(ps, wl.KEY_SEED, rots=rots)
    extra = [i for i, r in enumerate(rots) if r > ps.B]
    p.evk_lazy_o = {ps.B: p.evk_o[ps.B - 1]}
    for i in extra:
        p.evk_lazy_o[rots[i]] = p.o.evk_gen(km.s, rots[i], km.evk_a[i], km.evk_e[i])
    evk_extra = p.g.keygen_from_samples(km.s, [rots[i] for i in extra], km.evk_a[extra], km.evk_e[extra])
    assert np.array_equal(evk_extra, np.stack([p.evk_lazy_o[rots[i]] for i in extra]))
    p.g.load_keys(evk_extra, [rots[i] for i in extra])
    return p


class Query:
    """one encrypted query on both sides; the baby set is prepared once and reused by every level"""

    def __init__(self, p, qR, with_oracle=True):
        import torch

        self.p, self.qR, self.torch = p, qR, torch
        ct_o, ct_g = p.query(qR)
        assert np.array_equal(ct_o, ct_g)
        self.ct_o = ct_o
        self.ct_g = ct_g
        self.ct_dev = p.g.import_(p.b.KIND_CT, ct_g, 1)
        self.baby = p.g.query_prepare(self.ct_dev, p.ws)
        self.baby_o = p.o.baby_set(ct_o, p.evk_o) if with_oracle else None

    def score_level(self, rows, oracle_blocks=(), compact=False, one_call=False, host=False, lazy_blocks=()):
        """GPU scores of a level [n_rows]; blocks listed in oracle_blocks are compared bit for bit with the oracle"""
        p, g, b, ps = self.p, self.p.g, self.p.b, self.p.ps
        n_rows = rows.shape[0]
        nb = g.n_blocks(n_rows)
        ws = g.workspace(nb)
        rows_dev = self.torch.from_numpy(np.ascontiguousarray(rows)).to(g.device)
        if one_call:
            # the launch configuration bench.py times: the whole level in one hann_query_level call
            pt, inner, score = (g.alloc(nb * g.sizeof(b.SIZE_PT_BLOCK)), g.alloc(nb * g.sizeof(b.SIZE_INNER)),
                                g.alloc(nb * g.sizeof(b.SIZE_CT)))
            g.query_level(self.ct_dev, rows_dev, ws, self.baby, pt, inner, score)
        else:
            pt = g.encode_candidates(rows_dev, ws)
            inner = g.score_level(self.baby, pt, nb, ws)
            score = g.rotate_sum(inner, nb, ws)
        g.sync()
        score_h = g.export(b.KIND_CT, score, nb)
        for blk in oracle_blocks:
            sc_o, pt_o, in_o = p.o.score_block(rows[blk * ps.n:(blk + 1) * ps.n], self.baby_o, p.evk_o[ps.B - 1], True, True)
            ptw, inw = g.sizeof(b.SIZE_PT_BLOCK), g.sizeof(b.SIZE_INNER)
            pt_g = g.export(b.KIND_PT, pt, ps.R, offset_bytes=blk * ptw).reshape(ps.G, ps.B, ps.L, ps.N)
            in_g = g.export(b.KIND_CT, inner, ps.G, offset_bytes=blk * inw).reshape(ps.G, 2, ps.L, ps.N)
            assert np.array_equal(pt_g, pt_o), "encoded plaintexts of block %d" % blk
            assert np.array_equal(in_g, in_o), "partial sums of block %d" % blk
            assert np.array_equal(score_h[blk], sc_o), "score ciphertext of block %d" % blk
        if lazy_blocks:
            # the giant steps in the order bench.py's headline uses (distinct keys, one ModDown per block): the same partial
            # sums through hann_query_level / hann_rotate_sum with the knob set, against the oracle's evaluation in that order
            giant = np.stack([p.evk_lazy_o[gg * ps.B] for gg in range(1, ps.G)])
            g.set_tuning(b.TUNE_GIANT_LAZY, 1)
            lazy = g.rotate_sum(inner, nb, ws)
            g.sync()
            lazy_h = g.export(b.KIND_CT, lazy, nb)
            for blk in lazy_blocks:
                in_g = g.export(b.KIND_CT, inner, ps.G, offset_bytes=blk * g.sizeof(b.SIZE_INNER)).reshape(ps.G, 2, ps.L, ps.N)
                assert np.array_equal(lazy_h[blk], p.o.rotate_sum_lazy(in_g, giant)), "lazy score ciphertext of block %d" % blk
            got_l = g.decrypt_scores(p.km.s, lazy_h).reshape(-1)[:n_rows]
            assert float(np.abs(got_l - rows.astype(np.float64) @ self.qR.astype(np.float64)).max()) < 2.0 ** ps.tol_log2
            if host:
                ws_host = g.alloc(g.level_host_bytes(n_rows))
                assert np.array_equal(g.score_level_host(self.ct_g, np.ascontiguousarray(rows), ws_host), lazy_h)
                del ws_host
            g.set_tuning(b.TUNE_GIANT_LAZY, 0)
            del lazy
        if host:
            # the end-to-end call bench.py times: host buffers in, block groups scored while later groups upload
            ws_host = g.alloc(g.level_host_bytes(n_rows))
            assert np.array_equal(g.score_level_host(self.ct_g, np.ascontiguousarray(rows), ws_host), score_h)
            del ws_host
        got = g.decrypt_scores(p.km.s, score_h).reshape(-1)[:n_rows]
        want = rows.astype(np.float64) @ self.qR.astype(np.float64)
        err = float(np.abs(got - want).max())
        assert err < 2.0 ** ps.tol_log2, err
        if compact:
            # output compaction at full size: every block bit-identical to the oracle's compaction of the same
            # ciphertext; two limbs without rescale decrypt to identical scores, one limb after the rescale to scores
            # within the Laplace-tail bound of the division's rounding error (sigma = N / 6 / scale)
            two = g.export_limbs(g.compact_scores(score, nb, 2, False), nb * 2, 2).reshape(nb, 2, 2, ps.N)
            one = g.export_limbs(g.compact_scores(score, nb, 1, True, ws), nb * 2, 1).reshape(nb, 2, 1, ps.N)
            for blk in range(nb):
                assert np.array_equal(two[blk], p.o.compact(score_h[blk], 2, False))
                assert np.array_equal(one[blk], p.o.compact(score_h[blk], 1, True))
            assert np.array_equal(g.decrypt_compact(p.km.s, two, False).reshape(-1)[:n_rows], got)
            self.compact_scores = g.decrypt_compact(p.km.s, one, True).reshape(-1)[:n_rows]
            assert np.abs(self.compact_scores - got).max() < rescale_error_bound(ps.N, 2.0 ** (2 * ps.log_scale) / ps.q[-1], n_rows)
        del pt, inner, score
        return got, want


def test_face_like_level_full(pair16):
    """222,049 rows, 512 -> 128 dims, N = 2^16: 7 blocks, the last 77.6 % full.  First and last block at every
    conformance point, every row within 2^-18; the host-buffer call (three block groups) returns the same ciphertexts."""
    ps, lvl, qR, planted = wl.face_level()
    q = Query(pair16, qR)
    got, want = q.score_level(lvl.rows, oracle_blocks=(0, 6), compact=True, host=True, lazy_blocks=(0, 6))
    assert got.shape == (222_049,)
    # a quarter of the bytes on the wire (one limb instead of four) still ranks the same neighbours first
    assert np.array_equal(wl.topk_ids(q.compact_scores, lvl.ids, 10), wl.topk_ids(want, lvl.ids, 10))
    # the planted neighbour is the top score under both rankings
    assert int(np.argmax(got)) == planted == int(np.argmax(want))
    assert np.array_equal(wl.topk_ids(got, lvl.ids, 10), wl.topk_ids(want, lvl.ids, 10))


def route(cfg, q, scorer, memo):
    """coarse -> fine -> rerank with the given scorer(level) -> scores; returns (top-10 row ids, touched rows).  `memo`
    keeps the materialised levels of one query, so that two pipelines that open the same cells generate them once."""
    coarse = wl.coarse_level(cfg) if not hasattr(cfg, "_coarse") else cfg._coarse
    cfg._coarse = coarse
    cells = np.sort(wl.topk_ids(scorer(coarse), coarse.ids, cfg.nprobe))
    key = ("fine", cells.tobytes())
    fine = memo[key] if key in memo else memo.setdefault(key, wl.fine_level(cfg, cells))
    leaves = np.sort(wl.topk_ids(scorer(fine), fine.ids, cfg.leaf_beam))
    key = ("rerank", leaves.tobytes())
    rer = memo[key] if key in memo else memo.setdefault(key, wl.rerank_level(cfg, leaves))
    sc = scorer(rer)
    return wl.topk_ids(sc, rer.ids, 10), (coarse, fine, rer), sc


def same_up_to_near_ties(ids_a, ids_b, scores_by_id, tol):
    if np.array_equal(ids_a, ids_b):
        return True
    # differences are allowed only between scores closer than 2 * tol
    sa = np.array([scores_by_id[i] for i in ids_a])
    sb = np.array([scores_by_id[i] for i in ids_b])
    return set(ids_a) == set(ids_b) or bool(np.abs(np.sort(sa) - np.sort(sb)).max() < 2 * tol)


@pytest.mark.parametrize("name,n_queries", [("datacomp", 16), ("deep1b", 64)])
def test_hierarchy_routing_agrees_with_plaintext(pair16, name, n_queries):
    """The recall protocol at its stated breadth: 16 planted queries on the DataComp-like hierarchy and 64 on the
    Deep1B-like one (Sec. 4.3 compares the encrypted pipeline's recall@10 with plaintext routing on the same index).  For
    every query the FHE-steered pipeline (decrypt, top cells, top leaves, top-10 rows) and the float64 plaintext-steered
    pipeline must open the same cells, return the same top-10 ids (swaps only between scores closer than twice the
    tolerance) and agree on whether the planted neighbour is found; the first query is also checked against the oracle bit
    for bit on the first and last block of every level."""
    cfg = wl.datacomp_like() if name == "datacomp" else wl.deep1b_like()
    ps = cfg.ps
    hits_f = hits_p = 0
    for qi in range(n_queries):
        memo = {}
        qR, planted = wl.hier_query(cfg, qi)
        q = Query(pair16, qR, with_oracle=(qi == 0))

        def fhe(level):
            nb = (len(level.ids) + ps.n - 1) // ps.n
            # first query: first and last block of every level against the oracle
            blocks = sorted({0, nb - 1}) if qi == 0 else ()
            return q.score_level(level.rows, oracle_blocks=blocks)[0]

        def plain(level):
            return level.rows.astype(np.float64) @ qR.astype(np.float64)

        top_p, levels_p, sc_p = route(cfg, q, plain, memo)
        top_f, levels_f, sc_f = route(cfg, q, fhe, memo)
        # both pipelines open the same cells and return the same neighbours
        assert np.array_equal(levels_f[1].ids, levels_p[1].ids) and np.array_equal(levels_f[2].ids, levels_p[2].ids)
        by_id = dict(zip(levels_p[2].ids.tolist(), sc_p.tolist()))
        assert same_up_to_near_ties(top_f, top_p, by_id, 2.0 ** ps.tol_log2)
        assert (planted in top_f) == (planted in top_p)
        assert planted == top_p[0]  # the perturbed copy's nearest row is the planted row (recall@1 of the routing)
        hits_f += int(planted in top_f)
        hits_p += int(planted in top_p)
        if name == "datacomp" and qi == 0:
            assert len(levels_f[0].ids) == 65_536 and len(levels_f[1].ids) == 1_024 and len(levels_f[2].ids) == 97_976
        if name == "deep1b" and qi == 0:
            assert len(levels_f[0].ids) == 1_000 and len(levels_f[1].ids) == 16_000 and len(levels_f[2].ids) == 64_000
    print("%s: planted neighbour in the top 10 of %d/%d FHE-steered and %d/%d plaintext-steered queries"
          % (name, hits_f, n_queries, hits_p, n_queries))
    assert hits_f == hits_p == n_queries


def test_zero_padded_96_dim_rows_score_identically_on_gpu(pair16):
    """the 96 -> 128 zero-pad: rows given with dim = 96 and the same rows padded to 128 by the caller give the same bits"""
    import torch

    p = pair16
    g, b, ps = p.g, p.b, p.ps
    x96 = synth.toy_corpus(3, rows=5000, dim=96)
    x128 = synth.project_rows(x96.astype(np.float64), None, 128)
    pt_a = g.encode_candidates(torch.from_numpy(x96).to(g.device), p.ws)
    pt_b = g.encode_candidates(torch.from_numpy(x128).to(g.device), p.ws)
    g.sync()
    assert torch.equal(pt_a, pt_b)


def test_sweep_level_of_several_blocks_at_ring_2_15():
    """the scaling sweep at N = 2^15 (16,384 rows per block) on a level of several blocks: 2^14 wanted rows inflated x4 to
    2^16 scored rows = 4 blocks; first and last block at every conformance point, every score within 2^-18, and the
    host-buffer call returns the same ciphertexts"""
    ps2, lvl = wl.sweep_level(1 << 14, ps=synth.FULL15)
    assert lvl.rows.shape == (1 << 16, 128)
    p = Pair(synth.FULL15, key_seed=wl.KEY_SEED)
    q = Query(p, synth.toy_query(wl.query_seed(2), dim=128))
    got, want = q.score_level(lvl.rows, oracle_blocks=(0, 3), host=True)
    assert got.shape == (1 << 16,)
    assert np.array_equal(np.argsort(-got)[:10], np.argsort(-want)[:10])


@pytest.mark.parametrize("logN", [15, 16])
def test_sweep_level_with_padding_groups(logN, pair16):
    """scaling-sweep configuration at its smallest size: 2^12 wanted rows inflated x4 by seeded fixed groups to 2^14
    scored rows (one block at N = 2^15, half a block at N = 2^16), dim 128"""
    ps = synth.FULL15 if logN == 15 else synth.FULL16
    ps2, lvl = wl.sweep_level(1 << 12, ps=ps)
    assert lvl.rows.shape == (1 << 14, 128)
    p = pair16 if logN == 16 else Pair(ps, key_seed=wl.KEY_SEED)
    qR = synth.toy_query(wl.query_seed(0), dim=128)
    q = Query(p, qR)
    q.score_level(lvl.rows, oracle_blocks=(0,))


def test_sweep_maximum_size(pair16):
    """the largest point of the scaling sweep, through one hann_query_level call: 2^20 wanted rows inflated to 2^22 scored
    rows = 128 blocks (32 GiB of encoded plaintexts) at N = 2^16; first and last block at every conformance point, all
    4,194,304 scores within 2^-18"""
    ps2, lvl = wl.sweep_level(1 << 20, ps=synth.FULL16)
    assert lvl.rows.shape == (1 << 22, 128)
    q = Query(pair16, synth.toy_query(wl.query_seed(1), dim=128))
    got, want = q.score_level(lvl.rows, oracle_blocks=(0, 127), one_call=True)
    assert got.shape == (1 << 22,)
    assert np.array_equal(np.argsort(-got)[:10], np.argsort(-want)[:10])


def test_projection_under_encryption_then_scoring():
    """Rank reduction under encryption (Sec. 3.1 "How"), in this build's plaintext-resident variant: the server holds the
    512 -> 128 projection W in plaintext and applies it to the encrypted 512-dimensional query with the same diagonal
    baby-step/giant-step scorer -- the "candidate block" is W^T tiled down the n slots, so slot i of the result holds
    q_R[i mod 128], i.e. the projected query already tiled for the scoring levels.  The projected ciphertext (scale
    Delta^2) is then used as the query of an ordinary level (result at scale Delta^3).  Both stages are compared with the
    oracle bit for bit, the final scores with float64 within 2^-18."""
    import torch

    ps512 = synth.ParamSet("proj", 13, synth.Q50, synth.P60, 40, 512, 32, -18)
    ps128 = ps512.with_(R=128)
    pp, pc = Pair(ps512, key_seed=4), Pair(ps128, key_seed=4)
    assert np.array_equal(pp.evk_g, pc.evk_g)  # same client, same keys: rotations 1..32 serve both stages
    n = ps512.n
    W = synth.projection_matrix(wl.PROJ_SEED, 512, 128)
    q512 = synth.normalise(synth.gaussian_vectors(9, synth.S_QUERY, np.arange(1), 512))[0].astype(np.float32)
    WT = np.ascontiguousarray(W.T.astype(np.float32))                 # [128][512]
    block = np.ascontiguousarray(np.tile(WT, (n // 128, 1)))          # row i = W^T[i mod 128]
    # stage 1: projection
    ct_o, ct_g = pp.query(q512)
    assert np.array_equal(ct_o, ct_g)
    g, b = pp.g, pp.b
    baby = g.query_prepare(g.import_(b.KIND_CT, ct_g, 1), pp.ws)
    pt = g.encode_candidates(torch.from_numpy(block).to(g.device), pp.ws)
    proj = g.rotate_sum(g.score_level(baby, pt, 1, pp.ws), 1, pp.ws)
    g.sync()
    proj_o, _, _ = pp.o.score_block(block, pp.o.baby_set(ct_o, pp.evk_o), pp.evk_o[31])
    assert np.array_equal(g.export(b.KIND_CT, proj, 1)[0], proj_o)
    qR = (WT.astype(np.float64) @ q512.astype(np.float64))
    slots = g.decrypt_scores(pp.km.s, proj_o[None], log_scale_out=80)[0]
    assert np.abs(slots - np.tile(qR, n // 128)).max() < 2.0 ** -20
    # stage 2: an ordinary level with the projected ciphertext as its query (same ring, same keys, R = 128)
    rows = synth.project_rows(synth.toy_corpus(7, rows=n + 500, dim=512).astype(np.float64), W, 128)
    g2 = pc.g
    baby2 = g2.query_prepare(proj, pc.ws)   # the device ciphertext of stage 1 is the query of stage 2
    pt2 = g2.encode_candidates(torch.from_numpy(rows).to(g2.device), pc.ws)
    score = g2.rotate_sum(g2.score_level(baby2, pt2, 2, pc.ws), 2, pc.ws)
    g2.sync()
    score_g = g2.export(b.KIND_CT, score, 2)
    baby2_o = pc.o.baby_set(proj_o, pc.evk_o)
    for blk in range(2):
        sc_o, _, _ = pc.o.score_block(rows[blk * n:(blk + 1) * n], baby2_o, pc.evk_o[31])
        assert np.array_equal(score_g[blk], sc_o)
    got = g2.decrypt_scores(pc.km.s, score_g, log_scale_out=120).reshape(-1)[: rows.shape[0]]
    want = rows.astype(np.float64) @ qR
    assert np.abs(got - want).max() < 2.0 ** -18


@pytest.mark.parametrize("logN,D,R,B,B_score,lazy", [(13, 512, 128, 4, 32, False), (12, 128, 32, 8, 8, True), (16, 512, 128, 8, 32, False)])
def test_packed_projection_then_scoring(logN, D, R, B, B_score, lazy):
    """Rank reduction with the matrix packed by windows (Sec. 3.1 Detail): masks, packed diagonals, the in-window baby
    rotations after their rescale and the projected query are each compared with the oracle bit for bit; the projected
    query (two primes fewer, scale back at ~2^40) then serves an ordinary scoring level on the shorter chain, again bit
    for bit, with scores inside 2^-18 of the float64 products.  512 -> 128 at N = 2^13 and at N = 2^16."""
    import torch

    from oracle.oracle import PackedProjection, restrict_keys
    from paper_2608_21131_b200 import binding as b

    q, p, L = synth.Q50, synth.P60, 4
    pp = PackedProjection(logN, q, p, 40, D, R, B, 50, 50)
    n, N = pp.n, pp.N
    ps_top = synth.ParamSet("top", logN, q, p, 40, R, B, -18)
    top, mid = b.Context(ps_top), b.Context(ps_top.with_(q=q[:3]))
    ps_low = ps_top.with_(q=q[:2], B=B_score)
    low = b.Context(ps_low)
    giant = [g * B for g in range(1, pp.G)] if lazy else [B]
    rots_top = pp.baby_rotations()
    rots_mid = sorted(set(giant) | set(pp.fold_rotations()))
    rots_low = list(range(1, B_score + 1))
    rots = sorted(set(rots_top) | set(rots_mid) | set(rots_low))
    km = synth.key_material(ps_top, 61, rots=rots)
    evk = top.keygen_from_samples(km.s, km.rots, km.evk_a, km.evk_e)       # the client's keys, longest chain
    evk_o = dict(zip(rots, helpers_keys(pp.top, km)))
    assert np.array_equal(evk, np.stack([evk_o[r] for r in rots]))
    pick = lambda want: np.stack([evk[rots.index(r)] for r in want])
    top.load_keys(pick(rots_top), rots_top)
    mid.load_keys(b.restrict_keys(pick(rots_mid), L, 3), rots_mid)
    low.load_keys(b.restrict_keys(pick(rots_low), L, 2), rots_low)
    assert np.array_equal(b.restrict_keys(pick(rots_mid), L, 3), restrict_keys(pick(rots_mid), L, 3))
    if lazy:
        mid.set_tuning(b.TUNE_GIANT_LAZY, 1)
    rng = np.random.default_rng(5)
    W = np.linalg.qr(rng.standard_normal((D, R)))[0].astype(np.float32)
    qv = rng.standard_normal(D)
    qv = (qv / np.linalg.norm(qv)).astype(np.float32)
    # enrolment: masks on the top chain, packed matrix on the middle chain
    ws_top, ws_mid = top.workspace(1), mid.workspace(1)
    lo, hi = top.project_masks(50, ws_top)
    wpt = mid.project_enrol(torch.from_numpy(W).to(mid.device), 50, ws_mid)
    lo_o, hi_o = pp.mask_plaintexts()
    assert np.array_equal(top.export(b.KIND_PT, lo, B).reshape(B, L, N), lo_o)
    assert np.array_equal(top.export(b.KIND_PT, hi, B).reshape(B, L, N), hi_o)
    wpt_o = pp.enrol(W.astype(np.float64))
    assert np.array_equal(mid.export(b.KIND_PT, wpt, R).reshape(pp.G, B, 3, N), wpt_o)
    # the query: q tiled with period D (a "dimension D" query of a context whose R is D would do the same)
    ct = pp.top.encrypt(km.s, pp.top.encode(pp.query_slots(qv)), km.ct_a, km.ct_e)
    ct_dev = top.import_(b.KIND_CT, ct, 1)
    wsp = top.alloc(top.lib.hann_project_bytes(top.h, mid.h))
    cyc = top.rescale(top.project_baby(ct_dev, lo, hi, wsp), B, wsp)
    top.sync()
    cyc_o = pp.in_window_rotations(ct, evk_o)
    assert np.array_equal(top.export_limbs(cyc, 2 * B, 3).reshape(B, 2, 3, N), cyc_o)
    out = top.project_query(mid, ct_dev, lo, hi, wpt, D, wsp)
    top.sync()
    out_o = pp.project(ct, evk_o, wpt_o, lazy=lazy)
    assert np.array_equal(mid.export_limbs(out, 2, 2).reshape(2, 2, N), out_o)
    want_q = W.T.astype(np.float64) @ qv.astype(np.float64)
    slots = pp.low.decode(np.array([float(v) for v in pp.low.decrypt_int(km.s, out_o)]), pp.scale_out).real
    assert np.abs(slots - np.tile(want_q, n // R)).max() < 2.0 ** -20
    # an ordinary level on the shortest chain with the projected ciphertext as its query
    rows = synth.project_rows(synth.toy_corpus(7, rows=n + 300, dim=D).astype(np.float64), W.astype(np.float64), R)
    ws_low = low.workspace(2)
    baby = low.query_prepare(out, ws_low)
    score = low.rotate_sum(low.score_level(baby, low.encode_candidates(torch.from_numpy(rows).to(low.device), ws_low), 2, ws_low), 2, ws_low)
    low.sync()
    score_g = low.export(b.KIND_CT, score, 2)
    o_low = make_oracle(ps_low)
    evk_low = restrict_keys(np.stack([evk_o[r] for r in rots_low]), L, 2)
    baby_o = o_low.baby_set(out_o, evk_low)
    for blk in range(2):
        sc_o, _, _ = o_low.score_block(rows[blk * n:(blk + 1) * n], baby_o, evk_low[B_score - 1])
        assert np.array_equal(score_g[blk], sc_o), blk
    got = low.decrypt_scores(km.s, score_g, log_scale_out=80).reshape(-1)[: rows.shape[0]] * (2.0 ** 40 / pp.scale_out)
    assert np.abs(got - rows.astype(np.float64) @ want_q).max() < 2.0 ** -18


def helpers_keys(o, km):
    return [o.evk_gen(km.s, r, km.evk_a[i], km.evk_e[i]) for i, r in enumerate(km.rots)]


def test_projection_with_encrypted_matrix():
    """Rank reduction as the paper deploys it (Sec. 3.1 "How": the server holds W as ENCRYPTED diagonals, so that it never
    learns the projection): the same diagonal scorer with the encrypted block of W^T (ct x ct multiply-accumulate, one
    relinearisation per giant step, rotate-and-sum).  Bit-identical to the oracle; the slots of the result hold the
    projected query, tiled.  (Here W^T is stored as one 512-diagonal block; the window-packed form with its 0/1 masks
    and single fold, matrix in plaintext, is test_packed_projection_then_scoring.)"""
    import torch

    ps = synth.ParamSet("proj", 13, synth.Q50, synth.P60, 40, 512, 32, -18)
    p = Pair(ps, key_seed=4)
    g, o, b, n = p.g, p.o, p.b, ps.n
    ka = synth.uniform_residues(78, 50, list(ps.q) + [ps.p], ps.N, lead=(ps.L,))
    ke = synth.rounded_gaussian(78, 51, (ps.L, ps.N))
    rlk_o = o.rlk_gen(p.km.s, ka, ke)
    rlk_g = g.keygen_relin_from_samples(p.km.s, ka, ke)
    assert np.array_equal(rlk_g, rlk_o)
    g.load_keys(rlk_g[None], [0])
    W = synth.projection_matrix(wl.PROJ_SEED, 512, 128)
    WT = np.ascontiguousarray(W.T.astype(np.float32))
    block = np.ascontiguousarray(np.tile(WT, (n // 128, 1)))
    q512 = synth.normalise(synth.gaussian_vectors(9, synth.S_QUERY, np.arange(1), 512))[0].astype(np.float32)
    ct_o, ct_g = p.query(q512)
    baby = g.query_prepare(g.import_(b.KIND_CT, ct_g, 1), p.ws)
    baby_o = o.baby_set(ct_o, p.evk_o)
    # enrolment of W: encode its diagonals, encrypt them under the client's key
    pt = g.encode_candidates(torch.from_numpy(block).to(g.device), p.ws)
    a = synth.uniform_residues(300, 40, list(ps.q), ps.N, lead=(ps.R,))
    e = synth.rounded_gaussian(300, 41, (ps.R, ps.N))
    wdb = g.encrypt_block(p.km.s, pt, a, e)
    wdb_o = o.encrypt_block(p.km.s, o.encode_block(block), a, e)
    # projection under encryption, matrix and query both encrypted
    inner = g.score_level_ctdb(baby, wdb, 1, p.ws)
    proj = g.rotate_sum(inner, 1, p.ws)
    g.sync()
    d = o.mac_ct(wdb_o, baby_o)
    proj_o = o.rotate_sum(np.stack([o.relin(d[gi], rlk_o) for gi in range(ps.G)]), p.evk_o[31])
    assert np.array_equal(g.export(b.KIND_CT, proj, 1)[0], proj_o)
    qR = WT.astype(np.float64) @ q512.astype(np.float64)
    slots = g.decrypt_scores(p.km.s, proj_o[None], log_scale_out=80)[0]
    assert np.abs(slots - np.tile(qR, n // 128)).max() < 2.0 ** -20
