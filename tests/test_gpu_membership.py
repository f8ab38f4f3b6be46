"""The membership (threshold) circuit on the GPU (hann_membership_decide: Sec. 3.1 "The norm problem", Sec. 2 depth 11)
against the CPU oracle's evaluation of the same circuit (oracle/membership.py), ciphertext bits included: the threshold
ciphertext five levels down and the decision ciphertext on the last prime of a chain of 12."""
import numpy as np
import pytest

from oracle import membership as mb
from oracle.oracle import restrict_keys
from paper_2608_21131_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("logN,R,B,deg,iters,n_rows", [(10, 16, 4, 7, 3, 900), (9, 8, 2, 3, 1, 200), (9, 8, 2, 3, 2, 2500), (12, 32, 8, 7, 3, 2048),
                          (15, 128, 32, 7, 3, 16000)])   # the last: the ring, rank and baby steps of the benchmark's scan, one ragged block
def test_membership_circuit_bit_exact(logN, R, B, deg, iters, n_rows):
    import torch

    from paper_2608_21131_b200 import binding as b

    tau = 0.45
    m = mb.Membership(logN, R, tau, deg=deg, sign_iters=iters, B=B)
    ev = m.ev
    q, p, L = ev.q, ev.p, ev.L
    assert (L == 12 and m.depth == 11) if (deg, iters) == (7, 3) else L == m.depth + 1
    lv = np.zeros(2, dtype=np.int32)
    lib = b.load_library()
    assert lib.hann_membership_levels(deg, iters, lv[0:].ctypes.data, lv[1:].ctypes.data) == 0 and lv[0] == L
    score_level = int(lv[1])
    # the client's keys on the longest chain: relinearisation, fold rotations, the scorer's rotations
    ps = synth.ParamSet("mem", logN, tuple(q), p, 45, R, B, -10)
    rots = sorted(set(m.score_rotations()) | set(m.fold_rotations()))
    km = synth.key_material(ps, 31, rots=rots)
    top_o = ev.o[L]
    rot_keys = {r: top_o.evk_gen(km.s, r, km.evk_a[i], km.evk_e[i]) for i, r in enumerate(rots)}
    ka = synth.uniform_residues(31, 50, list(q) + [p], ps.N, lead=(L,))
    ke = synth.rounded_gaussian(31, 51, (L, ps.N))
    rlk = top_o.rlk_gen(km.s, ka, ke)
    ev.set_keys(rlk, rot_keys)
    # contexts: one per level for the arithmetic (R = B = 1), one scorer
    arith = [b.Context(synth.ParamSet("a%d" % l, logN, tuple(q[:l]), p, 45, 1, 1, -10)) for l in range(1, L + 1)]
    for l in range(2, L + 1):
        arith[l - 1].load_keys(restrict_keys(rlk, L, l)[None], [0])
    fold = m.fold_rotations()
    arith[L - 2].load_keys(restrict_keys(np.stack([rot_keys[r] for r in fold]), L, L - 1), fold)
    scorer = b.Context(synth.ParamSet("s", logN, tuple(q[:score_level]), p, 45, R, B, -10))
    srots = m.score_rotations()
    scorer.load_keys(restrict_keys(np.stack([rot_keys[r] for r in srots]), L, score_level), srots)
    # inputs: a query near a planted row, candidates enrolled times kappa / lam
    rows = synth.toy_corpus(3, rows=n_rows, dim=R)
    rng = np.random.default_rng(2)
    qR = rows[11] + rng.standard_normal(R) / np.sqrt(R)   # noise of norm ~1 beside the unit row: cosine ~0.7 at every R
    qR = (0.7 * qR / np.linalg.norm(qR)).astype(np.float32)
    ct = top_o.encrypt(km.s, top_o.encode(m.query_slots(qR), 45), km.ct_a, km.ct_e)
    ct_dev = arith[L - 1].import_(b.KIND_CT, ct, 1)
    nb = scorer.n_blocks(n_rows)
    pt = scorer.encode_candidates(torch.from_numpy(m.scaled_rows(rows)).to(scorer.device), scorer.workspace(nb))
    (out, out_scale), (thr, thr_level, thr_scale) = b.membership_decide(
        arith, scorer, R, deg, iters, 45, tau, m.t_lo, m.t_hi, m.coef, ct_dev, pt, nb, want_threshold=True)
    arith[L - 1].sync()
    # the oracle, same circuit
    octx = mb.Ct(ct, 2.0 ** 45)
    thr_o = m.threshold(octx)
    assert thr_level == thr_o.level == L - m.depth_threshold and thr_scale == thr_o.scale
    got_thr = arith[thr_level - 1].export(b.KIND_CT, thr, 1)[0]
    assert np.array_equal(got_thr, thr_o.res)
    outs = arith[0].export(b.KIND_CT, out, nb)
    direct_all = rows.astype(np.float64) @ qR.astype(np.float64) - tau * np.linalg.norm(qR.astype(np.float64))
    for blk in range(nb):
        part = rows[blk * ps.n:(blk + 1) * ps.n]
        dec_o = m.decide(octx, part)
        assert dec_o.level == 1 and dec_o.scale == out_scale
        assert np.array_equal(outs[blk], dec_o.res), blk
        got = ev.decrypt(km.s, dec_o).real[: part.shape[0]]
        direct = direct_all[blk * ps.n: blk * ps.n + part.shape[0]]
        clear = np.abs(direct) > (4e-3 if deg >= 7 else 0.05) * tau
        assert np.array_equal(np.sign(got[clear]), np.sign(direct[clear]))
    # the library's own decryption of its decision agrees with the plain-number circuit
    mine = arith[0].decrypt_scores(km.s, outs, log_scale_out=45).reshape(-1)[:n_rows] * (2.0 ** 45 / out_scale)
    want = m.plain(rows, qR)["out"]
    assert np.abs(mine - want).max() < 1e-3
    assert mine[11] > 0


@pytest.mark.parametrize("logN,L,count", [(10, 4, 1), (11, 3, 11), (12, 6, 3)])
def test_multiply_bit_exact(logN, L, count):
    """hann_multiply: `count` ciphertext pairs, degree-2 product and relinearisation, against the oracle's product of each
    pair; then the rescale of all of them in one call."""
    import torch

    from oracle.oracle import Oracle, find_primes
    from paper_2608_21131_b200 import binding as b

    q, p = find_primes(45, logN + 1, L), find_primes(60, logN + 1, 1)[0]
    ps = synth.ParamSet("mul", logN, tuple(q), p, 45, 1, 1, -10)
    o = Oracle(logN, q, p, 45, 1, 1)
    km = synth.key_material(ps, 5, rots=[])
    rlk = o.rlk_gen(km.s, synth.uniform_residues(5, 50, list(q) + [p], ps.N, lead=(L,)), synth.rounded_gaussian(5, 51, (L, ps.N)))
    c = b.Context(ps)
    c.load_keys(rlk[None], [0])
    mods = np.array(q, dtype=np.uint64)[None, None, :, None]
    x = synth.uniform_residues(6, 1, list(q), ps.N, lead=(count, 2)) % mods
    y = synth.uniform_residues(6, 2, list(q), ps.N, lead=(count, 2)) % mods
    xd, yd = c.import_(b.KIND_CT, x, count), c.import_(b.KIND_CT, y, count)
    ws = c.workspace(3)
    prod = c.multiply(xd, yd, count, ws)
    got = c.export(b.KIND_CT, prod, count)
    want = np.stack([o.relin(o.mac_ct(x[i][None], y[i][None])[0], rlk) for i in range(count)])
    assert np.array_equal(got, want)
    low = b.Context(synth.ParamSet("mul1", logN, tuple(q[:-1]), p, 45, 1, 1, -10))
    res = c.rescale(prod, count, ws)
    c.sync()
    got_r = low.export(b.KIND_CT, res, count)
    assert np.array_equal(got_r, np.stack([o.compact(want[i], L - 1, rescale=True) for i in range(count)]))
    # error paths; an empty batch is not an error
    lib = b.load_library()
    assert lib.hann_multiply(c.h, None, None, 0, None, None, 0) == b.OK
    assert lib.hann_multiply(c.h, b._ptr(xd), b._ptr(yd), -1, b._ptr(prod), b._ptr(ws), ws.numel() * 8) == b.EINVAL
    assert lib.hann_multiply(c.h, b._ptr(xd), b._ptr(yd), count, b._ptr(prod), b._ptr(ws), 1024) == b.EWORKSPACE
    nokey = b.Context(ps)
    assert lib.hann_multiply(nokey.h, b._ptr(xd), b._ptr(yd), count, b._ptr(prod), b._ptr(ws), ws.numel() * 8) == b.ENOKEY
