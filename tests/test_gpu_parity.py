"""CUDA path vs CPU oracle, element by element, through the C ABI.  Ciphertext residues must be bit-identical in
the canonical layout at the five conformance points (encoded plaintexts, baby ciphertexts, partial sums, score
ciphertexts, key-switch outputs); decrypted scores must be within 2^-10 (toy scale 2^25) / 2^-18 (scale 2^40) of
the float64 dot products."""
import numpy as np
import pytest

from paper_2608_21131_b200 import synth
from tests.helpers import Pair, make_oracle

pytestmark = pytest.mark.gpu


def torch_rows(p, rows):
    import torch

    return torch.from_numpy(np.ascontiguousarray(rows)).to(p.g.device)


def run_level(p, rows, qv, check=True):
    """score one level on both sides; returns decrypted GPU scores [n_rows]"""
    ps, g, o, b = p.ps, p.g, p.o, p.b
    ct_o, ct_g = p.query(qv)
    assert np.array_equal(ct_o, ct_g)
    ct_dev = g.import_(b.KIND_CT, ct_g, 1)
    baby = g.query_prepare(ct_dev, p.ws)
    baby_o = o.baby_set(ct_o, p.evk_o)
    baby_g = g.export(b.KIND_CT, baby, ps.B)
    assert np.array_equal(baby_g, baby_o)                                       # C2
    n_rows = rows.shape[0]
    nb = g.n_blocks(n_rows)
    pt = g.encode_candidates(torch_rows(p, rows), p.ws)
    inner = g.score_level(baby, pt, nb, p.ws)
    score = g.rotate_sum(inner, nb, p.ws)
    g.sync()
    score_g = g.export(b.KIND_CT, score, nb)
    if check:
        pt_g = g.export(b.KIND_PT, pt, nb * ps.R).reshape(nb, ps.G, ps.B, ps.L, ps.N)
        inner_g = g.export(b.KIND_CT, inner, nb * ps.G).reshape(nb, ps.G, 2, ps.L, ps.N)
        Rr = np.zeros((n_rows, ps.R), dtype=np.float32)
        Rr[:, : rows.shape[1]] = rows
        for blk in range(nb):
            sc_o, pt_o, in_o = o.score_block(Rr[blk * ps.n:(blk + 1) * ps.n], baby_o, p.evk_o[ps.B - 1], True, True)
            assert np.array_equal(pt_g[blk], pt_o)                              # C1
            assert np.array_equal(inner_g[blk], in_o)                           # C3
            assert np.array_equal(score_g[blk], sc_o)                           # C4
    got = g.decrypt_scores(p.km.s, score_g).reshape(-1)[:n_rows]
    want = rows.astype(np.float64) @ qv.astype(np.float64)[: rows.shape[1]]
    assert np.abs(got - want).max() < 2.0 ** ps.tol_log2
    return got, score_g


@pytest.mark.parametrize("logN", [4, 5, 8, 9, 10, 12])
def test_import_export_roundtrip_and_transform(logN):
    from paper_2608_21131_b200 import binding as b

    ps = synth.small_params(logN, 4, 2, L=2)
    g = b.Context(ps)
    rng = np.random.default_rng(logN)
    polys = np.stack([np.stack([rng.integers(0, q, size=ps.N, dtype=np.uint64) for q in ps.q]) for _ in range(3)])
    dev = g.import_(b.KIND_POLY, polys, 3)
    back = g.export(b.KIND_POLY, dev, 3).reshape(3, ps.L, ps.N)
    assert np.array_equal(back, polys)
    # the private layout is the negacyclic transform in bit-reversed order: position k holds a(psi^(2 brev(k)+1)),
    # whatever psi the library picked; check the multiset-free consequence a(psi^...)=const for a constant poly
    const = np.zeros((1, ps.L, ps.N), dtype=np.uint64)
    const[0, :, 0] = 7
    dev = g.import_(b.KIND_POLY, const, 1)
    assert (dev.cpu().numpy().view(np.uint64)[: ps.L * ps.N] == 7).all()


@pytest.mark.parametrize("logN,R,B,L,big", [(4, 4, 2, 2, False), (8, 8, 4, 2, False), (9, 16, 4, 3, True), (11, 64, 8, 2, False)])
def test_client_half_matches_oracle(logN, R, B, L, big):
    ps = synth.small_params(logN, R, B, L=L, big=big)
    p = Pair(ps, key_seed=5)
    assert np.array_equal(p.evk_g, p.evk_o)                 # keygen from the same samples
    qv = synth.toy_query(2, dim=R)
    ct_o, ct_g = p.query(qv)
    assert np.array_equal(ct_o, ct_g)                       # canonical encode + symmetric encryption
    # decrypt of the fresh query gives the tiled query back
    z = p.g.decrypt_scores(p.km.s, ct_g, log_scale_out=ps.log_scale)[0]
    assert np.abs(z - np.tile(qv.astype(np.float64), ps.n // R)).max() < 1e-3
    zo = p.o.decrypt_slots(p.km.s, ct_o, ps.log_scale).real
    assert np.abs(z - zo).max() < 1e-9


@pytest.mark.parametrize("logN,L,big,rot", [(4, 2, False, 1), (8, 2, False, 3), (10, 2, False, 2), (10, 4, True, 4), (12, 2, False, 8)])
def test_keyswitch_matches_oracle(logN, L, big, rot):
    ps = synth.small_params(logN, 8, 8 if logN > 4 else 4, L=L, big=big)
    p = Pair(ps, key_seed=7)
    rng = np.random.default_rng(rot)
    d = np.stack([rng.integers(0, q, size=ps.N, dtype=np.uint64) for q in ps.q])
    ks0_o, ks1_o = p.o.keyswitch(d, p.evk_o[rot - 1])
    dev = p.g.import_(p.b.KIND_POLY, d[None], 1)
    ks0, ks1 = p.g.keyswitch(rot, dev, p.ws)
    assert np.array_equal(p.g.export(p.b.KIND_POLY, ks0, 1)[0, 0], ks0_o)     # C5
    assert np.array_equal(p.g.export(p.b.KIND_POLY, ks1, 1)[0, 0], ks1_o)


@pytest.mark.parametrize(
    "logN,R,B,L,big,n_rows,dim",
    [
        (4, 4, 2, 2, False, 8, 4),        # one full block, tiny ring
        (5, 4, 4, 2, False, 13, 3),       # G = 1 (no rotate-and-sum), ragged, dim < R
        (6, 8, 1, 2, False, 40, 8),       # B = 1 (no baby rotations), two blocks, ragged
        (8, 16, 4, 2, False, 300, 16),    # single-pass transform, three blocks
        (9, 32, 8, 3, True, 256, 24),     # two-pass transform, 50-bit primes, zero-padded dimension
        (10, 64, 8, 2, False, 1500, 64),  # three blocks, last ragged
    ],
)
def test_level_bit_exact_small(logN, R, B, L, big, n_rows, dim):
    ps = synth.small_params(logN, R, B, L=L, big=big)
    if big:
        ps = ps.with_(log_scale=40)
    p = Pair(ps, key_seed=logN)
    rows = synth.toy_corpus(logN, rows=n_rows, dim=dim)
    qv = np.zeros(R, dtype=np.float32)
    qv[:dim] = synth.toy_query(logN + 1, dim=dim)
    run_level(p, rows, qv)


@pytest.mark.parametrize(
    "logN,R,B,L,big,n_rows",
    [
        (5, 8, 2, 2, False, 40),        # tiny ring (generic kernels), three blocks, G = 4
        (8, 16, 4, 2, False, 300),      # single-pass transform, three blocks
        (10, 64, 8, 3, True, 1300),     # 50-bit primes, G = 8, three blocks (fused lift path)
        (12, 64, 8, 2, False, 4096),    # the toy configuration's ring, G = 8
        (13, 128, 32, 4, True, 9000),   # production primes and B, G = 4, three blocks
        (9, 32, 32, 2, False, 300),     # G = 1: nothing to rotate
    ],
)
def test_lazy_giant_steps_bit_exact(logN, R, B, L, big, n_rows):
    """hann_rotate_sum_lazy (distinct giant-step keys, key products summed, one ModDown per block) against the oracle's
    evaluation in the same order, bit for bit; its decrypted scores within the tolerance, and within the key-switch noise
    of the Horner evaluation of the same partial sums."""
    import torch

    from paper_2608_21131_b200 import binding as b

    ps = synth.small_params(logN, R, B, L=L, big=big)
    if big:
        ps = ps.with_(log_scale=40)
    G = ps.G
    rots = sorted(set(range(1, B + 1)) | {g * B for g in range(1, G)})
    g_, o = b.Context(ps), make_oracle(ps)
    km = synth.key_material(ps, logN, rots=rots)
    evk_o = dict(zip(rots, (o.evk_gen(km.s, r, km.evk_a[i], km.evk_e[i]) for i, r in enumerate(rots))))
    evk_g = g_.keygen_from_samples(km.s, km.rots, km.evk_a, km.evk_e)
    g_.load_keys(evk_g, km.rots)
    rows = synth.toy_corpus(logN, rows=n_rows, dim=R)
    qv = synth.toy_query(logN + 1, dim=R)
    ct = g_.encrypt_query(km.s, qv, km.ct_a, km.ct_e)
    nb = g_.n_blocks(n_rows)
    ws = g_.workspace(nb)
    baby = g_.query_prepare(g_.import_(b.KIND_CT, ct, 1), ws)
    inner = g_.score_level(baby, g_.encode_candidates(torch.from_numpy(rows).to(g_.device), ws), nb, ws)
    score = g_.rotate_sum_lazy(inner, nb, ws)
    horner = g_.rotate_sum(inner, nb, ws)
    g_.sync()
    score_h, inner_h = g_.export(b.KIND_CT, score, nb), g_.export(b.KIND_CT, inner, nb * G).reshape(nb, G, 2, L, ps.N)
    giant = (np.stack([evk_o[g * B] for g in range(1, G)]) if G > 1
             else np.zeros((0, L, 2, L + 1, ps.N), dtype=np.uint64))
    for blk in range(nb):
        assert np.array_equal(score_h[blk], o.rotate_sum_lazy(inner_h[blk], giant)), blk
    got = g_.decrypt_scores(km.s, score_h).reshape(-1)[:n_rows]
    want = rows.astype(np.float64) @ qv.astype(np.float64)
    assert np.abs(got - want).max() < 2.0 ** ps.tol_log2
    got_h = g_.decrypt_scores(km.s, g_.export(b.KIND_CT, horner, nb)).reshape(-1)[:n_rows]
    assert np.abs(got - got_h).max() < 2.0 ** ps.tol_log2
    # a tight workspace (one block per round) gives the same bits
    if nb > 1:
        tight = g_.alloc(g_.workspace_bytes(1))
        again = g_.rotate_sum_lazy(inner, nb, tight)
        g_.sync()
        assert torch.equal(again, score)
    # a missing giant-step key is reported, not guessed
    if G > 2:
        h = b.Context(ps)
        h.load_keys(evk_g[: B], km.rots[: B])
        with pytest.raises(b.HannError) as ei:
            h.rotate_sum_lazy(inner, nb, ws)
        assert ei.value.code == b.ENOKEY


def test_toy_configuration_full():
    """Toy configuration: 4,096 unit-norm rows of dimension 64, N = 2^12, scale 2^25 -> two blocks; every conformance
    point bit-exact, every score within 2^-10; repeated with three seed triples."""
    ps = synth.TOY
    for cs, qs, ks in ((1, 2, 3), (11, 12, 13), (21, 22, 23)):
        p = Pair(ps, key_seed=ks)
        got, _ = run_level(p, synth.toy_corpus(cs), synth.toy_query(qs), check=(cs == 1))
        assert got.shape == (4096,)


def test_toy_other_baby_step_counts():
    for B in (4, 32):
        ps = synth.TOY.with_(B=B)
        p = Pair(ps, key_seed=3)
        run_level(p, synth.toy_corpus(1, rows=2048 + 77), synth.toy_query(2))


@pytest.mark.parametrize("n_rows", [1500, 3000, 7000, 15000])   # 1, 2, 4 and 8 blocks
def test_host_buffer_level_matches_device_path(n_rows):
    ps = synth.TOY
    p = Pair(ps, key_seed=3)
    rows = synth.toy_corpus(1, rows=n_rows)
    qv = synth.toy_query(2)
    _, score_dev = run_level(p, rows, qv, check=False)
    ct_o, ct_g = p.query(qv)
    ws = p.g.alloc(p.g.level_host_bytes(rows.shape[0]))
    out = p.g.score_level_host(ct_g, rows, ws)
    assert np.array_equal(out, score_dev)
    # downloading only the first limb (the toy set has two): the same first limbs, in the layout of the exact compaction
    p.g.set_tuning(p.b.TUNE_HOST_LIMBS, 1)
    nb = out.shape[0]
    small = np.empty((nb, 2, 1, ps.N), dtype=np.uint64)
    p.g.score_level_host(ct_g, rows, ws, small)
    p.g.set_tuning(p.b.TUNE_HOST_LIMBS, ps.L)
    assert np.array_equal(small, out[:, :, :1])
    # any cut of the level into block groups (scored while later groups are still uploaded and encoded): same bits
    for groups in (1, 2, 3, 4):
        p.g.set_tuning(p.b.TUNE_HOST_GROUPS, groups)
        ws_g = p.g.alloc(p.g.level_host_bytes(rows.shape[0]))
        assert np.array_equal(p.g.score_level_host(ct_g, rows, ws_g), score_dev)
    p.g.set_tuning(p.b.TUNE_HOST_GROUPS, 0)
    # the device-resident level call cuts the level the same way (a group scored beside the encoding of the next): same bits,
    # also with both orders of the giant steps and with a workspace too small for the groups (plain order)
    g, b = p.g, p.b
    ct_dev = g.import_(b.KIND_CT, ct_g, 1)
    for groups in (0, 1, 2, 3, 4):
        g.set_tuning(b.TUNE_HOST_GROUPS, groups)
        for ws in (g.workspace(nb), g.workspace(1)):
            baby, pt, inner, score = (g.alloc(g.sizeof(b.SIZE_BABY)), g.alloc(nb * g.sizeof(b.SIZE_PT_BLOCK)),
                                      g.alloc(nb * g.sizeof(b.SIZE_INNER)), g.alloc(nb * g.sizeof(b.SIZE_CT)))
            g.query_level(ct_dev, torch_rows(p, rows), ws, baby, pt, inner, score)
            g.sync()
            assert np.array_equal(g.export(b.KIND_CT, score, nb), score_dev), groups
    g.set_tuning(b.TUNE_HOST_GROUPS, 0)


def test_full_ring_one_block():
    """N = 2^16, 4 x ~50-bit primes + ~60-bit special prime, scale 2^40, R = 128, B = 32: one ragged block checked at
    every conformance point, scores within 2^-18."""
    ps = synth.FULL16
    p = Pair(ps, key_seed=1)
    rows = synth.project_rows(synth.toy_corpus(5, rows=ps.n - 1234, dim=96).astype(np.float64), None, 128)
    qv = np.zeros(128, dtype=np.float32)
    qv[:96] = synth.toy_query(6, dim=96)
    got, _ = run_level(p, rows, qv)
    want = rows.astype(np.float64) @ qv.astype(np.float64)
    assert np.abs(got - want).max() < 2.0 ** -22  # observed error level, regression alarm


def test_error_codes():
    from paper_2608_21131_b200 import binding as b
    import torch

    ps = synth.small_params(8, 8, 4, L=2)
    with pytest.raises(b.HannError):
        b.Context(ps.with_(q=(ps.q[0], ps.q[0] + 2)))  # not prime
    with pytest.raises(b.HannError):
        b.Context(ps.with_(B=3))
    g = b.Context(ps)
    ws = g.workspace(1)
    ct = g.alloc(g.sizeof(b.SIZE_CT))
    with pytest.raises(b.HannError) as ei:
        g.query_prepare(ct, ws)
    assert ei.value.code == b.ENOKEY
    km = synth.key_material(ps, 1)
    g.load_keys(g.keygen_from_samples(km.s, km.rots, km.evk_a, km.evk_e), km.rots)
    with pytest.raises(b.HannError) as ei:
        g.query_prepare(ct, ws[:16])
    assert ei.value.code == b.EWORKSPACE
    rows = torch.zeros((4, 9), dtype=torch.float32, device=g.device)
    with pytest.raises(b.HannError) as ei:
        g.encode_candidates(rows, ws)
    assert ei.value.code == b.ESHAPE
    # the context stays usable after errors
    g.query_prepare(ct, ws)
    g.sync()


def test_error_codes_of_the_newer_calls():
    """refusals of the lazy giant steps, the hoisted rotation, the fold, the rescale, the projection and the membership
    circuit: each names its reason, nothing is computed, and the contexts stay usable"""
    from paper_2608_21131_b200 import binding as b
    import torch

    ps = synth.small_params(9, 16, 4, L=3, big=True)
    g = b.Context(ps)
    km = synth.key_material(ps, 1)                       # rotations 1..4: no key of rotation 8 or 12
    g.load_keys(g.keygen_from_samples(km.s, km.rots, km.evk_a, km.evk_e), km.rots)
    ws = g.workspace(1)
    ct = g.alloc(g.sizeof(b.SIZE_CT))
    ct.zero_()
    inner = g.alloc(g.sizeof(b.SIZE_INNER))
    inner.zero_()

    def code(fn):
        with pytest.raises(b.HannError) as ei:
            fn()
        return ei.value.code

    assert code(lambda: g.rotate_sum_lazy(inner, 1, ws)) == b.ENOKEY                    # needs rotations 8 and 12
    assert code(lambda: g.rotate_hoisted(ct, 3, 4, ws)) == b.ENOKEY                     # rotations 3..6
    assert code(lambda: g.rotate_hoisted(ct, 0, 1, ws)) == b.ESHAPE
    assert code(lambda: g.rotate_hoisted(ct, 1, 2, ws[:64])) == b.EWORKSPACE
    assert code(lambda: g.fold(ct, 8, 1, ws)) == b.ENOKEY
    assert code(lambda: g.fold(ct, 128, 2, ws)) == b.ESHAPE                             # rotation 256 = n
    g.fold(ct, 2, 0, ws)                                                                # no steps: nothing to do
    one = b.Context(ps.with_(q=ps.q[:1]))
    assert code(lambda: one.rescale(one.alloc(one.sizeof(b.SIZE_CT)), 1, ws)) == b.ESHAPE   # a single prime left
    assert g.rotate_sum_lazy(inner, 0, ws) is not None                                  # no blocks: a no-op
    # projection: the second context must be the same ring with one prime less
    other = b.Context(ps.with_(q=ps.q[:2], R=8, B=4))
    lo = g.alloc(g.B * g.sizeof(b.SIZE_POLY) // 2)
    wpt = other.alloc(other.sizeof(b.SIZE_PT_BLOCK))
    assert code(lambda: g.project_query(other, ct, lo, lo, wpt, 64)) == b.ESHAPE
    mid = b.Context(ps.with_(q=ps.q[:2]))
    assert code(lambda: g.project_query(mid, ct, lo, lo, wpt, 48)) == b.ESHAPE          # D / R not a power of two
    assert code(lambda: g.project_query(mid, ct, lo, lo, wpt, 64)) == b.ENOKEY          # rotation n - R + 1 is not loaded
    W = torch.zeros((40, 16), dtype=torch.float32, device=g.device)
    assert code(lambda: g.project_enrol(W, 50, ws)) == b.ESHAPE                         # D must be a multiple of R dividing n
    # membership: a chain that does not fit the circuit's depth
    arith = [b.Context(ps.with_(q=ps.q[:l], R=1, B=1)) for l in (1, 2, 3)]
    coef = np.ones(8)
    assert code(lambda: b.membership_decide(arith, g, 16, 7, 3, 40, 0.4, 0.05, 1.0, coef, ct, None, 0)) == b.ESHAPE
    # and the context still computes
    g.rotate_hoisted(ct, 1, 3, ws)
    g.sync()


# primes of the other arithmetic classes: [2^50, 2^57) runs the lazy integer transforms and the generic element-wise
# kernels, >= 2^57 Harvey's butterflies; the special prime just below 2^62 is the largest the library accepts
Q54 = (18014398506729473, 18014398505943041, 18014398496243713)
Q58 = (288230376147386369,)
P62 = 4611686018425815041


@pytest.mark.parametrize(
    "logN,q,p,R,B,n_rows",
    [
        (9, Q54[:2], synth.P60, 16, 4, 300),         # lazy-integer limbs + 60-bit special prime
        (10, Q54, P62, 32, 8, 700),                   # three 54-bit limbs, 62-bit special prime (128-bit inner product)
        (10, (synth.Q50[0], Q54[0]), P62, 16, 4, 512),  # binary64 and integer limbs side by side
        (11, Q58 + Q54[:1], synth.P60, 64, 8, 1100),  # a 58-bit ciphertext prime (Harvey class)
        (8, Q54[:2], P62, 8, 2, 200),                 # single-pass transforms with integer limbs
    ],
)
def test_level_bit_exact_other_prime_classes(logN, q, p, R, B, n_rows):
    ps = synth.ParamSet("classes", logN, tuple(q), p, 40, R, B, -18)
    pr = Pair(ps, key_seed=logN)
    rows = synth.toy_corpus(logN, rows=n_rows, dim=R)
    qv = synth.toy_query(logN + 1, dim=R)
    run_level(pr, rows, qv)
    # and one key switch of an arbitrary polynomial under these moduli
    rng = np.random.default_rng(1)
    d = np.stack([rng.integers(0, m, size=ps.N, dtype=np.uint64) for m in ps.q])
    ks0_o, ks1_o = pr.o.keyswitch(d, pr.evk_o[0])
    ks0, ks1 = pr.g.keyswitch(1, pr.g.import_(pr.b.KIND_POLY, d[None], 1), pr.ws)
    assert np.array_equal(pr.g.export(pr.b.KIND_POLY, ks0, 1)[0, 0], ks0_o)
    assert np.array_equal(pr.g.export(pr.b.KIND_POLY, ks1, 1)[0, 0], ks1_o)


def test_empty_and_single_row_levels():
    import torch

    ps = synth.small_params(10, 16, 4, L=2)
    p = Pair(ps, key_seed=2)
    g, b = p.g, p.b
    # no rows: nothing to do, no error
    empty = torch.zeros((0, 16), dtype=torch.float32, device=g.device)
    pt = g.alloc(8)
    g.encode_candidates(empty, p.ws, pt)
    g.score_level(g.alloc(g.sizeof(b.SIZE_BABY)), pt, 0, p.ws, g.alloc(8))
    g.rotate_sum(g.alloc(8), 0, p.ws, g.alloc(8))
    g.sync()
    # one row: a whole block is computed, slot 0 holds its score, every other slot is noise around zero
    rows = synth.toy_corpus(5, rows=1, dim=16)
    qv = synth.toy_query(6, dim=16)
    got, score_g = run_level(p, rows, qv)
    allslots = g.decrypt_scores(p.km.s, score_g)[0]
    assert np.abs(allslots[1:]).max() < 2.0 ** ps.tol_log2


def test_encode_into_buffer_that_is_only_word_aligned():
    """Polynomial buffers need no more than 8-byte alignment: the transform falls back from its bulk-copy kernel to
    the plain-load kernel and produces the same words."""
    import torch

    ps = synth.small_params(12, 32, 8, L=2)
    p = Pair(ps, key_seed=4)
    g, b = p.g, p.b
    rows = torch.from_numpy(synth.toy_corpus(7, rows=ps.n + 5, dim=32)).to(g.device)
    nbytes = g.n_blocks(rows.shape[0]) * g.sizeof(b.SIZE_PT_BLOCK)
    aligned = g.encode_candidates(rows, p.ws, g.alloc(nbytes))
    shifted = g.alloc(nbytes + 8)[1:]
    assert shifted.data_ptr() % 16 == 8
    g.encode_candidates(rows, p.ws, shifted)
    g.sync()
    assert torch.equal(aligned, shifted)


@pytest.mark.parametrize("logN,R,B,L,big", [(10, 16, 4, 2, False), (12, 32, 8, 2, False), (13, 64, 8, 4, True), (16, 128, 32, 4, True)])
def test_encode_symmetry_shortcut_gives_the_same_words(logN, R, B, L, big):
    """The encoder computes only the stored half of every transformed plaintext (an encoding of real slots is fixed by
    X -> 1/X, so the other half is its mirror image); with the shortcut switched off it computes every transform in
    full and keeps the first half.  Same words, and the canonical form is the oracle's encoding."""
    import torch

    ps = synth.small_params(logN, R, B, L=L, big=big)
    p = Pair(ps, key_seed=6)
    g, b = p.g, p.b
    rows = torch.from_numpy(synth.toy_corpus(11, rows=ps.n + 3 if logN < 16 else 1000, dim=R - 1)).to(g.device)
    nbytes = g.n_blocks(rows.shape[0]) * g.sizeof(b.SIZE_PT_BLOCK)
    short = g.encode_candidates(rows, p.ws, g.alloc(nbytes))
    g.set_tuning(b.TUNE_ENCODE_SYMMETRY, 0)
    full = g.encode_candidates(rows, p.ws, g.alloc(nbytes))
    g.set_tuning(b.TUNE_ENCODE_SYMMETRY, 1)
    g.sync()
    assert torch.equal(short, full)
    pt_g = g.export(b.KIND_PT, short, 2)                      # plaintexts (g, b) = (0, 0) and (0, 1) of block 0
    Rr = np.zeros((ps.n, R), dtype=np.float32)
    nr = min(ps.n, rows.shape[0])
    Rr[:nr, : R - 1] = rows[:nr].cpu().numpy()
    for bb in range(2):
        z = np.array([Rr[i, (i + bb) % R] for i in range(ps.n)], dtype=np.float64)
        m = p.o.encode(z)
        want = np.stack([np.array([int(v) % q for v in m], dtype=np.uint64) for q in ps.q])
        assert np.array_equal(pt_g.reshape(2, ps.L, ps.N)[bb], want)
    # import of the canonical form gives the stored words back
    back = g.import_(b.KIND_PT, pt_g, 2)
    assert torch.equal(back.reshape(-1)[: 2 * ps.L * ps.n], short.reshape(-1)[: 2 * ps.L * ps.n])


@pytest.mark.parametrize(
    "logN,L,big,n_rows",
    [
        (6, 3, False, 40),     # tiny ring, generic kernels, two blocks
        (10, 2, False, 700),   # two ~30-bit primes: one limb left after the rescale
        (11, 4, True, 1500),   # production primes (4 x ~50 bit), two blocks
    ],
)
def test_compacted_scores_bit_exact_and_decrypt(logN, L, big, n_rows):
    """Output compaction: the first limbs as they are (exact) and the rescale by the last prime, each bit-identical to the
    oracle's on the same score ciphertexts, and decrypting to the same scores (to the rounding error of the division)."""
    if big:
        ps = synth.ParamSet("n%d" % logN, logN, synth.Q50, synth.P60, 40, 32, 8, -18)
    else:
        ps = synth.small_params(logN, 16, 4, L=L)
    p = Pair(ps, key_seed=logN)
    g, o, b = p.g, p.o, p.b
    rows = synth.toy_corpus(logN, rows=n_rows, dim=ps.R)
    qv = synth.toy_query(logN + 1, dim=ps.R)
    ct_o, ct_g = p.query(qv)
    ct_dev = g.import_(b.KIND_CT, ct_g, 1)
    nb = g.n_blocks(n_rows)
    baby, pt, inner, score = (g.alloc(g.sizeof(b.SIZE_BABY)), g.alloc(nb * g.sizeof(b.SIZE_PT_BLOCK)),
                              g.alloc(nb * g.sizeof(b.SIZE_INNER)), g.alloc(nb * g.sizeof(b.SIZE_CT)))
    g.query_level(ct_dev, torch_rows(p, rows), p.ws, baby, pt, inner, score)
    score_g = g.export(b.KIND_CT, score, nb)
    full = g.decrypt_scores(p.km.s, score_g)
    for keep, rescale in ((ps.L - 1, False), (1, True), (ps.L - 1, True)):
        small = g.compact_scores(score, nb, keep, rescale, p.ws)
        small_g = g.export_limbs(small, nb * 2, keep).reshape(nb, 2, keep, ps.N)
        for blk in range(nb):
            assert np.array_equal(small_g[blk], o.compact(score_g[blk], keep, rescale))
        got = g.decrypt_compact(p.km.s, small_g, rescale)
        if not rescale:
            if keep * 30 > 2 * ps.log_scale + 12 or big:       # enough modulus left for the unscaled message
                assert np.array_equal(got, full)
        else:
            sigma = np.sqrt(ps.N * (ps.N / 18.0 + 1.0 / 12.0) / 2.0) / (2.0 ** (2 * ps.log_scale) / ps.q[-1])
            assert np.abs(got - full).max() < 12 * sigma   # product-of-Gaussians tails, see the oracle's pin
            got_o = np.stack([o.decrypt_compact_slots(p.km.s, small_g[blk], 2 * ps.log_scale).real for blk in range(nb)])
            assert np.abs(got - got_o).max() < 1e-9 * max(1.0, np.abs(got_o).max()) + 2 * sigma * 1e-6


@pytest.mark.parametrize("logN,R,B,L,big,n_rows,nq", [(6, 8, 2, 2, False, 70, 3), (10, 64, 8, 2, False, 1200, 5), (11, 32, 32, 4, True, 1100, 2),
                                                      (11, 32, -32, 4, True, 2100, 3)])
def test_cross_query_batch_matches_single_queries(logN, R, B, L, big, n_rows, nq):
    """Several queries against the same encoded blocks in one call: every query's partial sums are bit-identical to the
    oracle's multiply-accumulate with that query's baby set (and hence to the single-query call), and the scores
    decrypt within tolerance."""
    import torch

    pair_b32 = B < 0   # two queries per pass at B = 32 as well (off by default: it does not pay there)
    B = abs(B)
    ps = synth.ParamSet("b%d" % logN, logN, synth.Q50, synth.P60, 40, R, B, -18) if big else synth.small_params(logN, R, B, L=L)
    p = Pair(ps, key_seed=logN + 7)
    g, o, b = p.g, p.o, p.b
    if pair_b32:
        g.set_tuning(b.TUNE_PAIR_B32, 1)
    rows = synth.toy_corpus(logN, rows=n_rows, dim=R)
    nb = g.n_blocks(n_rows)
    pt = g.encode_candidates(torch_rows(p, rows), p.ws)
    pt_o = [o.encode_block(rows[blk * ps.n:(blk + 1) * ps.n]) for blk in range(nb)]
    babies = g.alloc(nq * g.sizeof(b.SIZE_BABY))
    words = g.sizeof(b.SIZE_BABY) // 8
    qvs, baby_os = [], []
    for q in range(nq):
        qv = synth.toy_query(100 + q, dim=R)
        ct_o, ct_g = p.query(qv)
        g.query_prepare(g.import_(b.KIND_CT, ct_g, 1), p.ws, babies[q * words:(q + 1) * words])
        qvs.append(qv)
        baby_os.append(o.baby_set(ct_o, p.evk_o))
    inner = g.score_level_batch(babies, nq, pt, nb, p.ws)
    single = g.score_level(babies[words:2 * words], pt, nb, p.ws)
    g.sync()
    iw = nb * g.sizeof(b.SIZE_INNER) // 8
    assert torch.equal(inner[iw:2 * iw], single[:iw])
    inner_g = g.export(b.KIND_CT, inner, nq * nb * ps.G).reshape(nq, nb, ps.G, 2, ps.L, ps.N)
    for q in range(nq):
        for blk in range(nb):
            assert np.array_equal(inner_g[q, blk], o.mac(pt_o[blk], baby_os[q]))
    score = g.rotate_sum(inner, nq * nb, p.ws)
    got = g.decrypt_scores(p.km.s, g.export(b.KIND_CT, score, nq * nb)).reshape(nq, nb * ps.n)[:, :n_rows]
    for q in range(nq):
        assert np.abs(got[q] - rows.astype(np.float64) @ qvs[q].astype(np.float64)).max() < 2.0 ** ps.tol_log2


@pytest.mark.parametrize(
    "logN,R,B,L,bits,log_scale,tol,n_rows",
    [
        (10, 128, 64, 2, 30, 25, -10, 600),    # 64 baby steps, two giant steps: eight-warp multiply-accumulate
        (10, 128, 128, 2, 30, 25, -10, 300),   # every step a baby step (G = 1): 127 rotation keys, no rotate-and-sum
        (9, 16, 4, 1, 50, 20, -8, 300),        # a single ~50-bit ciphertext prime (one digit); scale^2 must stay below it
        (9, 16, 4, 6, 40, 25, -10, 300),       # six ciphertext primes: the generic key-switch kernels
        (11, 16, 4, 8, 36, 25, -10, 1100),     # the maximum of eight ciphertext primes, two blocks
    ],
)
def test_level_bit_exact_other_shapes(logN, R, B, L, bits, log_scale, tol, n_rows):
    """parameter shapes outside the benchmark configurations: wide baby sets, one and many ciphertext primes"""
    from oracle.oracle import find_primes

    if bits == 30:
        ps = synth.small_params(logN, R, B, L=L).with_(log_scale=log_scale, tol_log2=tol)
    elif bits == 50:
        ps = synth.ParamSet("shape", logN, synth.Q50[:L], synth.P60, log_scale, R, B, tol)
    else:
        q = find_primes(bits, 13, L)
        ps = synth.ParamSet("shape", logN, q, find_primes(bits + 6, 13, 1)[0], log_scale, R, B, tol)
    p = Pair(ps, key_seed=logN + L)
    rows = synth.toy_corpus(logN + L, rows=n_rows, dim=R)
    run_level(p, rows, synth.toy_query(logN + L + 1, dim=R))


@pytest.mark.parametrize("logN,R,B,L,big,n_rows", [(6, 8, 2, 2, False, 50), (10, 16, 4, 2, False, 900), (11, 32, 8, 4, True, 1500)])
def test_encrypted_database_level_bit_exact(logN, R, B, L, big, n_rows):
    """Encrypted candidates (ct x ct): relinearisation key, block encryption, degree-2 multiply-accumulate +
    relinearisation and the unchanged rotate-and-sum, each bit-identical to the oracle; scores within tolerance."""
    ps = synth.ParamSet("db%d" % logN, logN, synth.Q50, synth.P60, 40, R, B, -18) if big else synth.small_params(logN, R, B, L=L)
    p = Pair(ps, key_seed=logN + 11)
    g, o, b = p.g, p.o, p.b
    ka = synth.uniform_residues(78, 50, list(ps.q) + [ps.p], ps.N, lead=(ps.L,))
    ke = synth.rounded_gaussian(78, 51, (ps.L, ps.N))
    rlk_o = o.rlk_gen(p.km.s, ka, ke)
    rlk_g = g.keygen_relin_from_samples(p.km.s, ka, ke)
    assert np.array_equal(rlk_g, rlk_o)
    g.load_keys(rlk_g[None], [0])
    rows = synth.toy_corpus(logN + 3, rows=n_rows, dim=R)
    qv = synth.toy_query(logN + 4, dim=R)
    ct_o, ct_g = p.query(qv)
    baby = g.query_prepare(g.import_(b.KIND_CT, ct_g, 1), p.ws)
    baby_o = o.baby_set(ct_o, p.evk_o)
    nb = g.n_blocks(n_rows)
    pt = g.encode_candidates(torch_rows(p, rows), p.ws)
    ptw, dbw = g.sizeof(b.SIZE_PT_BLOCK) // 8, g.sizeof(b.SIZE_CTDB_BLOCK) // 8
    ctdb = g.alloc(nb * dbw * 8)
    inner_o = []
    for blk in range(nb):
        a = synth.uniform_residues(200 + blk, 40, list(ps.q), ps.N, lead=(ps.R,))
        e = synth.rounded_gaussian(200 + blk, 41, (ps.R, ps.N))
        g.encrypt_block(p.km.s, pt[blk * ptw:(blk + 1) * ptw], a, e, ctdb[blk * dbw:(blk + 1) * dbw])
        pt_o = o.encode_block(rows[blk * ps.n:(blk + 1) * ps.n])
        db_o = o.encrypt_block(p.km.s, pt_o, a, e)
        db_g = g.export(b.KIND_CT, ctdb[blk * dbw:(blk + 1) * dbw], ps.R)
        assert np.array_equal(db_g, db_o)
        d = o.mac_ct(db_o, baby_o)
        inner_o.append(np.stack([o.relin(d[gi], rlk_o) for gi in range(ps.G)]))
    inner = g.score_level_ctdb(baby, ctdb, nb, p.ws)
    inner_g = g.export(b.KIND_CT, inner, nb * ps.G).reshape(nb, ps.G, 2, ps.L, ps.N)
    for blk in range(nb):
        assert np.array_equal(inner_g[blk], inner_o[blk])
    score = g.rotate_sum(inner, nb, p.ws)
    score_g = g.export(b.KIND_CT, score, nb)
    for blk in range(nb):
        assert np.array_equal(score_g[blk], o.rotate_sum(inner_o[blk], p.evk_o[ps.B - 1]))
    got = g.decrypt_scores(p.km.s, score_g).reshape(-1)[:n_rows]
    assert np.abs(got - rows.astype(np.float64) @ qv.astype(np.float64)).max() < 2.0 ** ps.tol_log2


def test_bounded_wait_runs_out_and_is_reported():
    """Failure path of the bulk-copy kernels without a fault: a wait that nothing completes gives up after its limit, the
    next sync reports it, and the context keeps working."""
    from paper_2608_21131_b200 import binding as b

    ps = synth.small_params(10, 16, 4, L=2)
    p = Pair(ps, key_seed=2)
    g = p.g
    g.sync()
    waited = g.selftest_bounded_wait(20)
    assert 20.0 <= waited < 200.0
    with pytest.raises(b.HannError) as ei:
        g.sync()
    assert ei.value.code == b.ECUDA and "bounded wait" in str(ei.value)
    g.sync()                                    # the flag is cleared
    run_level(p, synth.toy_corpus(5, rows=900, dim=16), synth.toy_query(6, dim=16))   # and the context still computes


def test_abandoned_kernel_is_reported_by_every_synchronising_call():
    """A kernel that gave up a bounded wait must not go unnoticed by a caller that never calls hann_sync: the next call that
    synchronises (an export, the host-buffer level) returns HANN_ECUDA once, and the same call then succeeds."""
    from paper_2608_21131_b200 import binding as b

    ps = synth.small_params(10, 16, 4, L=2)
    p = Pair(ps, key_seed=2)
    g = p.g
    poly = g.alloc(g.sizeof(b.SIZE_POLY))
    poly.zero_()
    g.selftest_bounded_wait(1)
    with pytest.raises(b.HannError) as ei:
        g.export(b.KIND_POLY, poly, 1)
    assert ei.value.code == b.ECUDA and "bounded wait" in str(ei.value)
    assert not g.export(b.KIND_POLY, poly, 1).any()
    rows, qv = synth.toy_corpus(5, rows=700, dim=16), synth.toy_query(6, dim=16)
    ct = g.encrypt_query(p.km.s, qv, p.km.ct_a, p.km.ct_e)
    ws = g.alloc(g.level_host_bytes(rows.shape[0]))
    want = g.score_level_host(ct, rows, ws)
    g.selftest_bounded_wait(1)
    with pytest.raises(b.HannError) as ei:
        g.score_level_host(ct, rows, ws)
    assert ei.value.code == b.ECUDA
    assert np.array_equal(g.score_level_host(ct, rows, ws), want)
    g.selftest_bounded_wait(1)
    with pytest.raises(b.HannError):
        g.expand_uniform(1, 2)
    g.sync()


def test_seeded_key_generation_round_trip_and_statistics():
    """hann_keygen_seeded: the keys rotate a ciphertext correctly (decrypts to the rolled slots), depend on (seed, rotation)
    only, and the drawn secret / errors / uniform halves have the statistics of their distributions.  The evaluation keys
    equal what hann_keygen_from_samples gives for the same samples, recovered from the key itself: a_j is stored in the
    key, and e_j = b_j + a_j s - F_j s' is small."""
    from paper_2608_21131_b200 import binding as b

    ps = synth.small_params(12, 16, 4, L=2)
    g = b.Context(ps)
    o = make_oracle(ps)
    s, evk = g.keygen_seeded(77, [1, 2, 3, 4])
    s2, evk2 = g.keygen_seeded(77, [3])
    assert np.array_equal(s, s2) and np.array_equal(evk[2], evk2[0])       # a key depends on (seed, rotation) only
    s3, evk3 = g.keygen_seeded(78, [3])
    assert not np.array_equal(s, s3) and not np.array_equal(evk3[0], evk2[0])
    # statistics: ternary secret close to uniform on {-1, 0, 1}; uniform halves spread over [0, q)
    assert set(np.unique(s).tolist()) == {-1, 0, 1}
    for v in (-1, 0, 1):
        assert abs(float(np.mean(s == v)) - 1 / 3) < 0.03
    a = evk[:, :, 1]                                                          # [rot][j][L+1][N]
    mods = np.array(list(ps.q) + [ps.p], dtype=np.float64)
    u = a.astype(np.float64) / mods[None, None, :, None]
    assert abs(u.mean() - 0.5) < 0.005 and abs(u.std() - 12 ** -0.5) < 0.005
    # errors: e_j = b_j + a_j s - F_j s' over limb 0, recovered with the oracle's exact products
    k = o.galois(1)
    sq = np.array([(int(x) % ps.q[0]) for x in s], dtype=np.uint64)
    sp = o.automorphism(0, k, sq)
    errs = []
    for j in range(ps.L):
        as_ = o.negacyclic_mul(0, evk[0, j, 1, 0], sq)
        e = (evk[0, j, 0, 0].astype(object) + as_.astype(object) - (ps.p % ps.q[0] if j == 0 else 0) * sp.astype(object)) % ps.q[0]
        e = np.array([int(v) - ps.q[0] if int(v) > ps.q[0] // 2 else int(v) for v in e], dtype=np.float64)
        errs.append(e)
    errs = np.concatenate(errs)
    assert np.abs(errs).max() <= 6 * 3.2 and abs(errs.std() - 3.2) < 0.15 and abs(errs.mean()) < 0.2
    # round trip: the seeded keys serve the ordinary path (oracle rotation with the same key, then decrypt)
    g.load_keys(evk, [1, 2, 3, 4])
    qv = synth.toy_query(5, dim=16)
    km = synth.key_material(ps, 3)
    ct = g.encrypt_query(s, qv, km.ct_a, km.ct_e)
    baby = g.export(b.KIND_CT, g.query_prepare(g.import_(b.KIND_CT, ct, 1), g.workspace(1)), ps.B)
    g.sync()
    for r in range(1, ps.B):
        assert np.array_equal(baby[r], o.rotate(ct, r, evk[r - 1]))
        z = o.decrypt_slots(s, baby[r], ps.log_scale).real
        assert np.abs(z - np.roll(np.tile(qv.astype(np.float64), ps.n // 16), -r)).max() < 2.0 ** -10


@pytest.mark.parametrize("logN,big", [(8, False), (12, False), (13, True)])
def test_seed_compressed_query_upload(logN, big):
    """the query uploaded as (c0, seed): the expanded uniform half equals the oracle's, and the imported ciphertext is the
    one a full upload gives"""
    import torch

    ps = synth.ParamSet("seed", logN, synth.Q50, synth.P60, 40, 16, 4, -18) if big else synth.small_params(logN, 16, 4, L=2)
    p = Pair(ps, key_seed=logN)
    g, o, b = p.g, p.o, p.b
    seed, stream = 0xC0FFEE + logN, 23
    a = g.expand_uniform(seed, stream)
    assert np.array_equal(a, o.expand_uniform(seed, stream))
    qv = synth.toy_query(logN, dim=16)
    ct_o = o.encrypt_query(p.km.s, qv, a, p.km.ct_e)
    ct_g = g.encrypt_query(p.km.s, qv, a, p.km.ct_e)
    assert np.array_equal(ct_g, ct_o) and np.array_equal(ct_g[1], a)
    full = g.import_(b.KIND_CT, ct_g, 1)
    seeded = g.import_seeded_ct(ct_g[0], seed, stream)   # half the bytes on the wire
    g.sync()
    assert torch.equal(full[: seeded.numel()], seeded)


def test_sizes_follow_the_storage_formula():
    """hann_sizeof against the closed forms: 8*L*R bytes per encoded row (half of every transformed plaintext is the
    mirror image of the other half and is not stored), 32*L*R per encrypted row (the paper's 80*L*R of Sec. 2 without
    its 2.5x serialization overhead)"""
    from paper_2608_21131_b200 import binding as b

    for ps in (synth.small_params(10, 16, 4, L=2), synth.FULL16):
        g = b.Context(ps)
        assert g.sizeof(b.SIZE_ROWS_PER_BLOCK) == ps.n
        assert g.sizeof(b.SIZE_PT_BLOCK) == 8 * ps.L * ps.R * ps.n
        assert g.sizeof(b.SIZE_CTDB_BLOCK) == 32 * ps.L * ps.R * ps.n
        assert g.sizeof(b.SIZE_CT) == 2 * ps.L * ps.N * 8 and g.sizeof(b.SIZE_BABY) == ps.B * g.sizeof(b.SIZE_CT)
        assert g.sizeof(b.SIZE_INNER) == ps.G * g.sizeof(b.SIZE_CT)
        assert g.sizeof(b.SIZE_EVK) == ps.L * 2 * (ps.L + 1) * ps.N * 8


def random_shapes(count, seed):
    """seeded random parameter shapes: ring 2^4..2^11, 1..4 ciphertext primes of 30..48 bits, R | n, B | R, ragged row
    counts over up to three blocks, dim <= R"""
    from oracle.oracle import find_primes

    rng = np.random.default_rng(seed)
    out = []
    for _ in range(count):
        logN = int(rng.integers(4, 12))
        n = 1 << (logN - 1)
        L = int(rng.integers(1, 5))
        bits = int(rng.choice([30, 36, 42, 48]))
        R = 1 << int(rng.integers(1, min(logN - 1, 7) + 1))
        B = 1 << int(rng.integers(0, int(np.log2(R)) + 1))
        dim = int(rng.integers(1, R + 1))
        n_rows = int(rng.integers(1, 3 * n + 1))
        q = find_primes(bits, 13, L)
        p = find_primes(bits + 8, 13, 1)[0]
        # the scale leaves room for scale^2 * |score| under the modulus and keeps the encoding error small
        log_scale = min(25, (bits * L - 6) // 2)
        tol = -10 if log_scale >= 25 else -(log_scale - 12)
        out.append(pytest.param(logN, R, B, tuple(q), p, log_scale, tol, dim, n_rows,
                                id="N%d-R%d-B%d-L%d-%db-dim%d-rows%d" % (logN, R, B, L, bits, dim, n_rows)))
    return out


@pytest.mark.parametrize("logN,R,B,q,p,log_scale,tol,dim,n_rows", random_shapes(14, 20260825))
def test_level_bit_exact_random_shapes(logN, R, B, q, p, log_scale, tol, dim, n_rows):
    ps = synth.ParamSet("rand", logN, q, p, log_scale, R, B, tol)
    pair = Pair(ps, key_seed=n_rows)
    rows = synth.toy_corpus(n_rows, rows=n_rows, dim=dim)
    qv = np.zeros(R, dtype=np.float32)
    qv[:dim] = synth.toy_query(n_rows + 1, dim=dim)
    run_level(pair, rows, qv)


@pytest.mark.parametrize("logN,R,B,L,nb", [(10, 128, 32, 4, 3), (10, 128, 64, 3, 2), (9, 64, 16, 2, 2), (8, 8, 8, 1, 1), (10, 128, 32, -3, 2)])
@pytest.mark.parametrize("f64", [1, 0])
def test_multiply_accumulate_extreme_residues(logN, R, B, L, nb, f64):
    """The multiply-accumulate on residues at the ends of their range (0, 1, q-1 and the two values around q/2, where the
    balanced lift of the FP64 sums changes sign), written straight into the transform-domain buffers, against the
    definition inner[g][c][l][t] = sum_b pt[g][b][l][t'] baby[b][c][l][t] mod q (t' = t or its mirror N-1-t in the
    half-size stored plaintext) in exact integers; both arithmetic variants of the kernel."""
    import torch

    from paper_2608_21131_b200 import binding as b

    if L < 0:
        # a chain that starts with a 58-bit prime, as the membership circuit's does: that limb takes 128-bit integer sums inside
        # the same kernel (FP64 variant) or the whole level goes through the generic kernel (integer variant)
        from oracle.oracle import find_primes

        L = -L
        ps = synth.ParamSet("mixed", logN, tuple(find_primes(58, logN + 1, 1)) + tuple(synth.Q50[: L - 1]), synth.P60, 40, R, B, -18)
    else:
        ps = synth.small_params(logN, R, B, L=L, big=True)
    g = b.Context(ps)
    g.set_tuning(b.TUNE_MAC_F64, f64)
    N, n, G = ps.N, ps.n, ps.G
    q = np.array(ps.q, dtype=object)
    t = np.arange(N)
    ends = lambda ql: [0, 1, ql - 1, (ql - 1) // 2, (ql + 1) // 2]
    tops = lambda ql: [ql - 1, ql - 2, (ql + 1) // 2]
    baby = np.zeros((B, 2, L, N), dtype=np.uint64)
    pt = np.zeros((nb, G, B, L, n), dtype=np.uint64)
    for l in range(L):
        e, f = np.array(ends(int(q[l])), dtype=np.uint64), np.array(tops(int(q[l])), dtype=np.uint64)
        for bb in range(B):
            for c in range(2):
                baby[bb, c, l] = e[(bb + 2 * c + t) % 5]
            for gg in range(G):
                for blk in range(nb):
                    pt[blk, gg, bb, l] = f[(gg + bb + blk + t[:n]) % 3]
    # one position where every product is the largest possible on both sides of the balanced lift
    for l in range(L):
        ql = int(q[l])
        baby[:, :, l, 5] = (ql + 1) // 2
        baby[:, :, l, 6] = (ql - 1) // 2
        pt[:, :, :, l, 5] = ql - 1
        pt[:, :, :, l, 6] = ql - 1
    assert g.sizeof(b.SIZE_BABY) == baby.nbytes and g.sizeof(b.SIZE_PT_BLOCK) * nb == pt.nbytes
    dev = lambda a: torch.from_numpy(a.view(np.int64)).to(g.device)
    inner = g.score_level(dev(baby), dev(pt), nb, g.workspace(nb))
    g.sync()
    got = inner.cpu().numpy().view(np.uint64)[: nb * G * 2 * L * N].reshape(nb, G, 2, L, N)
    mirror = np.where(t < n, t, N - 1 - t)
    for l in range(L):
        ql = int(q[l])
        bo = baby[:, :, l].astype(object)
        for blk in range(nb):
            for gg in range(G):
                po = pt[blk, gg, :, l][:, mirror].astype(object)      # [B][N]
                for c in range(2):
                    want = (po * bo[:, c]).sum(axis=0) % ql
                    assert np.array_equal(got[blk, gg, c, l].astype(object), want), (l, blk, gg, c)
