"""The stand-ins for a memory checker (none is available on the GPUs this library is developed on): workspace guards behind
every sub-buffer, checked after real work, and a -DHANN_DEBUG build whose kernels range-check their gathered indices.  Every
check here is expected to PASS: nothing provokes a bad access."""
import os
import subprocess
import sys

import numpy as np
import pytest

from paper_2608_21131_b200 import build, synth
from tests.helpers import Pair

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("logN,R,B,L,big,n_rows", [(10, 64, 8, 2, False, 1500), (12, 64, 8, 3, True, 4200)])
def test_workspace_guards_survive_a_level(logN, R, B, L, big, n_rows):
    """guards behind every workspace sub-buffer of the server-side calls (baby rotations, encoding, Horner and lazy giant
    steps, key switch, rescale, the host-buffer level) are intact afterwards, and the results are the oracle's bits"""
    import torch

    ps = synth.small_params(logN, R, B, L=L, big=big)
    if big:
        ps = ps.with_(log_scale=40)
    p = Pair(ps, key_seed=logN)
    g, o, b = p.g, p.o, p.b
    rows, qv = synth.toy_corpus(logN, rows=n_rows, dim=R), synth.toy_query(logN + 1, dim=R)
    ct_o, ct_g = p.query(qv)
    nb = g.n_blocks(n_rows)
    ws = g.workspace(nb)
    g.debug_canaries(True)
    baby = g.query_prepare(g.import_(b.KIND_CT, ct_g, 1), ws)
    checked, damaged = g.debug_verify()
    assert checked >= 4 and damaged == 0
    pt = g.encode_candidates(torch.from_numpy(rows).to(g.device), ws)
    inner = g.score_level(baby, pt, nb, ws)
    score = g.rotate_sum(inner, nb, ws)
    checked, damaged = g.debug_verify()
    assert checked >= 5 and damaged == 0
    d = np.stack([np.random.default_rng(1).integers(0, q, size=ps.N, dtype=np.uint64) for q in ps.q])
    ks0, ks1 = g.keyswitch(3, g.import_(b.KIND_POLY, d[None], 1), ws)
    assert g.debug_verify() == (4, 0)
    small = g.rescale(score, nb, ws)
    assert g.debug_verify() == (2, 0)
    # a later call on the same workspace retires the guards its own sub-buffers cover: nothing is reported as damaged
    g.keyswitch(3, g.import_(b.KIND_POLY, d[None], 1), ws)
    g.rescale(score, nb, ws)
    checked, damaged = g.debug_verify()
    assert 2 <= checked <= 6 and damaged == 0
    ws_host = g.alloc(g.level_host_bytes(n_rows))
    host = g.score_level_host(ct_g, rows, ws_host)
    checked, damaged = g.debug_verify()
    assert checked >= 9 and damaged == 0
    g.debug_canaries(False)
    # the guarded runs computed the right thing
    baby_o = o.baby_set(ct_o, p.evk_o)
    score_h = g.export(b.KIND_CT, score, nb)
    for blk in range(nb):
        sc_o, _, _ = o.score_block(rows[blk * ps.n:(blk + 1) * ps.n], baby_o, p.evk_o[B - 1])
        assert np.array_equal(score_h[blk], sc_o) and np.array_equal(host[blk], sc_o)
    k0, k1 = o.keyswitch(d, p.evk_o[2])
    assert np.array_equal(g.export(b.KIND_POLY, ks0, 1)[0, 0], k0) and np.array_equal(g.export(b.KIND_POLY, ks1, 1)[0, 0], k1)
    got = g.export_limbs(small, 2 * nb, L - 1).reshape(nb, 2, L - 1, ps.N)
    assert np.array_equal(got[0], o.compact(score_h[0], L - 1, True))
    assert g.debug_verify() == (0, 0)       # switched off: nothing is carved with guards any more


def test_a_damaged_guard_is_reported():
    """the verify kernel does notice an overwritten guard: the test itself overwrites one word of a guard (a host-side
    copy into the caller's own workspace: no kernel misbehaves), verify reports exactly one damaged guard, and the context
    keeps working"""
    from paper_2608_21131_b200 import binding as b

    ps = synth.small_params(10, 16, 4, L=2)
    p = Pair(ps, key_seed=2)
    g = p.g
    ct = g.import_(b.KIND_CT, p.query(synth.toy_query(3, dim=16))[1], 1)
    ws = g.workspace(1)
    g.debug_canaries(True)
    g.query_prepare(ct, ws)
    g.sync()
    # the first sub-buffer of the call is c1 (L * N words); its guard follows it
    ws[ps.L * ps.N + 5] = 12345
    with pytest.raises(b.HannError) as ei:
        g.debug_verify()
    assert ei.value.code == b.ECUDA and "past the end" in str(ei.value)
    g.query_prepare(ct, ws)
    assert g.debug_verify()[1] == 0


def test_debug_build_passes_its_own_range_checks():
    """the -DHANN_DEBUG library (every gather index checked, a failing check skips the access and raises the context's
    flag) runs the small-ring parity tests of the release library in a process of its own: same bits, no flag raised"""
    lib = build.build_debug()
    code = (
        "import sys\n"
        "from paper_2608_21131_b200 import binding as b\n"
        "assert b.load_library().hann_debug_build() == 1\n"
        "import pytest\n"
        "sys.exit(pytest.main(['-q', '-x', '-m', 'gpu', '-p', 'no:cacheprovider', 'tests/test_gpu_parity.py', '-k',\n"
        "    'level_bit_exact_small or lazy_giant_steps or keyswitch_matches or seed_compressed or host_buffer_level']))\n"
    )
    env = dict(os.environ, HANN_LIB=lib)
    out = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert out.returncode == 0, out.stdout[-3000:] + out.stderr[-2000:]
    assert " passed" in out.stdout and "failed" not in out.stdout
    # and the release library says what it is
    from paper_2608_21131_b200 import binding as b

    assert b.load_library().hann_debug_build() == 0
