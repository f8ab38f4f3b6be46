"""hann_keyswitch_static -- the key switch for hosts that cannot allocate device memory or lend a workspace (a request
handler that must not hit the device-wide synchronisation of cudaMalloc, a process whose memory pool is fully
committed).  Its scratch is a fixed array inside the library, shared by all calls on a device and never cleared, so
the check is: through the C ABI, two calls in a row with different inputs must each give exactly the bits the CPU
oracle's key switch gives -- and therefore those of hann_keyswitch, which is compared as well (integer work: no
tolerance) -- whatever the previous call left behind, and the call must leave the amount of free device memory as it
found it.  Rings too large for the built-in
array must be refused with a clear error.  This file sorts last on purpose: a run that stops at the first failure has
then already run every other test."""
import numpy as np
import pytest

from paper_2608_21131_b200 import synth
from tests.helpers import make_oracle, oracle_keys

pytestmark = pytest.mark.gpu


def test_static_scratch_keyswitch_matches_workspace_keyswitch_twice():
    from paper_2608_21131_b200 import binding as b

    ps = synth.TOY  # N = 2^12, L = 2: 0.6 MiB of scratch, inside the 4 MiB limit
    g = b.Context(ps)
    km = synth.key_material(ps, 9, rots=[1, 8])
    g.load_keys(g.keygen_from_samples(km.s, km.rots, km.evk_a, km.evk_e), km.rots)
    o = make_oracle(ps)
    evk_o = dict(zip(km.rots, oracle_keys(o, km)))
    ws = g.workspace(1)
    assert g.lib.hann_static_scratch_bytes() == 4 << 20
    # the scratch one key switch carves is what the workspace variant is promised, and fits the built-in array
    assert g.workspace_bytes(1) >= 0 and g.lib.hann_keyswitch_bytes(g.h) <= min(g.workspace_bytes(1), 4 << 20)
    rng = np.random.default_rng(5)
    ks0s, ks1s = g.alloc(g.sizeof(b.SIZE_POLY)), g.alloc(g.sizeof(b.SIZE_POLY))
    for call, rot in enumerate((8, 1)):  # second call: other key, other input, scratch still dirty from the first
        d = np.stack([rng.integers(0, q, size=ps.N, dtype=np.uint64) for q in ps.q])
        dev = g.import_(b.KIND_POLY, d[None], 1)
        want0, want1 = g.keyswitch(rot, dev, ws)
        g.sync()
        ks0s.zero_(); ks1s.zero_()
        g.torch.cuda.synchronize()
        free_before = g.torch.cuda.mem_get_info(g.device)[0]
        got0, got1 = g.keyswitch_static(rot, dev, ks0s, ks1s)
        g.sync()
        assert g.torch.cuda.mem_get_info(g.device)[0] == free_before, "the call changed the free device memory"
        ks0_o, ks1_o = o.keyswitch(d, evk_o[rot])
        got0, got1 = g.export(b.KIND_POLY, got0, 1), g.export(b.KIND_POLY, got1, 1)
        assert np.array_equal(got0[0, 0], ks0_o) and np.array_equal(got1[0, 0], ks1_o), call
        assert np.array_equal(got0, g.export(b.KIND_POLY, want0, 1)), call
        assert np.array_equal(got1, g.export(b.KIND_POLY, want1, 1)), call


def test_static_scratch_keyswitch_refuses_large_rings_and_profiling():
    from paper_2608_21131_b200 import binding as b

    ps = synth.ParamSet("n15-small", 15, synth.Q50, synth.P60, 40, 128, 32, -18)
    g = b.Context(ps)
    km = synth.key_material(ps, 9, rots=[1])
    g.load_keys(g.keygen_from_samples(km.s, km.rots, km.evk_a, km.evk_e), km.rots)
    poly = g.alloc(g.sizeof(b.SIZE_POLY))
    poly.zero_()
    with pytest.raises(b.HannError) as ei:
        g.keyswitch_static(1, poly)
    assert ei.value.code == b.ESHAPE and "too large" in str(ei.value)
    # the workspace variant still serves this ring
    g.keyswitch(1, poly, g.workspace(1))
    g.sync()
    small = b.Context(synth.TOY)
    small.kernel_profile(True)
    with pytest.raises(b.HannError) as ei:
        small.keyswitch_static(1, small.alloc(small.sizeof(b.SIZE_POLY)))
    assert ei.value.code == b.EINVAL
    small.kernel_profile(False)
