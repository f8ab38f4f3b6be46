"""The C-ABI library: it loads, exports every function the header declares, the binding covers them, and argument
validation that needs no GPU returns the documented codes.  No compute call is made here."""
import ctypes as C
import os
import re

import pytest

from paper_2608_21131_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def declared_functions():
    src = open(os.path.join(ROOT, "include", "hann.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(hann_[a-z0-9_]+)\s*\(", src)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_functions()
    assert len(names) >= 20 and "hann_score_level" in names and "hann_keyswitch" in names
    for n in names:
        f = getattr(lib, n)  # raises AttributeError if the symbol is missing
        assert f.argtypes is not None or n in ("hann_kernel_classes",), n


def test_binding_constants_match_the_header():
    """Every enumerator and #define of the header that the binding mirrors has the header's value (status codes, size and
    kind selectors, tuning knobs, the prime-count limit)."""
    src = open(os.path.join(ROOT, "include", "hann.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    header = {n: int(v) for n, v in re.findall(r"\b(HANN_[A-Z0-9_]+)\s*=\s*(-?\d+)", src)}
    header.update({n: int(v) for n, v in re.findall(r"#define\s+(HANN_[A-Z0-9_]+)\s+\(?(-?\d+)\)?", src)})
    assert len(header) >= 25
    mirrored = 0
    for name, value in header.items():
        short = name[len("HANN_"):]
        for cand in (name, short, short[1:] if short.startswith("E") and short[1:] in ("INVAL", "SHAPE", "NOKEY", "WORKSPACE", "CUDA", "NOMEM") else None):
            if cand and hasattr(binding, cand):
                assert getattr(binding, cand) == value, (name, value, getattr(binding, cand))
                mirrored += 1
                break
    assert mirrored >= 20
    # every tuning knob of the header is mirrored
    for name in header:
        if name.startswith("HANN_TUNE_"):
            assert hasattr(binding, name[len("HANN_"):]), name


def test_parameter_validation_without_a_device(lib):
    ps = synth.small_params(8, 8, 4, L=2)

    def create(**kw):
        p = binding.Params()
        q = kw.get("q", ps.q)
        p.logN, p.L, p.p = kw.get("logN", ps.logN), len(q), kw.get("p", ps.p)
        p.log_scale, p.R, p.B, p.device = ps.log_scale, kw.get("R", ps.R), kw.get("B", ps.B), kw.get("device", 0)
        for i, v in enumerate(q):
            p.q[i] = v
        h = C.c_void_p()
        rc = lib.hann_ctx_create(C.byref(p), C.byref(h))
        if rc == 0:
            lib.hann_ctx_destroy(h)
        return rc

    assert create(logN=3) == binding.EINVAL
    assert create(logN=17) == binding.EINVAL
    assert create(B=3) == binding.EINVAL                      # B must divide R
    assert create(R=24) == binding.EINVAL                     # R must divide n
    assert create(q=(ps.q[0], ps.q[0] + 2)) == binding.EINVAL  # composite
    assert create(q=(ps.q[0], ps.q[0])) == binding.EINVAL      # repeated prime
    assert create(p=97) == binding.EINVAL                     # prime but not 1 mod 2N
    assert create(device=99) in (binding.ECUDA,)              # no such device
    assert lib.hann_ctx_create(None, None) == binding.EINVAL
    assert lib.hann_sizeof(None, binding.SIZE_CT) == binding.EINVAL
    assert lib.hann_workspace_bytes(None, 1) == binding.EINVAL
    assert lib.hann_sync(None) == binding.EINVAL
    assert lib.hann_last_error(None) == b"null context"
    lib.hann_ctx_destroy(None)  # a no-op


def test_context_refuses_to_run_without_cuda():
    import torch

    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(RuntimeError):
        binding.Context(synth.TOY)


def test_product_path_is_independent_of_the_oracle_and_of_scratch_files():
    """the package never imports the CPU oracle (only tests, the smoke check and bench.py's CPU legs may), the oracle never
    imports the package's CUDA side, and nothing that is committed reads the scratch folder"""
    import subprocess

    pkg = os.path.join(ROOT, "paper_2608_21131_b200")
    for name in os.listdir(pkg):
        if name.endswith(".py"):
            src = open(os.path.join(pkg, name)).read()
            assert not re.search(r"^\s*(from|import)\s+oracle\b", src, flags=re.M), name
    for name in ("oracle.py",):
        src = open(os.path.join(ROOT, "oracle", name)).read()
        assert not re.search(r"paper_2608_21131_b200\s*(\.|import)\s*(binding|build)", src) and "libhann.so" not in src
    csrc = os.path.join(pkg, "csrc")
    for name in os.listdir(csrc):
        assert "oracle" not in open(os.path.join(csrc, name)).read().lower(), name
    assert "hann.h" not in open(os.path.join(ROOT, "oracle", "hann_oracle.c")).read()
    tracked = subprocess.run(["git", "ls-files"], cwd=ROOT, capture_output=True, text=True).stdout.split()
    for f in tracked:
        if f.endswith((".py", ".cu", ".cuh", ".h", ".c", ".cpp")) and f != "tests/test_abi.py":
            assert not re.search(r"(^|[\"'/\s])_work(/|[\"'])", open(os.path.join(ROOT, f)).read()), f
