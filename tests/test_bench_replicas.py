"""bench.py across ranks: the path has no exchange step, so N ranks are N independent replicas; the only cross-rank
logic is the barrier and the max-over-ranks of the measured time.  Covered here with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent(
    """
    import os, sys, json
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    dist.barrier()
    ms = bench.max_over_ranks(10.0 * (rank + 1), dist, torch.device("cpu"))
    val = bench.replica_throughput(1000, world, ms * 1e-3)
    with open(os.path.join(%r, "rank%%d.json" %% rank), "w") as f:
        json.dump({"rank": rank, "ms": ms, "value": val}, f)
    dist.destroy_process_group()
    """
)


def test_max_over_ranks_and_replica_value_with_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % (ROOT, str(tmp_path)))
    out = subprocess.run(
        [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
         "--master-port", "29731", str(script)],
        capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    recs = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in (0, 1)]
    assert sorted(r["rank"] for r in recs) == [0, 1]
    for r in recs:
        assert r["ms"] == 20.0                 # the slower rank's time on both ranks
        assert abs(r["value"] - 2 * 1000 / 0.020) < 1e-6


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, timeout=120, env=env, cwd=ROOT)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_gpus_flag_launches_the_ranks_itself():
    """`python bench.py --gpus 2` with no launcher around it starts two ranks under torch's launcher (rendezvous on
    127.0.0.1, a free port) and rank 0 prints the one JSON line -- exercised on CPU with the reference arm (the oracle on
    the toy configuration), whose other rank exits without work"""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--config", "0",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0 and rec["cpu_baseline"]["kind"] == "oracle"


def test_single_process_identity():
    sys.path.insert(0, ROOT)
    import torch
    import bench

    assert bench.max_over_ranks(3.5, None, torch.device("cpu")) == 3.5
    assert bench.replica_throughput(100, 1, 0.5) == 200.0


def test_algorithmic_work_matches_the_per_row_figures():
    """the roofline numerators of bench.py against the closed forms of the design: a scored row costs the multiply-
    accumulate 8*L*R bytes of stored plaintext read (half of every transformed plaintext mirrors the other half) +
    32*L*G bytes of partial sums written (4,096 + 512 at L = 4, R = 128, G = 4), the baby set is read once per level,
    and pass B of a block's encoding is R*L half-size transforms"""
    import types

    import bench

    L, logN, R, B = 4, 16, 128, 32
    N, n, G = 1 << logN, 1 << (logN - 1), R // B
    ctx = types.SimpleNamespace(L=L, N=N, n=n, logN=logN, R=R, B=B, G=G)
    for n_blocks in (1, 7):
        w = bench.algorithmic_work(ctx, n_blocks, n_blocks * n)
        bound, mac_bytes, units = w["mac"]
        assert bound == "hbm" and units == n_blocks
        assert mac_bytes == n_blocks * n * (8 * L * R + 32 * L * G) + B * 2 * L * N * 8
        assert 8 * L * R + 32 * L * G == 4608
        # pass B of the forward transforms: 8 of the 16 stages, 8 binary64 instructions per butterfly; the plaintexts'
        # transforms run on half of the chunks
        pt_polys = n_blocks * R * L
        ks_polys = (L * (L + 1) + (B - 1) * 2 * L) + (G - 1) * n_blocks * (L * (L + 1) + 2 * L)
        assert w["ntt_fwd_b"][2] == pt_polys + ks_polys
        assert w["ntt_fwd_b"][1] == (pt_polys * (N // 4) + ks_polys * (N // 2)) * 8 * 8
        # and the bytes those transforms move: half-size plaintext polynomials W/2 in and out, key-switch polynomials W
        assert bench.algorithmic_work.transform_bytes["ntt_fwd_b"] == (pt_polys + 2 * ks_polys) * 8 * N
