#!/usr/bin/env python
"""Benchmark of the encrypted scoring hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 0..4]

One "step" is one pass of the whole server-side path for one encrypted query over one routing level:
query_prepare (hoisted baby rotations) + encode_candidates + score_level (ct x pt multiply-accumulate) +
rotate_sum (Horner with hybrid key switching).  The default workload is the face-corpus-like single level
(222,049 rows, 512 -> 128 dims, N = 2^16, 4 x ~50-bit + ~60-bit primes, scale 2^40), all inputs synthetic.
Prints ONE JSON line on rank 0.  With N > 1 every rank runs an independent replica of the workload on its own
GPU (the path has no exchange step); the value is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "encrypted candidates scored/sec"
UNIT = "candidates/s"


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d.get("sm_max_mhz", 1965.0)), "measured"
    return 6650.0, 1965.0, "fallback"


class ClockSampler:
    """samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs"""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for ln in self.proc.stdout:
            self.lines.append(ln)

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(x, dist, device):
    """the slowest rank's value of a per-rank scalar (identity without a process group)"""
    import torch

    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(units_per_rank, world, seconds_slowest):
    """whole-job throughput of `world` independent replicas: all units divided by the slowest rank's time"""
    return world * units_per_rank / seconds_slowest


def bench_keys(ctx, ps, args):
    """key material of a run: rotations 1..B, plus 2B..(G-1)B when the giant steps are evaluated in the lazy order"""
    from paper_2608_21131_b200 import binding, synth, workloads as wl

    rots = list(range(1, ps.B + 1)) + [g * ps.B for g in range(2, ps.G)]
    if args.giant == "lazy":
        ctx.set_tuning(binding.TUNE_GIANT_LAZY, 1)
    if args.lazy_lanes:
        ctx.set_tuning(binding.TUNE_LAZY_LANES, args.lazy_lanes)
    if args.mac_f64 is not None:
        ctx.set_tuning(binding.TUNE_MAC_F64, args.mac_f64)
    if args.pair_b32:
        ctx.set_tuning(binding.TUNE_PAIR_B32, 1)
    if args.groups is not None:
        ctx.set_tuning(binding.TUNE_HOST_GROUPS, args.groups)
    km = synth.key_material(ps, wl.KEY_SEED, rots=rots)
    ctx.load_keys(ctx.keygen_from_samples(km.s, km.rots, km.evk_a, km.evk_e), km.rots)
    return km


def build_workload(config, rows_override=None, logn=16, baby=None):
    from paper_2608_21131_b200 import workloads as wl, synth

    if baby:
        ps, rows, q, name = build_workload(config, rows_override, logn)
        return ps.with_(B=baby), rows, q, name + ", B=%d" % baby
    if config == 0:
        ps, rows, q = wl.toy()
        return ps, rows, q, "toy: 4,096 rows, dim 64, N=2^12, scale 2^25"
    if config == 1:
        n = rows_override or 222_049
        ps, lvl, q, _ = wl.face_level(rows=n)
        return ps, lvl.rows, q, "face-like flat level: %d rows, dim 512->128, N=2^16, 4x50b+60b primes, scale 2^40" % n
    if config == 4:
        base = rows_override or (1 << 18)
        ps, lvl = wl.sweep_level(base, ps=synth.FULL15 if logn == 15 else synth.FULL16)
        q = synth.toy_query(wl.query_seed(0), dim=ps.R)
        return ps, lvl.rows, q, "sweep: %d wanted rows inflated x4 to %d scored rows, dim 128, N=2^%d" % (base, lvl.rows.shape[0], ps.logN)
    raise SystemExit("unknown config %r" % config)


# DRAM bytes (read + write) per unit of work of the transform kernels, from the ncu captures summarised under profiles/
# (small case: one block of 32,768 rows; traffic grows in proportion to the units): pass B of a half-size plaintext
# transform, pass B of a full key-switch transform, the fused FFT tail + pass A per plaintext
NCU_DRAM_BYTES = {"pass_b_plaintext_poly": 212.4e6 / 512, "pass_b_full_poly": 490.4e6 / 512, "fft_b_plaintext": 153.6e6 / 128}


def ncu_traffic_per_step(kernel, ctx, n_blocks):
    """DRAM traffic of one step of a kernel class, scaled from the ncu captures (None where none was taken)"""
    L, B, G, R = ctx.L, ctx.B, ctx.G, ctx.R
    if kernel == "ntt_fwd_b":
        ks_polys = (L * (L + 1) + (B - 1) * 2 * L) + (G - 1) * n_blocks * (L * (L + 1) + 2 * L)
        return n_blocks * R * L * NCU_DRAM_BYTES["pass_b_plaintext_poly"] + ks_polys * NCU_DRAM_BYTES["pass_b_full_poly"]
    if kernel == "fft_b":
        return n_blocks * R * NCU_DRAM_BYTES["fft_b_plaintext"]
    return None


def algorithmic_work(ctx, n_blocks, n_rows):
    """Algorithmic work of ONE step per kernel class: bytes for the HBM-bound kernels, binary64 instructions for the
    transform kernels (moduli below 2^50 run their butterflies on the FP64 pipe: exact product = multiply + fma,
    quotient = multiply + round, remainder = fma + add, butterfly = add + subtract: 8 per butterfly; an FFT butterfly with
    separately rounded products and sums is 10).  The transform of an encoded plaintext takes every value twice, so only
    its first stage (a product and a sum per pair: 7 instructions) runs in full; the other stages and the stored
    plaintext are half size.  Returns {class: (bound, amount, units per step)}."""
    L, N, B, G, R = ctx.L, ctx.N, ctx.B, ctx.G, ctx.R
    n, logN = ctx.n, ctx.logN
    b = min(logN, 8)
    a = logN - b
    W = 8 * N
    items_rot = (G - 1) * n_blocks  # key switches of the rotate-and-sum
    pt_polys = n_blocks * R * L       # half-size transforms
    ks_polys = (L * (L + 1) + (B - 1) * 2 * L) + items_rot * (L * (L + 1) + 2 * L)
    inv_polys = (L + (B - 1) * 2) + items_rot * (L + 2)
    lift_src = [(L, L + 1), ((B - 1) * 2, L)] + [(items_rot * L, L + 1), (items_rot * 2, L)]  # (sources, targets each)
    lift_ops = sum(src * (1 + tgt) * a * (N // 2) * 8 for src, tgt in lift_src)
    pass_a_half = (N // 2) * 7 + (a - 1) * (N // 4) * 8  # first stage in full (one output per pair), then half the butterflies
    # the transform kernels also move their polynomials through HBM once in and once out (half-size plaintexts: W/2 each
    # way); whichever ceiling gives the longer ideal time is the bound the roofline reports
    transform_bytes = {
        "ntt_fwd_b": pt_polys * W + ks_polys * 2 * W,
        "ntt_inv_b": inv_polys * 2 * W,
        "fft_b": n_blocks * R * (n * 16 + L * (W // 2)),
    }
    algorithmic_work.transform_bytes = transform_bytes
    return {
        "mac": ("hbm", n_blocks * R * L * (W // 2) + B * 2 * L * W + n_blocks * G * 2 * L * W, n_blocks),
        # one digit set under B-1 streamed keys (query_prepare) / one key under many digit sets (rotate_sum, L2-resident key)
        "ks_inner_keys": ("hbm", (B - 1) * (L * 2 * (L + 1) * W + 2 * (L + 1) * W) + L * (L + 1) * W, B - 1),
        "ks_inner": ("hbm", (G - 1) * (L * 2 * (L + 1) * W + n_blocks * (L * (L + 1) * W + 2 * (L + 1) * W)), items_rot),
        "ntt_fwd_b": ("alu", (pt_polys * (N // 4) + ks_polys * (N // 2)) * b * 8, pt_polys + ks_polys),
        "ntt_inv_b": ("alu", inv_polys * (N // 2) * b * 8, inv_polys),
        "lift_digits": ("alu", lift_ops, inv_polys),
        "fft_a": ("hbm", n_blocks * R * (n * 16) + n_rows * R * 4, n_blocks * R),
        "fft_b": ("alu", n_blocks * R * ((a - 1) * (n // 2) * 10 + L * pass_a_half), n_blocks * R),
    }


def run_ours(args):
    import torch
    from paper_2608_21131_b200 import binding, synth, workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the scoring path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    ps, rows_np, qR, wname = build_workload(args.config, args.rows, args.logn, args.baby)
    n_rows = rows_np.shape[0]
    ctx = binding.Context(ps, device=local)
    if args.encode_group:
        ctx.set_tuning(binding.TUNE_ENCODE_GROUP, args.encode_group)
    km = bench_keys(ctx, ps, args)
    ct_host = ctx.encrypt_query(km.s, qR, km.ct_a, km.ct_e)
    ct_dev = ctx.import_(binding.KIND_CT, ct_host, 1)
    rows_dev = torch.from_numpy(rows_np).to(ctx.device)
    nb = ctx.n_blocks(n_rows)
    ws = ctx.workspace(nb)
    baby = ctx.alloc(ctx.sizeof(binding.SIZE_BABY))
    pt = ctx.alloc(nb * ctx.sizeof(binding.SIZE_PT_BLOCK))
    inner = ctx.alloc(nb * ctx.sizeof(binding.SIZE_INNER))
    score = ctx.alloc(nb * ctx.sizeof(binding.SIZE_CT))

    def step():
        ctx.query_level(ct_dev, rows_dev, ws, baby, pt, inner, score)

    def step_staged():  # the same work as four separate calls on one stream (per-stage timing)
        ctx.query_prepare(ct_dev, ws, baby)
        ctx.encode_candidates(rows_dev, ws, pt)
        ctx.score_level(baby, pt, nb, ws, inner)
        ctx.rotate_sum(inner, nb, ws, score)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    if args.lean:
        # profiling aid (ncu launch lists and captures): W warm-up steps, K steps, nothing else, no JSON line
        if args.staged:
            # the configuration of the per-kernel timing pass below: four calls per step on one stream, rotate-and-sum on
            # one lane (the launch list of this mode is the one whose shares compare with the "kernels" of the JSON line)
            ctx.kernel_profile(True)
        for _ in range(args.warmup + args.steps):
            step_staged() if args.staged else step()
        torch.cuda.synchronize()
        print("lean run: %d steps, %d kernel launches" % (args.warmup + args.steps, ctx.get_stats()["launches"]))
        return 0

    # the clock sampler runs from the warm-up on (nvidia-smi needs ~0.1 s to produce its first line); warm-up and timed
    # steps are the same work, so every sample is taken under the timed region's load
    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    # The timed quantity is a block of exactly K steps between two events.  The block is repeated back to back (no host
    # synchronisation in between) until the timed region has lasted MIN_TIMED_S, so that the clocks are sampled tens of times
    # under sustained load whatever K is; the reported time is the MEDIAN block, the slowest rank's.
    barrier()
    t_probe = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_probe[0].record()
    step()
    t_probe[1].record()
    torch.cuda.synchronize()
    est_block_ms = max(t_probe[0].elapsed_time(t_probe[1]) * args.steps, 1e-3)
    n_timed_blocks = int(min(max(1, np.ceil(args.min_timed_s * 1e3 / est_block_ms)), 2000))
    if dist is not None:  # every rank runs the same number of blocks
        nbt = torch.tensor([n_timed_blocks], device=ctx.device)
        dist.all_reduce(nbt, op=dist.ReduceOp.MAX)
        n_timed_blocks = int(nbt.item())
    l0 = ctx.get_stats()["launches"]
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_timed_blocks + 1)]
    barrier()
    marks[0].record()
    for bi in range(n_timed_blocks):
        for _ in range(args.steps):
            step()
        marks[bi + 1].record()
    barrier()
    clocks = sampler.stop()
    block_ms = [marks[i].elapsed_time(marks[i + 1]) for i in range(n_timed_blocks)]
    launches = ctx.get_stats()["launches"] - l0            # all kernels of the timed region (every block of K steps)
    ms_step = max_over_ranks(float(np.median(block_ms)), dist, ctx.device) / args.steps
    value = replica_throughput(n_rows, world, ms_step * 1e-3)

    # the other evaluation order of the giant steps, same steps, one block of K (reported beside the headline)
    other_order = "horner" if args.giant == "lazy" else "lazy"
    ctx.set_tuning(binding.TUNE_GIANT_LAZY, 1 if other_order == "lazy" else 0)
    for _ in range(3):
        step()
    o0, o1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    o0.record()
    for _ in range(args.steps):
        step()
    o1.record()
    torch.cuda.synchronize()
    other_ms = max_over_ranks(o0.elapsed_time(o1), dist, ctx.device) / args.steps
    got_other = ctx.decrypt_scores(km.s, ctx.export(binding.KIND_CT, score, nb)).reshape(-1)[:n_rows]
    ctx.set_tuning(binding.TUNE_GIANT_LAZY, 1 if args.giant == "lazy" else 0)
    step()

    # correctness of what was timed: decrypted scores against float64 dot products
    score_host = ctx.export(binding.KIND_CT, score, nb)
    got = ctx.decrypt_scores(km.s, score_host).reshape(-1)[:n_rows]
    want = rows_np.astype(np.float64) @ qR.astype(np.float64)
    max_err = float(np.abs(got - want).max())
    check_ok = bool(max_err < 2.0 ** ps.tol_log2)
    other_giant = {"order": other_order, "ms_per_step": other_ms, "value": replica_throughput(n_rows, world, other_ms * 1e-3),
                   "max_abs_score_error": float(np.abs(got_other - want).max())}
    check_ok = check_ok and other_giant["max_abs_score_error"] < 2.0 ** ps.tol_log2

    # per-stage device time (library event timers), median of the timed steps
    aux_steps = min(args.steps, 20)  # the breakdown passes need no more repetitions than that
    ctx.set_timing(True)
    stage = {k: [] for k in ("ms_query_prepare", "ms_encode", "ms_score_level", "ms_rotate_sum")}
    for _ in range(aux_steps):
        step_staged()
        st = ctx.get_stats()
        for k in stage:
            stage[k].append(st[k])
    ctx.set_timing(False)
    stage_ms = {k[3:]: float(np.median(v)) for k, v in stage.items()}

    # output compaction of the level's score ciphertexts (not part of the step: an optional call after it): device time of
    # both forms, bytes the client would download, and the decrypted scores of what comes out
    compaction = {}
    if ps.L >= 2:
        for name, keep, rescale in (("first_2_limbs_exact", min(2, ps.L), False), ("rescale_to_1_limb", 1, True)):
            if keep > ps.L - (1 if rescale else 0) or (not rescale and keep == ps.L):
                continue
            out_c = ctx.alloc(ctx.lib.hann_compact_bytes(ctx.h, nb, keep))
            ctx.compact_scores(score, nb, keep, rescale, ws, out_c)
            torch.cuda.synchronize()
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record()
            for _ in range(aux_steps):
                ctx.compact_scores(score, nb, keep, rescale, ws, out_c)
            c1.record()
            torch.cuda.synchronize()
            small = ctx.export_limbs(out_c, nb * 2, keep).reshape(nb, 2, keep, ps.N)
            got_c = ctx.decrypt_compact(km.s, small, rescale).reshape(-1)[:n_rows]
            compaction[name] = {"ms": c0.elapsed_time(c1) / aux_steps, "bytes_out": int(small.nbytes),
                                "bytes_uncompacted": int(score_host.nbytes),
                                "max_abs_score_error": float(np.abs(got_c - want).max()),
                                "same_top10": bool(np.array_equal(np.argsort(-got_c)[:10], np.argsort(-want)[:10]))}
            del out_c

    # per-kernel device time, live, with an event pair around every launch of the same steps
    ctx.kernel_profile(True)
    for _ in range(aux_steps):
        step_staged()
    kt = ctx.kernel_times()
    ctx.kernel_profile(False)
    total_k = sum(v[0] for v in kt.values()) or 1.0
    kernels = {k: {"ms_per_step": v[0] / aux_steps, "launches_per_step": v[1] / aux_steps, "share": v[0] / total_k}
               for k, v in kt.items() if v[1]}
    hbm_peak, sm_max_mhz, peak_src = read_peaks()
    # arithmetic ceilings measured on this device by the library's own probe kernels: register-resident binary64 modular
    # butterflies (no memory traffic) and 32 x 32 -> 64 multiply-adds
    bfly_peak, madd_peak = ctx.probe_rates()
    work = algorithmic_work(ctx, nb, n_rows)
    dom = max((k for k in kernels if k in work), key=lambda k: kernels[k]["ms_per_step"])
    bound, amount, units = work[dom]
    dom_s = kernels[dom]["ms_per_step"] * 1e-3
    dom_launches = max(kernels[dom]["launches_per_step"], 1)
    # transform work is counted in binary64 instructions, 8 per modular butterfly; the measured ceiling is in butterflies
    alu_peak = bfly_peak / 1e12
    alu_src = "measured: register-resident binary64 modular butterflies of the library's probe kernel"
    other = None
    if bound == "alu":
        # a transform kernel has two ceilings: its butterflies and its polynomial bytes; report the tighter
        tbytes = algorithmic_work.transform_bytes.get(dom)
        amount = amount / 8.0
        alu_frac = amount / dom_s / 1e12 / alu_peak
        if tbytes:
            hbm_frac = tbytes / dom_s / 1e9 / hbm_peak
            if hbm_frac > alu_frac:
                other = {"bound": "alu", "achieved": amount / dom_s / 1e12, "peak": alu_peak, "unit": "T butterflies/s", "frac": alu_frac,
                         "peak_source": alu_src}
                bound, amount = "hbm", tbytes
            else:
                other = {"bound": "hbm", "achieved": tbytes / dom_s / 1e9, "peak": hbm_peak, "unit": "GB/s", "frac": hbm_frac,
                         "peak_source": peak_src + " copy bandwidth"}
    if bound == "hbm":
        achieved, peak, runit = amount / dom_s / 1e9, hbm_peak, "GB/s"
        psrc = peak_src + " copy bandwidth"
    else:
        achieved, peak, runit = amount / dom_s / 1e12, alu_peak, "T butterflies/s"
        psrc = alu_src
    traffic_step = ncu_traffic_per_step(dom, ctx, nb)
    roofline = {"kernel": dom, "bound": bound, "achieved": achieved, "peak": peak, "unit": runit, "frac": achieved / peak,
                "peak_source": psrc, "launches_per_step": kernels[dom]["launches_per_step"],
                "avg_launch_ms": kernels[dom]["ms_per_step"] / dom_launches,
                "algorithmic_per_launch": amount / dom_launches,
                "other_ceiling": other,
                "traffic": traffic_step / dom_launches if traffic_step else None,
                "traffic_source": "ncu dram bytes per polynomial on the 1-block case x polynomials per launch" if traffic_step else None}
    # the streaming kernels against THEIR ceilings: bytes against the measured copy bandwidth, and residue products against the
    # pipe they run on.  By default (HANN_TUNE_MAC_F64) products of residues below 2^50 are summed in pairs of binary64 words,
    # four FP64 operations each, against the FP64 rate the probe's butterflies reach (8 operations per butterfly); products
    # modulo the 60-bit special prime (one limb in L + 1 of the key-switch inner products), and all of them with --mac-f64 0,
    # are 32 x 32 -> 64 multiply-adds (three per product below 2^50, four above) against the measured multiply-add rate.
    L_, N_, B_, G_, R_ = ctx.L, ctx.N, ctx.B, ctx.G, ctx.R
    f64_on = args.mac_f64 is None or args.mac_f64 != 0
    f64_peak = 8.0 * bfly_peak
    # (products on ciphertext-prime limbs, products on the special-prime limb)
    products = {"mac": (nb * R_ * L_ * N_ * 2, 0),
                "ks_inner_keys": ((B_ - 1) * L_ * 2 * L_ * N_, (B_ - 1) * L_ * 2 * N_),
                "ks_inner": ((G_ - 1) * nb * L_ * 2 * L_ * N_, (G_ - 1) * nb * L_ * 2 * N_)}
    hbm_kernels = {}
    for k in ("mac", "ks_inner_keys", "ks_inner"):
        if k in kernels:
            sec = kernels[k]["ms_per_step"] * 1e-3
            gbs = work[k][1] / sec / 1e9
            small, special = products[k]
            f64_ops = 4.0 * small / sec if f64_on else 0.0
            madds = (4.0 * special + (0.0 if f64_on else 3.0 * small)) / sec
            fracs = {"hbm": gbs / hbm_peak, "fp64": f64_ops / f64_peak, "multiply-add": madds / madd_peak}
            hbm_kernels[k] = {"GB/s": gbs, "frac_of_measured_copy": gbs / hbm_peak, "frac_of_8TBps_nominal": gbs / 8000.0,
                              "T_f64_ops_per_s": f64_ops / 1e12, "frac_of_measured_f64_rate": f64_ops / f64_peak,
                              "T_madds_per_s": madds / 1e12, "frac_of_measured_madd_rate": madds / madd_peak,
                              "tighter_ceiling": max(fracs, key=fracs.get)}

    # end to end through the host-buffer entry point: pinned host inputs, copies inside the timed region
    rows_pin = torch.from_numpy(rows_np).pin_memory()
    ct_pin = torch.from_numpy(ct_host.view(np.int64)).pin_memory()
    out_pin = torch.empty((nb, 2, ctx.L, ctx.N), dtype=torch.int64).pin_memory()
    del pt, inner, score, baby, ws
    torch.cuda.empty_cache()
    ws_host = ctx.alloc(ctx.level_host_bytes(n_rows))

    def e2e_step():
        ctx.lib.hann_score_level_host(ctx.h, ct_pin.data_ptr(), rows_pin.data_ptr(), n_rows, rows_np.shape[1], out_pin.data_ptr(),
                                      ws_host.data_ptr(), ws_host.numel() * 8)

    e2e_steps = min(args.steps, 50)
    for _ in range(3):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    torch.cuda.synchronize()
    t_e2e = max_over_ranks(time.perf_counter() - t0, dist, ctx.device)
    e2e_value = replica_throughput(n_rows * e2e_steps, world, t_e2e)
    e2e_same = bool(np.array_equal(out_pin.numpy().view(np.uint64), score_host))
    e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(rows_np.nbytes + ct_host.nbytes),
           "d2h_bytes_per_step": int(out_pin.numel() * 8), "steps": e2e_steps, "matches_device_path": e2e_same}
    # the same call downloading only the first two limbs of the score ciphertexts (exact compaction; the client decrypts
    # the same scores from half the bytes)
    if ps.L > 2:
        ctx.set_tuning(binding.TUNE_HOST_LIMBS, 2)
        out2_pin = torch.empty((nb, 2, 2, ctx.N), dtype=torch.int64).pin_memory()

        def e2e2_step():
            ctx.lib.hann_score_level_host(ctx.h, ct_pin.data_ptr(), rows_pin.data_ptr(), n_rows, rows_np.shape[1], out2_pin.data_ptr(),
                                          ws_host.data_ptr(), ws_host.numel() * 8)

        for _ in range(3):
            e2e2_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e2_step()
        torch.cuda.synchronize()
        t2 = max_over_ranks(time.perf_counter() - t0, dist, ctx.device)
        ctx.set_tuning(binding.TUNE_HOST_LIMBS, ps.L)
        got2 = ctx.decrypt_compact(km.s, out2_pin.numpy().view(np.uint64), False).reshape(-1)[:n_rows]
        e2e["two_limb_download"] = {"value": replica_throughput(n_rows * e2e_steps, world, t2), "unit": UNIT,
                                    "d2h_bytes_per_step": int(out2_pin.numel() * 8),
                                    "scores_identical_to_full_download": bool(np.array_equal(got2, got))}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = cpu_baseline(ps, rows_np, qR, km, n_rows, args.giant)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "timed_blocks": {"count": n_timed_blocks, "steps_each": args.steps, "reported": "median block",
                                                     "ms_min": float(min(block_ms)), "ms_max": float(max(block_ms)),
                                                     "region_s": float(sum(block_ms)) * 1e-3},
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64",
            "data": "synthetic",
            "config": {"workload": wname, "rows": n_rows, "blocks": nb, "R": ps.R, "B": ps.B, "G": ps.G, "logN": ps.logN, "L": ps.L,
                       "giant_steps": "Horner: one key, G-1 key switches in sequence" if args.giant == "horner" else
                                      "lazy: keys of rotations B..(G-1)B, key products summed, one ModDown per block",
                       "l2": "working set per step (%.1f GB of encoded plaintexts) exceeds L2; no flush" %
                             (nb * ctx.sizeof(binding.SIZE_PT_BLOCK) / 1e9),
                       "replicas": "each rank scores the whole level on its own GPU" if world > 1 else "single GPU"},
            "ms_per_query_level": ms_step, "stage_ms": stage_ms, "other_giant_order": other_giant,
            # candidates already encoded and resident (the paper's "warm" case): prepare + multiply-accumulate + rotate-and-sum
            "warm_value": world * n_rows / ((stage_ms["query_prepare"] + stage_ms["score_level"] + stage_ms["rotate_sum"]) * 1e-3),
            "kernels": kernels, "hbm_kernels": hbm_kernels, "roofline": roofline,
            "measured_ceilings": {"f64_butterflies_per_s": bfly_peak, "f64_ops_per_s": 8.0 * bfly_peak, "int32_madds_per_s": madd_peak, "hbm_gbs": hbm_peak,
                                  "ntt_butterflies_per_s": {k: work[k][1] / 8.0 / (kernels[k]["ms_per_step"] * 1e-3)
                                                            for k in ("ntt_fwd_b", "ntt_inv_b", "lift_digits") if k in kernels}}, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": int(launches), "gpu_launches_per_step": launches / (n_timed_blocks * args.steps), "clocks": clocks, "compaction": compaction,
            "check": {"max_abs_score_error": max_err, "tolerance": 2.0 ** ps.tol_log2, "ok": check_ok},
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0 if check_ok else 1


def run_batch(args):
    """Cross-query batching (Sec. 7: score a batch of queries against each loaded region): Q encrypted queries against ONE
    level.  A step = encode the level once + Q query preparations + the batched multiply-accumulate (plaintexts streamed
    once per pair of queries) + rotate-and-sum of the Q x blocks partial sums.  Prints one JSON line: milliseconds per
    batch and per query, candidate-query pairs per second, every query's scores checked against float64 dot products."""
    import torch
    from paper_2608_21131_b200 import binding, synth, workloads as wl

    torch.cuda.set_device(0)
    ps, rows_np, qR, wname = build_workload(args.config, args.rows, args.logn)
    n_rows, Q = rows_np.shape[0], args.queries
    ctx = binding.Context(ps, device=0)
    if args.pair_b32:
        ctx.set_tuning(binding.TUNE_PAIR_B32, 1)
    if args.mac_f64 is not None:
        ctx.set_tuning(binding.TUNE_MAC_F64, args.mac_f64)
    km = synth.key_material(ps, wl.KEY_SEED)
    ctx.load_keys(ctx.keygen_from_samples(km.s, km.rots, km.evk_a, km.evk_e), km.rots)
    rng = np.random.default_rng(wl.KEY_SEED)
    # query 0 is the workload's; the others are its rows' neighbours: unit vectors near random candidates
    qs = [qR] + [(lambda v: (v / np.linalg.norm(v)).astype(np.float32))(rows_np[int(rng.integers(n_rows))] + 0.05 * rng.standard_normal(ps.R))
                 for _ in range(Q - 1)]
    cts = [ctx.import_(binding.KIND_CT, ctx.encrypt_query(km.s, q, km.ct_a, km.ct_e), 1) for q in qs]
    rows_dev = torch.from_numpy(rows_np).to(ctx.device)
    nb = ctx.n_blocks(n_rows)
    ws = ctx.workspace(min(8, Q * nb))
    bw = ctx.sizeof(binding.SIZE_BABY) // 8
    babies = ctx.alloc(Q * bw * 8)
    pt = ctx.alloc(nb * ctx.sizeof(binding.SIZE_PT_BLOCK))
    inner = ctx.alloc(Q * nb * ctx.sizeof(binding.SIZE_INNER))
    score = ctx.alloc(Q * nb * ctx.sizeof(binding.SIZE_CT))

    def step():
        ctx.encode_candidates(rows_dev, ws, pt)
        for q in range(Q):
            ctx.query_prepare(cts[q], ws, babies[q * bw:(q + 1) * bw])
        ctx.score_level_batch(babies, Q, pt, nb, ws, inner)
        ctx.rotate_sum(inner, Q * nb, ws, score)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    ctx.kernel_profile(True)
    for _ in range(min(args.steps, 10)):
        step()
    kt = ctx.kernel_times()
    ctx.kernel_profile(False)
    k_steps = min(args.steps, 10)
    mac_ms = kt["mac"][0] / k_steps
    got = ctx.decrypt_scores(km.s, ctx.export(binding.KIND_CT, score, Q * nb)).reshape(Q, -1)[:, :n_rows]
    errs = [float(np.abs(got[q] - rows_np.astype(np.float64) @ qs[q].astype(np.float64)).max()) for q in range(Q)]
    pt_bytes = nb * ctx.sizeof(binding.SIZE_PT_BLOCK)
    passes = (Q + 1) // 2 if ps.B <= 16 else Q  # two queries share a pass where their baby-step words fit the registers
    print(json.dumps({
        "metric": "encrypted candidate-query pairs scored/sec", "value": n_rows * Q / (ms * 1e-3), "unit": "pairs/s", "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "ms_per_query": ms / Q, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": wname + ", %d queries batched against the level" % Q, "rows": n_rows, "blocks": nb, "queries": Q},
        "mac": {"ms_per_batch": mac_ms, "ms_per_query": mac_ms / Q, "launches_per_batch": kt["mac"][1] / k_steps,
                "plaintext_passes": passes,
                "GB/s": (passes * pt_bytes + Q * (ctx.sizeof(binding.SIZE_BABY) + nb * ctx.sizeof(binding.SIZE_INNER))) / (mac_ms * 1e-3) / 1e9},
        "check": {"max_abs_score_error": max(errs), "tolerance": 2.0 ** ps.tol_log2, "ok": bool(max(errs) < 2.0 ** ps.tol_log2)},
    }))
    return 0 if max(errs) < 2.0 ** ps.tol_log2 else 1


def run_encrypted_db(args):
    """Encrypted database (Sec. 2, deployment setting): the level's candidate diagonals are ciphertexts, enrolled once
    (encode + encrypt, outside the timed region) and resident in HBM -- the paper's "warm" case.  A step = query
    preparation + ct x ct multiply-accumulate with one relinearisation per (blk, g) + rotate-and-sum.  One JSON line."""
    import torch
    from paper_2608_21131_b200 import binding, synth, workloads as wl

    torch.cuda.set_device(0)
    ps, rows_np, qR, wname = build_workload(args.config, args.rows, args.logn)
    n_rows = rows_np.shape[0]
    ctx = binding.Context(ps, device=0)
    if args.mac_f64 is not None:
        ctx.set_tuning(binding.TUNE_MAC_F64, args.mac_f64)
    km = synth.key_material(ps, wl.KEY_SEED)
    ctx.load_keys(ctx.keygen_from_samples(km.s, km.rots, km.evk_a, km.evk_e), km.rots)
    ka = synth.uniform_residues(wl.KEY_SEED, 50, list(ps.q) + [ps.p], ps.N, lead=(ps.L,))
    ke = synth.rounded_gaussian(wl.KEY_SEED, 51, (ps.L, ps.N))
    ctx.load_keys(ctx.keygen_relin_from_samples(km.s, ka, ke)[None], [0])
    ct_dev = ctx.import_(binding.KIND_CT, ctx.encrypt_query(km.s, qR, km.ct_a, km.ct_e), 1)
    nb = ctx.n_blocks(n_rows)
    ws = ctx.workspace(nb)
    pt = ctx.encode_candidates(torch.from_numpy(rows_np).to(ctx.device), ws)
    ptw, dbw = ctx.sizeof(binding.SIZE_PT_BLOCK) // 8, ctx.sizeof(binding.SIZE_CTDB_BLOCK) // 8
    ctdb = ctx.alloc(nb * dbw * 8)
    t_enrol = time.perf_counter()
    for blk in range(nb):
        a = synth.uniform_residues(wl.CORPUS_SEED + blk, 40, list(ps.q), ps.N, lead=(ps.R,))
        e = synth.rounded_gaussian(wl.CORPUS_SEED + blk, 41, (ps.R, ps.N))
        ctx.encrypt_block(km.s, pt[blk * ptw:(blk + 1) * ptw], a, e, ctdb[blk * dbw:(blk + 1) * dbw])
    t_enrol = time.perf_counter() - t_enrol
    del pt
    baby = ctx.alloc(ctx.sizeof(binding.SIZE_BABY))
    inner = ctx.alloc(nb * ctx.sizeof(binding.SIZE_INNER))
    score = ctx.alloc(nb * ctx.sizeof(binding.SIZE_CT))
    iw = ctx.sizeof(binding.SIZE_INNER) // 8

    if args.from_host:
        # the paper's warm case as it measures it: the enrolled ciphertexts are NOT resident; every query loads its
        # candidates' ciphertexts (here from page-locked host memory) block by block into two device slots while the
        # previous block is scored
        host_db = torch.empty(nb * dbw, dtype=torch.int64).pin_memory()
        host_db.copy_(ctdb)
        torch.cuda.synchronize()
        del ctdb
        torch.cuda.empty_cache()
        slots = [ctx.alloc(dbw * 8) for _ in range(2)]
        copy_stream = torch.cuda.Stream()
        main = torch.cuda.current_stream()
        ready = [torch.cuda.Event() for _ in range(2)]
        free = [torch.cuda.Event() for _ in range(2)]

        def step():
            ctx.query_prepare(ct_dev, ws, baby)
            for blk in range(nb):
                k = blk % 2
                with torch.cuda.stream(copy_stream):
                    if blk >= 2:
                        copy_stream.wait_event(free[k])
                    slots[k].copy_(host_db[blk * dbw:(blk + 1) * dbw], non_blocking=True)
                    ready[k].record(copy_stream)
                main.wait_event(ready[k])
                ctx.score_level_ctdb(baby, slots[k], 1, ws, inner[blk * iw:(blk + 1) * iw])
                free[k].record(main)
            ctx.rotate_sum(inner, nb, ws, score)
            copy_stream.wait_stream(main)   # the next step's first copies must not overtake this step's scoring
    else:
        def step():
            ctx.query_prepare(ct_dev, ws, baby)
            ctx.score_level_ctdb(baby, ctdb, nb, ws, inner)
            ctx.rotate_sum(inner, nb, ws, score)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    k_steps = min(args.steps, 10)
    ctx.kernel_profile(True)
    for _ in range(k_steps):
        step()
    kt = ctx.kernel_times()
    ctx.kernel_profile(False)
    mac_ms = kt["mac"][0] / k_steps
    got = ctx.decrypt_scores(km.s, ctx.export(binding.KIND_CT, score, nb)).reshape(-1)[:n_rows]
    err = float(np.abs(got - rows_np.astype(np.float64) @ qR.astype(np.float64)).max())
    db_bytes = nb * dbw * 8
    print(json.dumps({
        "metric": METRIC, "value": n_rows / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": wname + (", ENCRYPTED candidates loaded from page-locked host memory per query (ct x ct, warm load)"
                                        if args.from_host else ", ENCRYPTED candidates resident in HBM (ct x ct, warm)"),
                   "rows": n_rows, "blocks": nb, "h2d_bytes_per_step": (nb * dbw * 8 if args.from_host else 0),
                   "database_bytes": db_bytes, "enrolment_s_per_block_incl_host_randomness": t_enrol / nb},
        "mac_ct": {"ms_per_step": mac_ms, "GB/s": (db_bytes + ctx.sizeof(binding.SIZE_BABY) + nb * ps.G * 3 * ps.L * ps.N * 8) / (mac_ms * 1e-3) / 1e9},
        "kernels_ms_per_step": {k: v[0] / k_steps for k, v in kt.items() if v[1]},
        "check": {"max_abs_score_error": err, "tolerance": 2.0 ** ps.tol_log2, "ok": bool(err < 2.0 ** ps.tol_log2)},
    }))
    return 0 if err < 2.0 ** ps.tol_log2 else 1


def run_project(args):
    """Rank reduction under encryption (Sec. 3.1: Enc(q_R) = W^T Enc(q), matrix packed by windows): device time of one
    projection of a 512-dimensional encrypted query, for every baby-step count of the sweep and both evaluation orders of the
    giant steps (the paper's projection-latency figure: the optimum sits below sqrt(R) because a baby step costs two slot
    rotations here and a giant step one).  N = 2^16, 4 x 50-bit primes, masks and matrix at scale 2^50.  One JSON line."""
    import torch
    from paper_2608_21131_b200 import binding, synth, workloads as wl

    torch.cuda.set_device(0)
    D, R, L, logN = 512, args.project_rank, 4, 16
    q, p = synth.Q50, synth.P60
    rng = np.random.default_rng(wl.PROJ_SEED)
    W = np.linalg.qr(rng.standard_normal((D, R)))[0].astype(np.float32)
    qv = synth.normalise(synth.gaussian_vectors(wl.query_seed(0), synth.S_QUERY, np.arange(1), D))[0].astype(np.float32)
    want = W.T.astype(np.float64) @ qv.astype(np.float64)
    sweep = []
    for B in [int(x) for x in args.project_sweep.split(",")]:
        if R % B:
            continue
        G = R // B
        ps = synth.ParamSet("proj", logN, q, p, 40, R, B, -18)
        top, mid = binding.Context(ps), binding.Context(ps.with_(q=q[:3]))
        n = top.n
        rots_top = list(range(1, B)) + [n - R + b for b in range(1, B)]
        fold = [R << t for t in range((D // R).bit_length() - 1)]
        rots_mid = sorted(set(g * B for g in range(1, G)) | set(fold))
        rots = sorted(set(rots_top) | set(rots_mid))
        km = synth.key_material(ps, wl.KEY_SEED, rots=rots)
        evk = top.keygen_from_samples(km.s, km.rots, km.evk_a, km.evk_e)
        pick = lambda wanted: np.stack([evk[rots.index(r)] for r in wanted])
        if rots_top:
            top.load_keys(pick(rots_top), rots_top)
        mid.load_keys(binding.restrict_keys(pick(rots_mid), L, 3), rots_mid)
        del evk
        lo, hi = top.project_masks(50, top.workspace(1))
        wpt = mid.project_enrol(torch.from_numpy(W).to(mid.device), 50, mid.workspace(1))
        # the query: q tiled with period D = one "candidate-free" encryption of a D-dimensional vector
        qctx = binding.Context(ps.with_(R=D, B=1))
        ct_dev = top.import_(binding.KIND_CT, qctx.encrypt_query(km.s, qv, km.ct_a, km.ct_e), 1)
        del qctx
        wsp = top.alloc(top.lib.hann_project_bytes(top.h, mid.h))
        rec = {"B": B, "G": G, "slot_rotations": {"baby": 2 * (B - 1), "giant": G - 1, "fold": len(fold)}}
        for order in ("horner", "lazy"):
            mid.set_tuning(binding.TUNE_GIANT_LAZY, 1 if order == "lazy" else 0)
            for _ in range(3):
                out = top.project_query(mid, ct_dev, lo, hi, wpt, D, wsp)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                out = top.project_query(mid, ct_dev, lo, hi, wpt, D, wsp)
            e1.record()
            torch.cuda.synchronize()
            rec["ms_" + order] = e0.elapsed_time(e1) / args.steps
            # what came out: decrypt on the two-prime chain at the exact scale Delta 2^50/q_3 2^50/q_2
            lowctx = binding.Context(ps.with_(q=q[:2]))
            can = mid.export_limbs(out, 2, 2).reshape(1, 2, 2, top.N)
            slots = lowctx.decrypt_scores(km.s, can, log_scale_out=40)[0] * (2.0 ** 40 / (2.0 ** 40 * (2.0 ** 50 / q[3]) * (2.0 ** 50 / q[2])))
            rec["max_abs_error_" + order] = float(np.abs(slots - np.tile(want, n // R)).max())
            del lowctx
        sweep.append(rec)
        del top, mid, lo, hi, wpt, wsp, ct_dev
        torch.cuda.empty_cache()
    best = min(sweep, key=lambda r: min(r["ms_horner"], r["ms_lazy"]))
    ok = all(max(r["max_abs_error_horner"], r["max_abs_error_lazy"]) < 2.0 ** -20 for r in sweep)
    print(json.dumps({
        "metric": "encrypted projections/sec", "value": 1e3 / min(best["ms_horner"], best["ms_lazy"]), "unit": "projections/s", "n_gpus": 1,
        "steps": args.steps, "warmup": 3, "ms_per_step": min(best["ms_horner"], best["ms_lazy"]), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": "packed projection %d -> %d of one encrypted query, N=2^16, 4x50b primes, masks and matrix at 2^50" % (D, R),
                   "sqrt_R": R ** 0.5, "best_B": best["B"]},
        "sweep": sweep, "check": {"tolerance": 2.0 ** -20, "ok": ok},
    }))
    return 0 if ok else 1


def run_membership(args):
    """Membership (threshold) scan of the face task (Sec. 3.1 norm problem; Sec. 2: depth 11, ring 2^15, 45-bit scale): one
    encrypted query against the face-like level, the server returning per candidate a ciphertext slot whose sign says whether
    <x, q_R> >= tau |q_R|.  A step = the whole circuit (hann_membership_decide) with the candidates encoded and resident.
    Chain of 12 primes (58-bit first prime, 45/46-bit scaling primes), R = 128.  One JSON line; the decisions are checked
    against the direct comparison outside the polynomial's error band."""
    import torch
    from paper_2608_21131_b200 import binding, synth, workloads as wl

    torch.cuda.set_device(0)
    logN, R, B, deg, iters, tau, t_lo, t_hi, log_scale = 15, 128, 32, 7, 3, 0.45, 0.05, 1.0, 45
    n_rows = args.rows or 222_049
    _, lvl, qR, planted = wl.face_level(rows=n_rows, ps=synth.FULL15)
    qR = (0.7 * qR / np.linalg.norm(qR)).astype(np.float32)      # |q_R|^2 = 0.49, inside [t_lo, t_hi]
    lib = binding.load_library()
    lv = np.zeros(2, dtype=np.int32)
    lib.hann_membership_levels(deg, iters, lv[0:].ctypes.data, lv[1:].ctypes.data)
    L, score_level = int(lv[0]), int(lv[1])
    # the chain: largest primes below 2^58 / 2^45 / 2^46 / 2^60 that are 1 mod 2N, consumed from the end (see hann.h)
    def primes_below(bits, count):
        import sympy

        out, c = [], (1 << bits) - (2 << logN) + 1
        while len(out) < count:
            if sympy.isprime(c):
                out.append(c)
            c -= 2 << logN
        return out
    n_thr = 1 + 3 + 1
    p45, p46 = primes_below(log_scale, n_thr + iters), primes_below(log_scale + 1, iters)
    consumed = p45[:n_thr]
    for i in range(iters):
        consumed += [p45[n_thr + i], p46[i]]
    q = primes_below(58, 1) + consumed[::-1]
    p = primes_below(60, 1)[0]
    a_aff = 2.0 / (t_hi - t_lo)
    lam, kappa = float(np.sqrt(a_aff * q[-1] / 2.0 ** log_scale)), 0.5
    k = np.arange(deg + 1)
    nodes = np.cos(np.pi * (k + 0.5) / (deg + 1))
    vals = kappa * tau * np.sqrt(0.5 * (t_hi - t_lo) * nodes + 0.5 * (t_hi + t_lo))
    coef = np.array([2.0 / (deg + 1) * np.sum(vals * np.cos(np.pi * j * (k + 0.5) / (deg + 1))) for j in range(deg + 1)])
    coef[0] *= 0.5
    ps = synth.ParamSet("mem", logN, tuple(q), p, log_scale, R, B, -10)
    fold = [1 << t for t in range(R.bit_length() - 1)]
    rots = sorted(set(range(1, B + 1)) | set(fold))
    km = synth.key_material(ps, wl.KEY_SEED, rots=rots)
    topc = binding.Context(synth.ParamSet("a", logN, tuple(q), p, log_scale, 1, 1, -10))
    evk = topc.keygen_from_samples(km.s, km.rots, km.evk_a, km.evk_e)
    ka = synth.uniform_residues(wl.KEY_SEED, 50, list(q) + [p], ps.N, lead=(L,))
    ke = synth.rounded_gaussian(wl.KEY_SEED, 51, (L, ps.N))
    rlk = topc.keygen_relin_from_samples(km.s, ka, ke)
    arith = [binding.Context(synth.ParamSet("a%d" % l, logN, tuple(q[:l]), p, log_scale, 1, 1, -10)) for l in range(1, L)] + [topc]
    for l in range(2, L + 1):
        arith[l - 1].load_keys(binding.restrict_keys(rlk, L, l)[None], [0])
    pick = lambda wanted: np.stack([evk[rots.index(r)] for r in wanted])
    arith[L - 2].load_keys(binding.restrict_keys(pick(fold), L, L - 1), fold)
    scorer = binding.Context(synth.ParamSet("s", logN, tuple(q[:score_level]), p, log_scale, R, B, -10))
    srots = list(range(1, B + 1))
    scorer.load_keys(binding.restrict_keys(pick(srots), L, score_level), srots)
    del evk
    # the client encodes lam * q_R tiled with period R: a "dimension R" query of a context of that rank on the full chain
    qctx = binding.Context(synth.ParamSet("q", logN, tuple(q), p, log_scale, R, 1, -10))
    ct_dev = topc.import_(binding.KIND_CT, qctx.encrypt_query(km.s, (lam * qR.astype(np.float64)).astype(np.float32), km.ct_a, km.ct_e), 1)
    del qctx
    rows_scaled = (lvl.rows.astype(np.float64) * (kappa / lam)).astype(np.float32)
    nb = scorer.n_blocks(n_rows)
    pt = scorer.encode_candidates(torch.from_numpy(rows_scaled).to(scorer.device), scorer.workspace(nb))

    def step():
        return binding.membership_decide(arith, scorer, R, deg, iters, log_scale, tau, t_lo, t_hi, coef, ct_dev, pt, nb)

    l0 = sum(c.get_stats()["launches"] for c in arith + [scorer])
    out, out_scale = step()
    launches = sum(c.get_stats()["launches"] for c in arith + [scorer]) - l0
    for _ in range(max(args.warmup, 2)):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        out, out_scale = step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    dec = arith[0].decrypt_scores(km.s, arith[0].export(binding.KIND_CT, out, nb), log_scale_out=log_scale).reshape(-1)[:n_rows] * (2.0 ** log_scale / out_scale)
    q64 = (lam * qR.astype(np.float64)).astype(np.float32).astype(np.float64) / lam       # the query as the client encoded it
    direct = (rows_scaled.astype(np.float64) * (lam / kappa)) @ q64 - tau * np.linalg.norm(q64)
    clear = np.abs(direct) > 4e-3 * tau
    agree = bool(np.array_equal(np.sign(dec[clear]), np.sign(direct[clear])))
    print(json.dumps({
        "metric": "encrypted membership decisions/sec", "value": n_rows / (ms * 1e-3), "unit": "candidates/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 2), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64",
        "data": "synthetic",
        "config": {"workload": "membership (threshold) scan of the face-like level: %d rows, R=128, N=2^15, 12 primes (58b + 45/46b), depth 11" % n_rows,
                   "blocks": nb, "tau": tau, "chebyshev_degree": deg, "sign_iterations": iters, "candidates": "encoded and resident"},
        "gpu_launches": int(launches),
        "check": {"decisions_agree_outside_error_band": agree, "rows_outside_band": int(clear.sum()), "matches": int((dec > 0).sum()),
                  "planted_row_matches": bool(dec[planted] > 0), "ok": bool(agree and dec[planted] > 0)},
    }))
    return 0 if agree else 1


def oracle_setup(ps, qR, km):
    from oracle.oracle import Oracle

    o = Oracle(ps.logN, ps.q, ps.p, ps.log_scale, ps.R, ps.B)
    ct = o.encrypt_query(km.s, qR, km.ct_a, km.ct_e)
    evk = np.stack([o.evk_gen(km.s, r, km.evk_a[i], km.evk_e[i]) for i, r in enumerate(km.rots)])
    return o, ct, evk


def oracle_single_thread(ps, rows_np, qR, km, n_rows, o, ct, evk):
    """The oracle on ONE thread.  Its work is a sum of independent operations with no reuse between them (every rotation,
    every plaintext encoding, every plaintext x ciphertext product is computed from scratch), so the level's time is the
    time of one operation of each kind, measured on one thread, times the number of such operations: B-1 rotations for the
    query, and per block R encodings, R plaintext x ciphertext products and G-1 rotations."""
    import ctypes
    from oracle.oracle import Oracle

    omp = ctypes.CDLL("libgomp.so.1")
    threads = o.num_threads()
    omp.omp_set_num_threads(1)
    try:
        t0 = time.perf_counter()
        o.rotate(ct, 1, evk[0])
        t_rot = time.perf_counter() - t0
        one = Oracle(ps.logN, ps.q, ps.p, ps.log_scale, 1, 1)   # R = B = 1: one diagonal, one product
        col = np.ascontiguousarray(rows_np[: ps.n, :1])
        t0 = time.perf_counter()
        pt1 = one.encode_block(col)
        t_enc = time.perf_counter() - t0
        t0 = time.perf_counter()
        one.mac(pt1, ct[None])
        t_mac = time.perf_counter() - t0
    finally:
        omp.omp_set_num_threads(threads)
    nb = (n_rows + ps.n - 1) // ps.n
    total = (ps.B - 1) * t_rot + nb * (ps.R * (t_enc + t_mac) + (ps.G - 1) * t_rot)
    return {"value": n_rows / total, "unit": UNIT, "cores": 1,
            "sample": "one rotation (%.2f s), one plaintext encoding (%.3f s) and one plaintext x ciphertext product (%.3f s) timed "
                      "on one thread; level time = (B-1) rotations + blocks x (R encodings + R products + (G-1) rotations)"
                      % (t_rot, t_enc, t_mac)}


def oracle_block(o, ps, rows, baby, evk, giant):
    """one block through the oracle, the giant steps in the order the timed GPU path uses"""
    if giant == "lazy" and ps.G > 1 and len(evk) >= ps.B + ps.G - 2:
        inner = o.mac(o.encode_block(np.ascontiguousarray(np.pad(rows, ((0, 0), (0, ps.R - rows.shape[1]))))), baby)
        return o.rotate_sum_lazy(inner, np.stack([evk[ps.B - 1]] + [evk[ps.B + g - 2] for g in range(2, ps.G)]))
    return o.score_block(rows, baby, evk[ps.B - 1])[0]


def cpu_baseline(ps, rows_np, qR, km, n_rows, giant="horner"):
    """the oracle as it stands on the host cores: one query_prepare + one block, scaled to the level by block count; and the
    same level on a single thread"""
    o, ct, evk = oracle_setup(ps, qR, km)
    t0 = time.perf_counter()
    baby = o.baby_set(ct, evk)
    t_prep = time.perf_counter() - t0
    t0 = time.perf_counter()
    oracle_block(o, ps, rows_np[: ps.n], baby, evk, giant)
    t_blk = time.perf_counter() - t0
    nb = (n_rows + ps.n - 1) // ps.n
    single = oracle_single_thread(ps, rows_np, qR, km, n_rows, o, ct, evk) if ps.B > 1 else None
    return {"value": n_rows / (t_prep + nb * t_blk), "unit": UNIT, "cores": o.num_threads(), "kind": "oracle",
            "sample": "query_prepare once (%.1f s) + block 0 of %d (%d rows, %.1f s) timed; level time = prepare + blocks x "
                      "block time (per-block work is constant)" % (t_prep, nb, min(ps.n, n_rows), t_blk),
            "single_thread": single}


def run_hierarchy(args):
    """Configs 2 and 3: the client-steered hierarchy (coarse -> fine -> rerank), one query after the other.  The timed
    quantity is the server-side scoring of each level (rows resident in HBM, CUDA events); the client steps between the
    levels (decrypt, rank, fetch the next candidates) are outside.  The baby rotations are prepared once per query and
    reused by its three levels.  Prints one JSON line with the latency distribution per level."""
    import torch
    from paper_2608_21131_b200 import binding, synth, workloads as wl

    torch.cuda.set_device(0)
    cfg = wl.datacomp_like() if args.config == 2 else wl.deep1b_like()
    ps = cfg.ps
    ctx = binding.Context(ps, device=0)
    km = bench_keys(ctx, ps, args)
    coarse = wl.coarse_level(cfg)
    max_rows = max(len(coarse.ids), cfg.nprobe * cfg.h.fan, cfg.leaf_beam * cfg.h.leaf)
    nb_max = ctx.n_blocks(max_rows)
    ws = ctx.workspace(nb_max)
    baby = ctx.alloc(ctx.sizeof(binding.SIZE_BABY))
    pt = ctx.alloc(nb_max * ctx.sizeof(binding.SIZE_PT_BLOCK))
    inner = ctx.alloc(nb_max * ctx.sizeof(binding.SIZE_INNER))
    score = ctx.alloc(nb_max * ctx.sizeof(binding.SIZE_CT))
    coarse_dev = torch.from_numpy(coarse.rows).to(ctx.device)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]

    def timed(fn):
        ev[0].record()
        fn()
        ev[1].record()
        torch.cuda.synchronize()
        return ev[0].elapsed_time(ev[1])

    def level(rows_dev, n_rows):
        nb = ctx.n_blocks(n_rows)
        ms = timed(lambda: (ctx.encode_candidates(rows_dev, ws, pt), ctx.score_level(baby, pt, nb, ws, inner),
                            ctx.rotate_sum(inner, nb, ws, score)))
        sc = ctx.decrypt_scores(km.s, ctx.export(binding.KIND_CT, score, nb)).reshape(-1)[:n_rows]
        return ms, sc

    times = {"query_prepare": [], "coarse": [], "fine": [], "rerank": []}
    rows_scored, hits, worst = 0, 0, 0.0
    n_q = args.steps + args.warmup
    for qi in range(n_q):
        qR, planted = wl.hier_query(cfg, qi)
        ct_dev = ctx.import_(binding.KIND_CT, ctx.encrypt_query(km.s, qR, km.ct_a, km.ct_e), 1)
        t_prep = timed(lambda: ctx.query_prepare(ct_dev, ws, baby))
        t_c, sc = level(coarse_dev, len(coarse.ids))
        worst = max(worst, float(np.abs(sc - coarse.rows.astype(np.float64) @ qR.astype(np.float64)).max()))
        fine = wl.fine_level(cfg, np.sort(wl.topk_ids(sc, coarse.ids, cfg.nprobe)))
        t_f, sf = level(torch.from_numpy(fine.rows).to(ctx.device), len(fine.ids))
        rer = wl.rerank_level(cfg, np.sort(wl.topk_ids(sf, fine.ids, cfg.leaf_beam)))
        t_r, sr = level(torch.from_numpy(rer.rows).to(ctx.device), len(rer.ids))
        worst = max(worst, float(np.abs(sr - rer.rows.astype(np.float64) @ qR.astype(np.float64)).max()))
        if qi >= args.warmup:
            for k, v in zip(("query_prepare", "coarse", "fine", "rerank"), (t_prep, t_c, t_f, t_r)):
                times[k].append(v)
            rows_scored += len(coarse.ids) + len(fine.ids) + len(rer.ids)
            hits += int(planted in wl.topk_ids(sr, rer.ids, 10))
    total_ms = sum(sum(v) for v in times.values())
    pct = lambda v, p: float(np.percentile(v, p))
    print(json.dumps({
        "metric": METRIC, "value": rows_scored / (total_ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": cfg.name + " hierarchy, one query at a time", "giant_steps": args.giant, "levels": {"coarse": len(coarse.ids), "fine": len(fine.ids),
                                                                                        "rerank": len(rer.ids)},
                   "logN": ps.logN, "L": ps.L, "R": ps.R, "B": ps.B},
        "ms_per_query_level": {k: {"p50": pct(v, 50), "p95": pct(v, 95)} for k, v in times.items()},
        "ms_per_query": {"p50": pct(np.sum(list(times.values()), axis=0), 50), "p95": pct(np.sum(list(times.values()), axis=0), 95)},
        "planted_neighbour_in_top10": hits / args.steps,
        "check": {"max_abs_score_error": worst, "tolerance": 2.0 ** ps.tol_log2, "ok": bool(worst < 2.0 ** ps.tol_log2)},
    }))
    return 0


def run_reference(args):
    """reference arm: the CPU oracle, unmodified, on the host cores; a step is query_prepare + one block"""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return 0
    from paper_2608_21131_b200 import synth, workloads as wl

    ps, rows_np, qR, wname = build_workload(args.config, args.rows, args.logn)
    n_rows = rows_np.shape[0]
    km = synth.key_material(ps, wl.KEY_SEED, rots=list(range(1, ps.B + 1)) + [g * ps.B for g in range(2, ps.G)])
    o, ct, evk = oracle_setup(ps, qR, km)
    sample_rows = min(ps.n, n_rows)

    def step():
        baby = o.baby_set(ct, evk)
        oracle_block(o, ps, rows_np[:sample_rows], baby, evk, args.giant)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    value = sample_rows / dt
    sample = "each step = query_prepare + encode/MAC/rotate-sum of block 0 (%d of %d rows)" % (sample_rows, n_rows)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u64", "data": "synthetic", "config": {"workload": wname, "rows": n_rows, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": o.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))
    return 0


def relaunch_under_torchrun(n, argv=None):
    """run this script again as n ranks on this node and return the launcher's exit code"""
    import socket

    with socket.socket() as sk:  # a free port for the rendezvous
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n), "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + list(sys.argv[1:] if argv is None else argv)
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1, help="0 toy, 1 face-like level (default), 2 DataComp-like and 3 Deep1B-like "
                    "hierarchies (latency per level), 4 scaling sweep point (--rows = wanted rows, --logn 15|16)")
    ap.add_argument("--logn", type=int, default=16, help="ring of the sweep configuration")
    ap.add_argument("--min-timed-s", type=float, default=2.0, help="the K-step block is repeated until the timed region lasted this long")
    ap.add_argument("--membership", action="store_true", help="membership (threshold) scan of the face-like level at depth 11, N = 2^15")
    ap.add_argument("--project", action="store_true", help="packed projection 512 -> R of one encrypted query: baby-step sweep")
    ap.add_argument("--project-rank", type=int, default=128, help="R of --project (128 or 256)")
    ap.add_argument("--project-sweep", default="1,2,4,8,16,32", help="baby-step counts of --project")
    ap.add_argument("--giant", default="lazy", choices=["horner", "lazy"],
                    help="evaluation order of the giant steps of the rotate-and-sum (the library's own default is Horner)")
    ap.add_argument("--groups", type=int, default=None, help="tuning: block groups a level is cut into (scored beside the encoding of the next group); default: plain order")
    ap.add_argument("--pair-b32", action="store_true", help="tuning (--queries): two queries per pass over the plaintexts at B = 32 too")
    ap.add_argument("--mac-f64", type=int, default=None, help="tuning: 1 (default): the multiply-accumulate sums on the FP64 pipe, 0: on the integer multiplier")
    ap.add_argument("--lazy-lanes", type=int, default=None, help="tuning: block ranges the lazy rotate-and-sum runs side by side (1..4)")
    ap.add_argument("--baby", type=int, default=None, help="baby-step count B (default: the configuration's; must divide R)")
    ap.add_argument("--rows", type=int, default=None, help="override the row count (debugging, ncu captures)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--encode-group", type=int, default=None, help="tuning: plaintexts per encode launch group")
    ap.add_argument("--from-host", action="store_true", help="with --encrypted-db: load the ciphertexts from pinned host memory every query")
    ap.add_argument("--encrypted-db", action="store_true", help="encrypted candidates resident in HBM (ct x ct, warm case)")
    ap.add_argument("--queries", type=int, default=1, help="queries batched against the level (cross-query batching mode when > 1)")
    ap.add_argument("--staged", action="store_true", help="with --lean: run the steps as the per-kernel timing pass does")
    ap.add_argument("--lean", action="store_true", help="only run warm-up + steps (for ncu); prints no JSON line")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as `python bench.py --gpus N`: become N ranks, one per GPU, under torch's launcher (independent replicas;
        # rank 0 prints the line)
        return relaunch_under_torchrun(args.gpus)
    if args.impl == "reference":
        args.steps = 2 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        return run_reference(args)
    if args.project:
        args.steps = 10 if args.steps is None else args.steps
        return run_project(args)
    if args.membership:
        args.steps = 5 if args.steps is None else args.steps
        args.warmup = 2 if args.warmup is None else args.warmup
        return run_membership(args)
    if args.config in (2, 3):
        args.steps = (16 if args.config == 2 else 64) if args.steps is None else args.steps
        args.warmup = 2 if args.warmup is None else args.warmup
        return run_hierarchy(args)
    if args.encrypted_db:
        args.steps = 20 if args.steps is None else args.steps
        args.warmup = 3 if args.warmup is None else args.warmup
        return run_encrypted_db(args)
    if args.queries > 1:
        args.steps = 20 if args.steps is None else args.steps
        args.warmup = 3 if args.warmup is None else args.warmup
        return run_batch(args)
    args.steps = 200 if args.steps is None else args.steps
    args.warmup = 20 if args.warmup is None else args.warmup
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
