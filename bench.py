#!/usr/bin/env python
"""Throughput of the sign+vote hot path on seeded synthetic replica sets.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl reference]

One step = one pass of the whole hot path over one replica set: chunk
signatures for every replica, strict-majority vote, compaction and (config 4)
the certify roll-up.  The metric is GB/s of replica data scanned.  Prints ONE
JSON line on rank 0.

  value         inputs resident in HBM, CUDA-event time over exactly K steps
  e2e           the same metric through scout_certify_host: replicas in pinned
                HOST memory, host->device copies inside the timed region
  roofline      the scan kernel alone (in-stream CUDA events inside the library)
                against the measured HBM copy bandwidth
  cpu_baseline  the CPU oracle, as it stands, on a bounded sample of the workload

With N > 1 every rank scans its own replica set (no data-path collective):
weak scaling, value = bytes of all ranks / max-over-ranks time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "replica GB/s scanned (sign+vote)"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126 << 20
BENCH_CASE = {2: "mantissa"}   # config 2 is timed on its one-flip case, so every config carries a fault
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes (read + write) per algorithmic byte of the scan kernel, from the ncu
# captures summarised under profiles/: 1.8006 GB read + 0.0256 GB written for
# 1.8000 GB scanned (fp32), 4.5997 + 0.021 for 4.5993 GB (bf16, ratio 1.0046).  Traffic
# grows in proportion to the bytes scanned, so a full-size launch is scaled by this.
# To be measured again whenever the scan kernel changes.
SCAN_TRAFFIC_RATIO = 1.0146
SCAN_TRAFFIC_SOURCE = ("ncu capture of the scan kernel on 1.8 GB at commit a9c0242, scaled to the launch "
                       "(summary under profiles/)")


# SM cycles per 512-byte row and scheduler of the scan's row routine with its data already on the
# SM (`python -m paper_2608_11034_b200.microbench`, its output is summarised under profiles/): the
# compute bound of a uniform-dtype workload at SM clock f is 512 B * 4 * SMs * f / cycles.
ROW_COST_CYCLES = {"bf16": 74.7, "f16": 75.6, "f32": 45.1, "i64": 41.2, "u8": 28.1}
N_SMS = 148


def compute_bound(w, clocks, value):
    """The scan rate the row routine allows at the SM clock sampled during the timed region."""
    dtypes = {s.dtype for s in w.specs}
    if len(dtypes) != 1 or next(iter(dtypes)) not in ROW_COST_CYCLES or not clocks or not clocks.get("sm_mhz"):
        return None
    cyc = ROW_COST_CYCLES[next(iter(dtypes))]
    bound = 512 * 4 * N_SMS * clocks["sm_mhz"] * 1e6 / cyc / 1e9
    return {"bound": "alu", "cycles_per_row_per_scheduler": cyc, "sm_mhz_sampled": clocks["sm_mhz"],
            "bound_gbs": bound, "frac": value / bound,
            "source": "row_cost microbenchmark (python -m paper_2608_11034_b200.microbench)"}


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--scale", type=float, default=1.0, help="shrink the workload (debugging only)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--variant", type=int, default=None)
    ap.add_argument("--tile-bytes", type=int, default=None)
    ap.add_argument("--work-streams", type=int, default=None, help="plan key 'work_streams'")
    ap.add_argument("--fused", type=int, default=None, help="plan key 'fused': 1, 0 or -1 (default)")
    ap.add_argument("--custom", default=None, metavar="DTYPE,TOTAL_MIB,R,CHUNK_KIB",
                    help="instead of a numbered config: one tensor per replica of that dtype (f32, bf16, ...), "
                         "TOTAL_MIB over all R replicas, that chunk size, one flipped bit in the last replica "
                         "(shape studies of the small-plan forms; not a headline workload)")
    ap.add_argument("--also", default=None,
                    help="comma-separated configs measured after the headline one and reported under "
                         "'also' (default: 3,5 for the default full-size run at N=1; '' for none)")
    return ap.parse_args()


# ------------------------------------------------------------------ clocks

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.path = tempfile.mktemp(suffix=".csv")
        self.proc = None
        try:
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        try:
            os.unlink(self.path)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "power_w_max": max(pw),
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------ CPU oracle legs

def oracle_sample(w, views, chunk_bytes, budget_bytes):
    """Whole leading chunks of replica 0's tensors, up to budget_bytes, as host
    arrays plus the matching tensor table (same dtype and shape tag, so the
    records are those of the full workload's chunks)."""
    from oracle import scout_oracle as orc
    from paper_2608_11034_b200 import inputs
    code = {"u8": 0, "f32": 1, "bf16": 2, "i64": 3, "f16": 4, "f64": 5, "i32": 6}
    per_tensor = max(chunk_bytes, budget_bytes // len(w.specs) // chunk_bytes * chunk_bytes)
    rows, arrays, picked, total = [], [], [], 0
    for t, s in enumerate(w.specs):
        if total >= budget_bytes:
            break
        n = min(s.nbytes, per_tensor)
        if n < s.nbytes:
            n = n // chunk_bytes * chunk_bytes
        rows.append((n, code[s.dtype], orc.shape_tag(list(s.shape))))
        arrays.append(inputs.to_numpy_bytes(views[0][t].view(-1).view(__import__("torch").uint8)[:n]))
        picked.append(t)
        total += n
    return orc.make_tensor_table(rows), arrays, picked, total


def time_oracle(tt, arrays, chunk_bytes, nthreads):
    import numpy as np
    from oracle import scout_oracle as orc
    n_chunks = len(orc.chunk_table(tt, chunk_bytes))
    sigs = np.zeros((n_chunks, 1), dtype=orc.SIG_DTYPE)
    t0 = time.perf_counter()
    orc.sign_replica(tt, arrays, chunk_bytes, sigs, 0, nthreads)
    orc.vote(np.repeat(sigs, 2, axis=1))      # the vote is part of the path (negligible)
    return time.perf_counter() - t0, sigs


def cpu_baseline(w, views, seconds):
    """Oracle GB/s on this host, all cores, on a bounded sample."""
    cores = os.cpu_count() or 1
    tt, arrays, picked, total = oracle_sample(w, views, w.chunk_bytes, 8 << 20)
    dt, _ = time_oracle(tt, arrays, w.chunk_bytes, 1)
    rate1 = total / dt
    budget = int(min(max(rate1 * cores * seconds * 0.6, 32 << 20), 16 << 30))
    tt, arrays, picked, total = oracle_sample(w, views, w.chunk_bytes, budget)
    dt, sigs = time_oracle(tt, arrays, w.chunk_bytes, cores)
    return {"value": total / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "single_thread_value": rate1 / 1e9,
            "sample": f"leading whole chunks of replica 0: {total} bytes of {len(picked)} tensors, "
                      f"{cores} threads over chunks, {dt:.1f} s"}, (tt, picked, sigs)


def run_reference(args):
    """The CPU oracle as the reference arm: same config, metric and unit; every
    step signs and votes a bounded sample of the workload on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from paper_2608_11034_b200 import inputs
    from oracle import scout_oracle as orc
    orc.build()
    w = inputs.workload(args.config, BENCH_CASE.get(args.config, "default"), args.scale)
    cores = os.cpu_count() or 1
    # generate only what is sampled: shrink each tensor to its leading chunks.  The sample
    # holds at least four chunks per host thread, so that every thread has work (a smaller
    # sample under-reports the oracle), and at most 2 GiB per step.
    budget = min(max(192 << 20, 4 * cores * w.chunk_bytes), 2 << 30)
    per_tensor = max(w.chunk_bytes, budget // len(w.specs) // w.chunk_bytes * w.chunk_bytes)
    specs, total = [], 0
    for s in w.specs:
        if total >= budget:
            break
        es = inputs.DTYPE_BYTES[s.dtype]
        n = min(s.nbytes, per_tensor)
        specs.append(inputs.TensorSpec(s.name, (n // es,), s.dtype, s.dist, s.std))
        total += n
    sw = inputs.Workload(w.name, w.config, "sample", w.R, w.chunk_bytes, specs, w.seed)
    _, views0 = inputs.generate_replica0(sw, "cpu")
    views = [views0]
    tt, arrays, picked, total = oracle_sample(sw, views, sw.chunk_bytes, budget)
    times = []
    for i in range(args.warmup + args.steps):
        dt, _ = time_oracle(tt, arrays, sw.chunk_bytes, cores)
        if i >= args.warmup:
            times.append(dt)
    t = sum(times)
    value = total * len(times) / t / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64+f64",
        "data": "synthetic",
        "config": dict(config_block(w, sum((x.nbytes + w.chunk_bytes - 1) // w.chunk_bytes for x in w.specs)),
                       parallelism="single GPU" if args.gpus == 1 else f"{args.gpus} independent replica sets"),
        "sample_bytes_per_step": total,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"one replica's leading chunks, {total} bytes per step, {cores} threads; "
                                   f"the CUDA arm's cpu_baseline leg times the same oracle once over a "
                                   f"larger sample of the resident data"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ the CUDA arm

def expected_pairs(w, plan_handle, binding, inputs):
    """(chunk, replica) pairs the fault patches must produce, from chunk geometry."""
    import bisect
    C = binding.scout_plan_num_chunks(plan_handle)
    # chunk ids of a tensor are consecutive; find each tensor's first chunk
    first, c = {}, 0
    for t, s in enumerate(w.specs):
        first[t] = c
        c += (s.nbytes + w.chunk_bytes - 1) // w.chunk_bytes
    assert c == C
    pairs = set()
    for p in w.patches:
        es = inputs.DTYPE_BYTES[w.specs[p.tensor].dtype]
        pairs.add((first[p.tensor] + (p.element * es) // w.chunk_bytes, p.replica))
    return sorted(pairs)


def config_block(w, C):
    """Names the workload; the same keys in both arms (no launch settings here)."""
    return {"workload": w.name, "R": w.R, "tensors": len(w.specs), "chunks": C,
            "chunk_bytes": w.chunk_bytes, "bytes_per_step_per_gpu": w.R * w.bytes_per_replica}


def run_config(cfg, args, rank, world, local, headline):
    """One config on this rank's GPU: warm-up, K timed steps (CUDA events on the current
    stream, max over ranks), the scan kernel's own time for every one of those steps,
    the read-only probe, and the check of the last step's answer.  -> dict."""
    import torch
    from paper_2608_11034_b200 import binding, dist_util, inputs

    if args.custom and headline:
        dtype, total_mib, R, chunk_kib = args.custom.split(",")
        R = int(R)
        numel = int(float(total_mib) * (1 << 20)) // R // inputs.DTYPE_BYTES[dtype]
        w = inputs.Workload(f"custom_{dtype}_{total_mib}MiB_R{R}_chunk{chunk_kib}KiB", 0, "custom", R,
                            int(chunk_kib) << 10,
                            [inputs.TensorSpec("x", (numel,), dtype,
                                               {"u8": "bytes", "i64": "randint40", "i32": "randfull"}.get(dtype, "normal"),
                                               0.02)], 7)
        w.patches = [inputs.Patch(R - 1, 0, numel // 2, "xor", 4)]
    else:
        w = inputs.workload(cfg, BENCH_CASE.get(cfg, "default"), args.scale)
    w.seed = dist_util.rank_seed(w.seed, rank)   # every rank scans its own replica set
    flats, views = inputs.generate(w, "cuda")
    total_bytes = w.R * w.bytes_per_replica
    small = total_bytes < (1 << 30)          # working set may sit in L2: flush between steps
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda") if small else None

    plan = binding.Plan(w.R, binding.make_tensor_table(w.specs), w.chunk_bytes)
    if args.tile_bytes:
        binding.scout_plan_set(plan.handle, "tile_bytes", args.tile_bytes)
    if args.variant is not None:
        binding.scout_plan_set(plan.handle, "variant", args.variant)
    if args.fused is not None:
        binding.scout_plan_set(plan.handle, "fused", args.fused)
    if args.work_streams is not None:
        binding.scout_plan_set(plan.handle, "work_streams", args.work_streams)
    plan.bind(views)
    use_certify = cfg == 4 and not args.custom

    def step():
        if use_certify:
            return plan.certify()
        plan.sign_and_vote()
        return None

    for _ in range(max(args.warmup, 0)):
        step()
    torch.cuda.synchronize()
    def timed_steps():
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(args.steps)]
        dist_util.barrier()
        torch.cuda.synchronize()
        out = None
        for i in range(args.steps):
            if flush is not None:
                flush.fill_(i & 255)
            ev[i][0].record()
            out = step()
            ev[i][1].record()
        torch.cuda.synchronize()
        dist_util.barrier()
        return [a.elapsed_time(b) for a, b in ev], out

    sampler = ClockSampler(local) if rank == 0 else None
    untimed_ms = None
    if small:
        # a step of a small plan takes tens of microseconds and the two event records the
        # library adds around its scan kernel cost about five: the step time is taken without
        # them, the scan kernel's own time in a second pass with them
        untimed_ms, _ = timed_steps()
    binding.scout_plan_set(plan.handle, "timing", 1)      # from here on every scan launch is timed
    step_ms, last = timed_steps()
    clocks = sampler.stop() if sampler else None
    n_scan = binding.scout_plan_get(plan.handle, "timed_sign_launches")
    scan_ns = binding.scout_plan_get(plan.handle, "timed_sign_ns")
    binding.scout_plan_set(plan.handle, "timing", 0)
    # the ring holds the last 256 launches: with more steps than that, compare like with like
    steps_cmp = step_ms[-n_scan:]
    if n_scan != min(args.steps, 256) or scan_ns * 1e-6 > sum(steps_cmp) * 1.0005:
        raise SystemExit(f"inconsistent timing: {n_scan} scan launches took {scan_ns * 1e-6:.3f} ms inside "
                         f"steps that took {sum(steps_cmp):.3f} ms")
    ms = dist_util.max_over_ranks(sum(untimed_ms if small else step_ms), dist_util.reduce_device())

    # the last timed step must have produced the right answer
    want = expected_pairs(w, plan.handle, binding, inputs)
    if use_certify:
        got, verdict = last["outliers"], last["report"]["verdict"]
    else:
        got, verdict = plan.fetch()["outliers"], None
    if got != want:
        raise SystemExit(f"{w.name}: wrong result: outliers {got[:8]} expected {want[:8]}")

    peak, peak_kind = measured_peak()
    scan_s = scan_ns * 1e-9 / n_scan
    achieved = total_bytes / scan_s / 1e9
    roofline = {
        "bound": "hbm", "kernel": "sign_tiles", "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak, "peak_kind": peak_kind,
        "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
        "algorithmic_bytes_per_launch": total_bytes,
        "avg_launch_ms": scan_s * 1e3, "launches_timed": n_scan,
        "scan_share_of_step_time": scan_ns * 1e-6 / sum(steps_cmp),
        "traffic": (SCAN_TRAFFIC_RATIO * total_bytes) if SCAN_TRAFFIC_RATIO else None,
        "traffic_source": SCAN_TRAFFIC_SOURCE,
    }

    # read-only probe on the same plan and buffers: what the memory system delivers to
    # this tiling with loads + XOR only (outside the timed region; records are scratch)
    default_variant = binding.scout_plan_get(plan.handle, "variant")
    binding.scout_plan_set(plan.handle, "variant", 3)
    binding.scout_plan_set(plan.handle, "timing", 1)
    probe_ns = []
    for i in range(6):
        if flush is not None:
            flush.fill_(i)
        plan.sign()
        torch.cuda.synchronize()
        probe_ns.append(binding.scout_plan_get(plan.handle, "last_sign_ns"))
    binding.scout_plan_set(plan.handle, "variant", default_variant)
    binding.scout_plan_set(plan.handle, "timing", 0)
    probe = total_bytes / (sorted(probe_ns[1:])[len(probe_ns[1:]) // 2] * 1e-9) / 1e9
    roofline["read_probe_gbs"] = probe
    roofline["frac_of_read_probe"] = achieved / probe

    one_launch = None
    if small and w.R >= 2:
        # the whole path as ONE kernel: scout_certify_launch enqueues it, scout_certify_collect
        # (outside the event pair) waits for the report the kernel wrote to pinned host memory
        def timed(fn_launch, fn_after, flush_between):
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in range(args.steps)]
            for _ in range(3):
                fn_launch(); fn_after()
            torch.cuda.synchronize()
            for i, (a0, a1) in enumerate(evs):
                if flush_between:
                    flush.fill_(i & 255)
                a0.record(); fn_launch(); a1.record(); fn_after()
            torch.cuda.synchronize()
            ts = sorted(a0.elapsed_time(a1) for a0, a1 in evs)
            medians.append(ts[len(ts) // 2])
            return sum(ts) / args.steps
        medians = []
        one_launch = {"call": "scout_certify_launch (+ scout_certify_collect outside the timed pair)"}
        # what an event pair costs on this machine with nothing, and with a trivial kernel, between
        scratch = torch.zeros(32, device="cuda")
        one_launch["event_pair_floor_ms"] = {"nothing": timed(lambda: None, lambda: None, False),
                                             "torch_fill_of_128_bytes": timed(lambda: scratch.fill_(1.0),
                                                                              lambda: None, False)}
        one_launch["default_form"] = binding.scout_plan_get(plan.handle, "certify_form")
        for name, fused in (("one_kernel_clusters", 2), ("one_kernel", 1), ("kernel_per_stage", 0)):
            try:
                binding.scout_plan_set(plan.handle, "fused", fused)
            except binding.ScoutError:       # the cluster form does not fit this plan
                continue
            cold = timed(plan.certify_launch, plan.certify_collect, True)
            warm1 = timed(plan.certify_launch, plan.certify_collect, False)
            t0 = time.perf_counter()
            for _ in range(args.steps):
                rep = plan.certify()
            wall = (time.perf_counter() - t0) / args.steps
            assert rep["outliers"] == want
            one_launch[name] = {"kernels_per_step": binding.scout_plan_get(plan.handle, "certify_kernels"),
                                "ms_per_step_l2_cold": cold, "ms_per_step_l2_warm": warm1,
                                "median_ms_l2_cold": medians[-2], "median_ms_l2_warm": medians[-1],
                                "value_l2_cold": total_bytes / (cold * 1e-3) / 1e9,
                                "scout_certify_wall_ms_l2_warm": wall * 1e3}
        binding.scout_plan_set(plan.handle, "fused", -1)

    rotating = None
    if small and w.R >= 2:
        # L2-cold without a flush: enough independent copies of the replica set (one plan
        # each) that a set has left L2 before its turn comes again; steps run back to back
        # under ONE event pair.  The written flush above leaves up to an L2 of dirty lines
        # whose write-back competes with the scan's reads; here the evicted lines are clean.
        n_sets = max(3, -(-2 * L2_BYTES // total_bytes) + 1)
        sets = [[f.clone() for f in flats] for _ in range(n_sets - 1)]
        plans = [plan]
        for s in sets:
            q = binding.Plan(w.R, binding.make_tensor_table(w.specs), w.chunk_bytes)
            if args.tile_bytes:
                binding.scout_plan_set(q.handle, "tile_bytes", args.tile_bytes)
            q.bind([inputs.tensor_views(f, w.specs) for f in s])
            plans.append(q)

        def back_to_back(launch, after):
            for q in plans:
                launch(q); after(q)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(args.steps):
                q = plans[i % n_sets]
                launch(q); after(q)
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / args.steps

        rotating = {"sets": n_sets, "bytes_resident": n_sets * total_bytes,
                    "timing": "one event pair around all steps, no flush, no host wait between steps"}
        ms_r = back_to_back(lambda q: q.sign_and_vote(), lambda q: None)
        rotating["sign_vote"] = {"ms_per_step": ms_r, "value": total_bytes / (ms_r * 1e-3) / 1e9}
        for q in plans:
            if q.fetch()["outliers"] != want:
                raise SystemExit(f"{w.name}: wrong result on a rotating copy")
        for name, fused in (("certify_one_kernel_clusters", 2), ("certify_one_kernel", 1),
                            ("certify_kernel_per_stage", 0)):
            try:
                for q in plans:
                    binding.scout_plan_set(q.handle, "fused", fused)
            except binding.ScoutError:
                continue
            ms_r = back_to_back(lambda q: q.certify_launch(), lambda q: q.certify_collect())
            rotating[name + "_host_wait_each_step"] = {"ms_per_step": ms_r,
                                                       "value": total_bytes / (ms_r * 1e-3) / 1e9}
        for q in plans:
            binding.scout_plan_set(q.handle, "fused", -1)
        for q in plans[1:]:
            q.close()
        del sets, plans

    warm = None
    if small:   # the same steps with the replicas left in L2 (no flush between steps)
        evw = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(args.steps)]
        for _ in range(3):
            step()
        torch.cuda.synchronize()
        for a0, a1 in evw:
            a0.record(); step(); a1.record()
        torch.cuda.synchronize()
        msw = sum(a0.elapsed_time(a1) for a0, a1 in evw)
        warm = {"value": total_bytes * args.steps / (msw * 1e-3) / 1e9, "ms_per_step": msw / args.steps}

    value = dist_util.aggregate_gbs(total_bytes, world, args.steps, ms)
    out = {
        "value": value, "ms_per_step": ms / args.steps,
        "config": config_block(w, plan.C),
        "launch": {"call": "scout_certify" if use_certify else "scout_sign_chunks+scout_consensus_vote",
                   "kernels_per_step": binding.scout_plan_get(plan.handle, "certify_kernels") if use_certify
                   else binding.scout_plan_get(plan.handle, "sign_kernels") + 1,
                   "tile_bytes": binding.scout_plan_get(plan.handle, "tile_bytes"),
                   "variant": binding.scout_plan_get(plan.handle, "variant"),
                   "l2": "512 MiB written between steps" if small else "inputs far larger than L2, no flush",
                   "timed_region_s": ms * 1e-3,
                   "ms_per_step_with_scan_kernel_events": sum(step_ms) / args.steps,
                   "regime": "burst clocks (timed region under 1 s)" if ms < 1000 else "sustained"},
        "frac_of_nominal_8TBs": value / world / NOMINAL_HBM_GBS,
        "frac_of_measured_copy": value / world / peak,
        "verified": True, "verdict": verdict, "clocks": clocks, "roofline": roofline, "l2_warm": warm,
        "l2_cold_rotating": rotating, "one_launch": one_launch, "compute_bound": compute_bound(w, clocks, value) if world == 1 else None,
    }

    # ---- end to end: replicas in pinned host memory, copies inside the timed region
    if headline:
        if not args.no_e2e and rank == 0 and world == 1:
            try:
                bad = sorted({p.replica for p in w.patches})
                base = torch.empty(flats[0].numel(), dtype=torch.uint8, pin_memory=True)
                clean = next(r for r in range(w.R) if r not in bad)
                base.copy_(flats[clean])
                host = {r: base for r in range(w.R) if r not in bad}
                for r in bad:
                    h = torch.empty(flats[0].numel(), dtype=torch.uint8, pin_memory=True)
                    h.copy_(flats[r])
                    host[r] = h
                hviews = [inputs.tensor_views(host[r], w.specs) for r in range(w.R)]
                hptrs = [v.data_ptr() for rep in hviews for v in rep]
                binding.scout_certify_host(plan.handle, hptrs)          # warm-up (allocates staging)
                t0 = time.perf_counter()
                for _ in range(args.e2e_steps):
                    rep = binding.scout_certify_host(plan.handle, hptrs)
                dt = time.perf_counter() - t0
                assert rep["outliers"] == want
                out["e2e"] = {"value": total_bytes * args.e2e_steps / dt / 1e9, "unit": UNIT,
                              "h2d_bytes_per_step": total_bytes,
                              "d2h_bytes_per_step": 576 + 16 * len(want),
                              "steps": args.e2e_steps, "call": "scout_certify_host",
                              "host_memory": f"pinned; {len(bad) + 1} distinct replica images "
                                             f"(clean replicas share one host image)"}
                del base, host, hviews
            except Exception as e:                                       # noqa: BLE001
                out["e2e"] = {"value": None, "unit": UNIT, "error": repr(e)[:200]}
        else:
            out["e2e"] = {"value": None, "unit": UNIT, "note": "measured on rank 0 at N=1 only"}

    # ---- CPU oracle on a bounded sample, with a parity spot check against the CUDA records
    if not args.no_cpu_baseline and rank == 0 and world == 1:
        from oracle import scout_oracle as orc
        orc.build()
        cb, (tt, picked, osigs) = cpu_baseline(w, views, args.cpu_seconds if headline else args.cpu_seconds / 3)
        plan.sign()                              # records into a torch-owned buffer
        torch.cuda.synchronize()
        all_sigs = plan.d_sigs.cpu().numpy().view(binding.SIG_DTYPE).reshape(plan.C, w.R)
        first, c = {}, 0
        for t, s in enumerate(w.specs):
            first[t] = c
            c += (s.nbytes + w.chunk_bytes - 1) // w.chunk_bytes
        oc, ok = 0, True
        for i, t in enumerate(picked):
            n_ch = (int(tt[i]["nbytes"]) + w.chunk_bytes - 1) // w.chunk_bytes
            for k in range(n_ch):
                g, o = all_sigs[first[t] + k, 0], osigs[oc, 0]
                ok &= int(g["hash"]) == int(o["hash"]) and g["nan_count"] == o["nan_count"]
                ok &= abs(g["sumsq"] - o["sumsq"]) <= 1e-12 * abs(o["sumsq"])
                oc += 1
        cb["parity_spot_check"] = {"chunks": oc, "ok": bool(ok)}
        out["cpu_baseline"] = cb
        if not ok:
            raise SystemExit(f"{w.name}: CUDA records disagree with the oracle on the sampled chunks")
    else:
        out["cpu_baseline"] = None

    plan.close()
    del plan, views, flats, flush
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    return out


def run_distributed(args, rank, world, local):
    """The deployed form of C3 on config 4's state: ONE replica per GPU (R = N), each
    rank signs its own 12 GB, the [C] records are all-gathered over NCCL, every rank
    votes on the gathered table.  Same metric: bytes all ranks scanned / slowest rank."""
    import torch
    from paper_2608_11034_b200 import binding, dist_c3, dist_util, inputs

    w = inputs.workload(4, "default", args.scale)       # same seed on every rank: equivalent replicas
    flat, views = inputs.generate_replica0(w, "cuda")
    mine = [inputs.Patch(0, p.tensor, p.element, p.op, p.value) for p in w.patches if p.replica % world == rank]
    inputs.apply_patches([views], w.specs, mine)
    c3 = dist_c3.DistributedC3(binding.make_tensor_table(w.specs), w.chunk_bytes)
    c3.bind(views)
    for _ in range(max(args.warmup, 0)):
        c3.step()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    dist_util.barrier()
    torch.cuda.synchronize()
    for a, b in ev:
        a.record(); c3.step(); b.record()
    torch.cuda.synchronize()
    dist_util.barrier()
    ms = dist_util.max_over_ranks(sum(a.elapsed_time(b) for a, b in ev), dist_util.reduce_device())
    got = c3.fetch()
    # chunks that hold a patch must be the ones named (attributed with R >= 3; with R = 2 a
    # difference cannot be attributed and the chunk is listed as undecided)
    per_tensor = (w.specs[0].nbytes + w.chunk_bytes - 1) // w.chunk_bytes
    want = sorted({p.tensor * per_tensor + (p.element * 4) // w.chunk_bytes for p in w.patches})
    named = sorted({c for c, _ in got["outliers"]} | set(got["undecided"]))
    if named != want:
        raise SystemExit(f"distributed C3: chunks named {named}, expected {want}")
    n_chunks, on_device = c3.C, c3.device_transport
    c3.close()
    return {"value": world * w.bytes_per_replica * args.steps / (ms * 1e-3) / 1e9, "unit": UNIT,
            "ms_per_step": ms / args.steps, "R": world, "bytes_per_rank_per_step": w.bytes_per_replica,
            "gathered_bytes_per_rank": n_chunks * 32,
            "transport": "nccl all_gather_into_tensor" if on_device else "host all_gather (gloo)",
            "chunks_named": named, "form": "one replica per GPU: sign, all-gather records, vote on every rank"}


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist
    from paper_2608_11034_b200 import dist_util

    rank, world, local = dist_util.rank_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the product path has no CPU fallback)")
    # Test hook for boxes with one GPU: every rank uses cuda:0 and the ranks talk over gloo, so the
    # N > 1 code path (barrier, max over ranks, distributed C3) can run; its numbers mean nothing.
    one_gpu = os.environ.get("SCOUT_BENCH_ALL_RANKS_ON_GPU0") == "1"
    if one_gpu:
        local = 0
    torch.cuda.set_device(local)
    if world > 1:
        dist_util.init("gloo" if one_gpu else "nccl", torch.device("cuda", local))

    head = run_config(args.config, args, rank, world, local, headline=True)
    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u64+f64", "data": "synthetic",
        "config": dict(head["config"], parallelism=f"{world} independent replica sets" if world > 1 else "single GPU"),
        "launch": head["launch"],
        "frac_of_nominal_8TBs": head["frac_of_nominal_8TBs"],
        "frac_of_measured_copy": head["frac_of_measured_copy"],
        "verified": head["verified"], "verdict": head["verdict"],
        "gpu_launches": head["launch"]["kernels_per_step"] * args.steps,
        "clocks": head["clocks"], "roofline": head["roofline"], "l2_warm": head["l2_warm"],
        "l2_cold_rotating": head["l2_cold_rotating"], "one_launch": head["one_launch"], "compute_bound": head["compute_bound"],
        "e2e": head["e2e"], "cpu_baseline": head["cpu_baseline"],
    }

    # The other two large configs (bf16 parameters; 10,000 mixed tensors), measured the same
    # way after the headline config's buffers have been freed.
    if args.also is None:
        also = [3, 5] if (args.config == 4 and args.scale == 1.0 and world == 1 and not args.custom) else []
    else:
        also = [int(x) for x in args.also.split(",") if x]
    if also:
        line["also"] = {}
        for cfg in also:
            # a config that cannot run here (say, a board with less free memory) or that fails its own
            # check is reported as such; it does not take the headline line down with it
            try:
                r = run_config(cfg, args, rank, world, local, headline=False)
            except (Exception, SystemExit) as e:                       # noqa: BLE001
                line["also"][f"cfg{cfg}"] = {"error": repr(e)[:300], "verified": False}
                import gc
                gc.collect()
                torch.cuda.empty_cache()
                continue
            line["also"][r["config"]["workload"]] = {
                "value": r["value"], "ms_per_step": r["ms_per_step"],
                "bytes_per_step": r["config"]["bytes_per_step_per_gpu"],
                "frac_of_nominal_8TBs": r["frac_of_nominal_8TBs"],
                "roofline": {k: r["roofline"][k] for k in ("achieved", "frac", "avg_launch_ms", "launches_timed",
                                                          "scan_share_of_step_time", "read_probe_gbs",
                                                          "frac_of_read_probe")},
                "clocks": r["clocks"], "verified": r["verified"], "regime": r["launch"]["regime"],
                "tile_bytes": r["launch"]["tile_bytes"], "compute_bound": r["compute_bound"],
                "parity_spot_check": (r["cpu_baseline"] or {}).get("parity_spot_check"),
                "cpu_oracle_gbs": (r["cpu_baseline"] or {}).get("value"),
            }

    if world > 1:       # the paper's deployment form, next to the independent-sets number above
        line["distributed_c3"] = run_distributed(args, rank, world, local)

    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
