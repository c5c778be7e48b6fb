"""Benchmark of the fused-cluster executor on the five synthetic programs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of all five programs (1-D chain, transpose-fuse-reduce, random
gather + scan, four Jacobi iterations, scatter histogram + diamond) through
`acc_run(FUSED)` under the planner's clustering.  The metric is effective HBM
bandwidth: compulsory bytes (every program input read once + every program output
written once) divided by device time.  Rank 0 prints one JSON line.

Beside the step the line carries, per program: the unfused executor; every legal clustering
timed on its own (median and best of individually timed runs, the planner's choice marked);
the outputs on the timed buffers compared with the CPU oracle at full size (`parity`); and,
outside the step value, the 1-D chain at 2^28 elements and four further programs (segmented
sums over skewed segments, the paper's greedyBottomUpBad at m = 10^6, scans with readers).

With N > 1 every rank runs an independent replica on its own GPU (the path has no
exchange step); the value is the sum of bytes over ranks divided by the slowest rank.
`--impl reference` times the CPU oracle on the same programs at the same sizes.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "fused-pipeline effective HBM bandwidth (compulsory bytes / time), 5 synthetic programs"
FULL = {1: dict(n=1 << 16), 2: dict(rows=8192), 3: dict(n=1 << 26), 4: dict(rows=8192), 5: dict(n=1 << 27)}
SAMPLE = {1: dict(n=1 << 16), 2: dict(rows=4096), 3: dict(n=1 << 24), 4: dict(rows=4096), 5: dict(n=1 << 25)}
WORKLOAD = "configs 1-5 back to back, full sizes (2^16; 8192^2; 2^26; 8192^2 x 4 iterations; 2^27 keys, 2^16 bins)"
ORDER = [2, 3, 4, 5, 1]
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of each program's dominant kernel at full size
# (profiles/): a kernel that has changed since its capture has no entry
NCU_TRAFFIC = {3: 1.7371e9 + 0.7147e9, 4: 268.5e6 + 217.4e6, 2: 270.8e6 + 6.6e6, 5: 542.6e6 + 3.6e6}


def extra_programs(shrink):
    """Programs timed beside the step (not part of its value): name -> program."""
    import workloads as W
    k = 1 << shrink
    return {
        "1_scaled": W.config1((1 << 28) // k),
        "segmented_sums": W.segmented_sums((1 << 27) // k, (1 << 20) // k),
        "greedy_bottom_up_bad": W.greedy_bottom_up_bad(16, 1000000 // k),
        "scan_consumers": W.scan_consumers((1 << 26) // k),
        "offsets_then_gather": W.offsets_then_gather((1 << 26) // k),
    }


def scaled(sizes, shrink):
    """Sizes with every element count divided by 2^shrink (square arrays shrink by 2^(shrink/2) per side)."""
    out = {}
    for k, v in sizes.items():
        out[k] = max(4, v >> shrink) if k == "n" else max(4, v >> (shrink // 2))
    return out


def count_of(nd):
    c = 1
    for e in nd.shape:
        c *= int(e)
    return c


def compulsory_bytes(prog):
    ins = sum(count_of(prog.nodes[i]) for i in prog.input_ids())
    outs = sum(count_of(prog.nodes[i]) for i in prog.outputs)
    return 4 * (ins + outs)


def elements_of(prog):
    return max(count_of(nd) for nd in prog.nodes)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed steps, and the same steps repeated
    right after them, run."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(index), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.25)
        self.proc.terminate()
        try:
            text, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            return out
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in text.splitlines():
            f = [t.strip() for t in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


class Workload:
    """One program at one size: graph, device buffers, pinned host mirrors."""

    def __init__(self, name, prog, device, host=True, recompute=0):
        import torch
        import workloads as W
        from paper_2407_13585_b200 import binding as B
        self.cfg = name
        self.prog = prog
        self.bytes = compulsory_bytes(self.prog)
        self.elements = elements_of(self.prog)
        self.g = B.Graph(self.prog.nodes, self.prog.outputs)
        n_ops = sum(nd.kind != "input" for nd in self.prog.nodes)
        # small graphs: best of all legal clusterings; larger ones: branch and bound from the greedy result
        self.plan_mode = "enumerate" if n_ops <= 12 else "branch_bound"
        t0 = time.perf_counter()
        self.pi = self.g.plan_recompute(self.plan_mode, "bytes", recompute) if recompute else self.g.plan(self.plan_mode, "bytes")
        self.plan_ms = (time.perf_counter() - t0) * 1e3
        self.plan_visited, self.plan_proven = self.g.plan_info()
        self.refined = 0
        if not recompute:
            # a legal cluster nobody instantiated falls apart into clusters that have kernels
            self.refined, self.pi = self.g.refine_to_kernels()
        self.inputs = W.make_inputs(self.prog, device=device)
        self.outputs = {}
        self.host = {}
        for i, t in self.inputs.items():
            self.g.bind(i, t)
            if host:
                h = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
                h.copy_(t)
                self.host[i] = h
                self.g.bind_host(i, h)
        for o in self.prog.outputs:
            nd = self.prog.nodes[o]
            dt = torch.float32 if nd.dtype == "f32" else torch.int32
            t = torch.empty(max(count_of(nd), 4), dtype=dt, device=device)
            self.outputs[o] = t
            self.g.bind(o, t)
            if host:
                h = torch.empty(max(count_of(nd), 4), dtype=dt, pin_memory=True)
                self.host[o] = h
                self.g.bind_host(o, h)
        self.ws = {}
        self.B = B

    def run(self, executor):
        # each executor keeps its own workspace so that switching does not reallocate
        g = self.g
        if executor not in self.ws:
            g.workspace = None
            self.ws[executor] = g.ensure_workspace(executor)
        g.workspace = self.ws[executor]
        g.run(executor, finish=False)

    def finish(self):
        self.g.finish()

    def drop_workspace(self, executor):
        import torch
        self.ws.pop(executor, None)
        self.g.workspace = self.ws.get(self.B.FUSED)
        torch.cuda.empty_cache()

    def results(self):
        """The program's outputs as they lie in the bound device buffers: {node: numpy array}."""
        import numpy as np
        got = {}
        for o, t in self.outputs.items():
            nd = self.prog.nodes[o]
            a = t[:count_of(nd)].cpu().numpy()
            got[o] = (a.view(np.float32) if nd.dtype == "f32" else a.view(np.uint32)).reshape(tuple(nd.shape))
        return got


def time_region(fn, reps):
    import torch
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record()
    for _ in range(reps):
        fn()
    end.record()
    torch.cuda.synchronize()
    return start.elapsed_time(end) / reps


def timed_runs(fn, reps):
    """Device time of each of `reps` calls, every call between two events of its own."""
    import torch
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    torch.cuda.synchronize()
    for a, b in evs:
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in evs]


def config4_cuts(prog):
    """Two clusterings of the Jacobi chain between the legal minimum (one cluster per iteration) and no
    fusion: every iteration as {c, n, s, e, t1, t2, t3} | {w, Y}, and as five stored shifts | {t1, t2, t3, Y}."""
    iters = (len(prog.nodes) - 1) // 9
    two, six = [-1], [-1]
    for t in range(iters):
        two += [2 * t] * 4 + [2 * t + 1] + [2 * t] * 3 + [2 * t + 1]           # c n s e | w | t1 t2 t3 | Y
        six += [6 * t + k for k in range(5)] + [6 * t + 5] * 4
    return {"two_clusters_per_iteration": two, "shifts_stored": six}


def time_clusterings(w, reps):
    """Every legal clustering of a small program (for the Jacobi chain: the planner's and two coarser cuts),
    fused, each timed run by run.  The stored clustering is the planner's again afterwards."""
    import torch
    B = w.B
    n_ops = sum(nd.kind != "input" for nd in w.prog.nodes)
    if n_ops <= 12:
        named = [(None, pi) for pi in w.g.enumerate()]
    else:
        named = [("planner", list(w.pi))] + list(config4_cuts(w.prog).items())
    rows = []
    for label, pi in named:
        w.g.workspace = None
        torch.cuda.empty_cache()
        try:
            w.g.set_partition(pi)
            w.g.ensure_workspace(B.FUSED)
            for _ in range(3):
                w.g.run(B.FUSED, finish=False)
            ms = timed_runs(lambda: w.g.run(B.FUSED, finish=False), reps)
            w.g.finish()
        except B.AccError as e:
            rows.append({"clustering": pi, "error": e.status})
            continue
        row = {"clustering": pi, "clusters": len({c for c in pi if c >= 0}), "launches": w.g.launch_count(),
               "ms_median": statistics.median(ms), "ms_best": min(ms), "planner_choice": list(pi) == list(w.pi),
               "cost_bytes": w.g.partition_cost(pi, "bytes")}
        if label:
            row["label"] = label
        rows.append(row)
    w.g.workspace = None
    torch.cuda.empty_cache()
    w.g.set_partition(w.pi)
    w.g.workspace = w.ws.get(B.FUSED)
    return rows


def oracle_pass(progs_inputs):
    """Runs the oracle once on every (program, numpy inputs) pair; returns (bytes, seconds, [results])."""
    from oracle import interp
    total_b, total_s, results = 0, 0.0, []
    for prog, inputs in progs_inputs:
        t0 = time.perf_counter()
        results.append(interp.run(prog.nodes, inputs))
        total_s += time.perf_counter() - t0
        total_b += compulsory_bytes(prog)
    return total_b, total_s, results


def oracle_parity(w, seconds_out=None):
    """Oracle on the very inputs the timed runs read, compared with the outputs the timed runs left in their
    buffers (bit for bit, or within the stated tolerance of fp32 folds, scans and scatters).  Returns "ok" or raises."""
    tests = os.path.join(ROOT, "tests")
    if tests not in sys.path:
        sys.path.insert(0, tests)
    from helpers import compare
    inputs = {k: v.cpu().numpy() for k, v in w.inputs.items()}
    b, s, (ref,) = oracle_pass([(w.prog, inputs)])
    if seconds_out is not None:
        seconds_out.append((b, s))
    compare(w.prog, ref, w.results(), "%s on the timed buffers" % w.prog.name)
    del ref
    return "ok"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import workloads as W
    sizes = SAMPLE if args.cpu_baseline == "sample" else FULL
    pairs = []
    for cfg in ORDER:
        prog = W.CONFIGS[cfg](**scaled(sizes[cfg], args.shrink))
        pairs.append((prog, {k: v.numpy() for k, v in W.make_inputs(prog).items()}))
    # one step is a pass of the oracle over all five programs (minutes at full size): two at most
    warm = 1 if args.cpu_baseline == "sample" and args.warmup else 0
    for _ in range(warm):
        oracle_pass(pairs)
    steps = max(1, min(args.steps, 2))
    tb = ts = 0.0
    for _ in range(steps):
        b, s, res = oracle_pass(pairs)
        del res
        tb += b
        ts += s
    value = tb / ts / 1e9
    desc = ("oracle.interp on configs 1-5 at full size, one thread" if sizes is FULL else
            "oracle.interp on configs 2-5 at 1/4 of the elements (4096^2, 2^24, 4096^2 x 4 iterations, 2^25) and config 1 in full")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus, "steps": steps,
        "warmup": warm, "ms_per_step": ts / steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32/i32", "data": "synthetic",
        "config": {"workload": WORKLOAD if sizes is FULL and args.shrink == 0 else "configs 1-5 back to back (bounded sample)", "sample": desc},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_ours(args):
    import torch
    import torch.distributed as dist
    import workloads as W
    from paper_2407_13585_b200 import binding as B
    from paper_2407_13585_b200.replicas import combine_replicas, effective_gbs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    order = [c for c in ORDER if c in args.configs]
    loads = [Workload(cfg, W.CONFIGS[cfg](**scaled(FULL[cfg], args.shrink)), device, host=not args.fused_only,
                      recompute=args.recompute_depth if args.fused_only else 0) for cfg in order]
    step_bytes = sum(w.bytes for w in loads)

    def step():
        for w in loads:
            w.run(B.FUSED)

    sampler = ClockSampler(local) if rank == 0 else None     # nvidia-smi needs a few tenths of a second to start
    for _ in range(max(args.warmup, 3)):
        step()
    for w in loads:
        w.finish()

    barrier()
    ms_step = time_region(step, args.steps)
    if sampler:
        # the timed region may be shorter than the sampler's start-up: keep the same load running
        # (untimed) for half a second so that the clocks are read under it
        t_end = time.perf_counter() + 0.5
        while time.perf_counter() < t_end:
            step()
            torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else {}
    barrier()
    launches = sum(w.g.launch_count() for w in loads)
    for w in loads:
        w.finish()
    ms_step, job_bytes = combine_replicas(ms_step, step_bytes, dist if world > 1 else None, device)
    value = effective_gbs(job_bytes, ms_step)
    if args.fused_only:
        # profiling aid: only the fused steps above, no unfused / end-to-end / CPU legs
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": "GB/s", "ms_per_step": ms_step,
                              "config": {"workload": "configs %s, sizes / 2^%d" % (order, args.shrink)},
                              "gpu_launches": launches * args.steps}))
        if world > 1:
            dist.destroy_process_group()
        return

    # the outputs the timed steps left behind, against the oracle (rank 0, one GPU: the oracle is the CPU baseline too)
    peak, peak_kind = measured_peak()
    oracle_times = []
    parity = {}
    check = rank == 0 and world == 1 and args.cpu_baseline != "none"
    if check and args.cpu_baseline == "full":
        for w in loads:
            parity[w.cfg] = oracle_parity(w, oracle_times)

    # per program: fused and unfused executors side by side (rank 0's GPU)
    per = {}
    reps = max(3, min(args.steps, 20))
    for w in loads:
        for _ in range(3):
            w.run(B.FUSED)
        ms_f = time_region(lambda: w.run(B.FUSED), reps)
        n_f = w.g.launch_count()
        w.finish()
        for _ in range(3):
            w.run(B.UNFUSED)
        ms_u = time_region(lambda: w.run(B.UNFUSED), reps)
        n_u = w.g.launch_count()
        w.finish()
        w.drop_workspace(B.UNFUSED)
        per[w.cfg] = {
            "clustering": w.pi, "planner": w.plan_mode, "planner_ms": w.plan_ms, "planner_visited": w.plan_visited,
            "planner_proven_optimal": w.plan_proven, "ms_fused": ms_f, "ms_unfused": ms_u, "speedup": ms_u / ms_f,
            "launches_fused": n_f, "launches_unfused": n_u, "compulsory_bytes": w.bytes,
            "effective_gbs": w.bytes / ms_f / 1e6, "pct_of_8TBs": 100.0 * w.bytes / ms_f / 1e6 / NOMINAL_HBM_GBS,
            "gelem_s": w.elements / ms_f / 1e6,
        }
        if w.cfg in parity:
            per[w.cfg]["parity"] = parity[w.cfg]
        if rank == 0 and not args.no_clusterings:
            per[w.cfg]["clusterings"] = time_clusterings(w, reps)

    # Beside the paper's model: the Jacobi chain under a clustering that recomputes (two stacked
    # iterations per kernel, the iterate in between kept in shared memory).  Not part of the timed step.
    for w in loads:
        if w.cfg != 4:
            continue
        strict_pi = list(w.pi)
        pi2 = w.g.plan_recompute("branch_bound", "bytes", 2)
        w.g.workspace = None
        ws2 = w.g.ensure_workspace(B.FUSED)
        for _ in range(3):
            w.g.run(B.FUSED, finish=False)
        ms_r = time_region(lambda: w.g.run(B.FUSED, finish=False), reps)
        n_r = w.g.launch_count()
        w.g.finish()
        per[4]["recompute_depth_2"] = {
            "clustering": pi2, "ms_fused": ms_r, "launches_fused": n_r, "effective_gbs": w.bytes / ms_r / 1e6,
            "pct_of_8TBs": 100.0 * w.bytes / ms_r / 1e6 / NOMINAL_HBM_GBS, "speedup_vs_unfused": per[4]["ms_unfused"] / ms_r,
            "note": "outside the paper's legality model (its Section 6 leaves duplicated work to future work)"}
        w.g.set_partition(strict_pi)
        del ws2
        w.g.workspace = w.ws[B.FUSED]
        torch.cuda.empty_cache()

    # end to end: pinned host inputs in, outputs out, every step
    # (the programs go to two streams in turn, so that one program's copy back overlaps the next
    # one's copy in; the step ends when every program has been waited for)
    main = torch.cuda.current_stream()
    lanes = [torch.cuda.Stream(), torch.cuda.Stream()]

    def e2e_step():
        up = down = 0
        for lane in lanes:
            lane.wait_stream(main)
        for k, w in enumerate(loads):
            w.g.workspace = w.ws[B.FUSED]
            with torch.cuda.stream(lanes[k % 2]):
                u, d = w.g.run_e2e(B.FUSED, finish=False)
            up, down = up + u, down + d
        for k, w in enumerate(loads):
            with torch.cuda.stream(lanes[k % 2]):
                w.finish()
        for lane in lanes:
            main.wait_stream(lane)
        return up, down

    e2e_step()
    barrier()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    e2e_reps = max(1, min(args.steps, 5))
    for _ in range(e2e_reps):
        up, down = e2e_step()
    t1.record()
    torch.cuda.synchronize()
    ms_e2e = t0.elapsed_time(t1) / e2e_reps
    ms_e2e, _ = combine_replicas(ms_e2e, step_bytes, dist if world > 1 else None, device)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # the kernel that takes the largest share of a step (for config 3 the cluster's seven launches count as one:
    # they are the passes of one gather + scan, and the algorithmic bytes are those of the cluster)
    kernel_bytes = {2: lambda w: w.bytes, 3: lambda w: w.bytes, 4: lambda w: 8 * w.elements, 5: lambda w: w.bytes, 1: lambda w: w.bytes}
    kernel_launches = {2: 1, 3: 1, 4: 4, 5: 1, 1: 1}
    top = max(per, key=lambda c: per[c]["ms_fused"])
    wtop = [w for w in loads if w.cfg == top][0]
    achieved = kernel_bytes[top](wtop) / (per[top]["ms_fused"] / kernel_launches[top]) / 1e6
    # per program, the second level of the report: the dominant kernel's algorithmic bytes per launch over the
    # time of a launch (for the Jacobi chain: one iteration kernel, whose legal clustering caps the whole-DAG
    # figure at a quarter of this one)
    for w in loads:
        if w.cfg in per:
            gbs = kernel_bytes[w.cfg](w) / (per[w.cfg]["ms_fused"] / kernel_launches[w.cfg]) / 1e6
            per[w.cfg]["kernel_algorithmic_gbs"] = gbs
            per[w.cfg]["kernel_frac_of_copy_peak"] = gbs / peak
            per[w.cfg]["kernel_pct_of_8TBs"] = 100.0 * gbs / NOMINAL_HBM_GBS
    names = {2: "k_tile_pair_tma<transpose+zip+fold>", 3: "k_slab_probe + k_slab_partition + 4 x k_slab_gather + k_scan_merge_pipelined<hash+gather+mask+scan> (one cluster, seven launches)", 4: "k_stencil<jacobi iteration>",
             5: "k_hist<hash+generate+permute+fold>", 1: "k_stream<chain>"}
    traffic = NCU_TRAFFIC.get(top) if args.shrink == 0 else None
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "kernel": names[top], "of": peak_kind,
                "dram_rate": None if traffic is None else traffic / (per[top]["ms_fused"] / kernel_launches[top]) / 1e6,
                "bytes_per_launch": kernel_bytes[top](wtop), "launches_per_step": kernel_launches[top]}

    # the step's programs make room for the further ones
    del loads, wtop, w
    torch.cuda.empty_cache()

    extras = {}
    if world == 1 and not args.no_extras and len(order) == 5:
        for name, prog in extra_programs(args.shrink).items():
            w = Workload(name, prog, device, host=False)
            for _ in range(3):
                w.run(B.FUSED)
            ms = timed_runs(lambda: w.run(B.FUSED), reps)
            n_f = w.g.launch_count()
            w.finish()
            med = statistics.median(ms)
            row = {"clustering": w.pi, "planner": w.plan_mode, "clusters_split_for_lack_of_a_kernel": w.refined, "launches_fused": n_f,
                   "ms_fused": med, "ms_best": min(ms), "compulsory_bytes": w.bytes, "effective_gbs": w.bytes / med / 1e6,
                   "frac_of_copy_peak": w.bytes / med / 1e6 / peak, "clustering_traffic_bytes": w.g.partition_cost(w.pi, "bytes"),
                   "gelem_s": w.elements / med / 1e6}      # (the largest array of the program, stored or not, per second)
            if check and args.cpu_baseline == "full":
                row["parity"] = oracle_parity(w)
            for _ in range(3):
                w.run(B.UNFUSED)
            ms_u = timed_runs(lambda: w.run(B.UNFUSED), reps)
            row["ms_unfused"] = statistics.median(ms_u)
            row["launches_unfused"] = w.g.launch_count()
            row["speedup"] = row["ms_unfused"] / row["ms_fused"]
            w.finish()
            extras[name] = row
            del w
            torch.cuda.empty_cache()

    cpu = None
    if check:
        if args.cpu_baseline == "full":
            b, s = sum(t[0] for t in oracle_times), sum(t[1] for t in oracle_times)
            desc = "oracle.interp on configs 1-5 at full size, on the inputs of the timed runs, one thread"
        else:
            pairs = []
            for cfg in ORDER:
                prog = W.CONFIGS[cfg](**SAMPLE[cfg])
                pairs.append((prog, {k: v.numpy() for k, v in W.make_inputs(prog).items()}))
            b, s, _ = oracle_pass(pairs)
            desc = "oracle.interp on configs 2-5 at 1/4 of the elements (4096^2, 2^24, 4096^2 x 4 iterations, 2^25) and config 1 in full"
        cpu = {"value": b / s / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": desc, "seconds": s}

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32/i32", "data": "synthetic",
        "config": {"workload": WORKLOAD if args.shrink == 0 and len(order) == 5 else "configs %s, sizes / 2^%d" % (order, args.shrink),
                   "l2": "every program but config 1 streams more than the 126 MB L2 between reuses; no explicit flush",
                   "parallelism": "replicas only" if world > 1 else "1 GPU", "compulsory_bytes_per_step": step_bytes},
        "pct_of_8TBs": 100.0 * value / world / NOMINAL_HBM_GBS,
        "clocks": {"sm_mhz": clocks.get("sm_mhz"), "sm_max_mhz": clocks.get("sm_max_mhz"), "reasons": clocks.get("reasons", []),
                   "samples": clocks.get("samples", 0)},
        "e2e": {"value": world * step_bytes / (ms_e2e * 1e-3) / 1e9, "unit": "GB/s", "h2d_bytes_per_step": up,
                "d2h_bytes_per_step": down, "ms_per_step": ms_e2e},
        "gpu_launches": launches * args.steps,
        "roofline": roofline,
        "cpu_baseline": cpu,
        "parity": ("ok" if parity and all(v == "ok" for v in parity.values()) else None),
        "per_config": per,
        "further_programs": extras,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-baseline", default="full", choices=["full", "sample", "none"],
                    help="full: the oracle at full size on the timed inputs, outputs compared (minutes of CPU time); "
                         "sample: the oracle on quarter-size programs, no comparison; none: neither")
    ap.add_argument("--no-extras", action="store_true", help="skip the programs timed beside the step")
    ap.add_argument("--no-clusterings", action="store_true", help="skip the per-clustering timings")
    ap.add_argument("--configs", default="1,2,3,4,5", help="programs to include (profiling aid)")
    ap.add_argument("--shrink", type=int, default=0, help="divide every element count by 2^SHRINK (profiling aid)")
    ap.add_argument("--fused-only", action="store_true", help="time the fused steps only (profiling aid)")
    ap.add_argument("--recompute-depth", type=int, default=0,
                    help="with --fused-only: plan with clusterings that recompute, this many stacked gather-like nodes (profiling aid)")
    args = ap.parse_args()
    args.configs = [int(c) for c in args.configs.split(",")]
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
