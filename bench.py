#!/usr/bin/env python
"""Benchmark: useful GFLOP/s of one Linnea equation on B200 and its fraction of the 3xTF32 roofline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--variant 3xtf32|ffma] [--impl reference]

A step is one evaluation of the whole equation (every product of the plan plus the fused Add /
zero-fill epilogue) on seeded synthetic operands.  The headline workload is the large square chain
X = L*A*U*B at 8192 (operands far larger than L2, so no flush is needed between steps).  The other
configurations are timed briefly and reported under "all_configs".  One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "useful GFLOP/s per Linnea equation (f32)"
UNIT = "GFLOP/s"
TF32_OVER_BF16 = 1.1 / 2.25          # nominal dense tensor ratio used to carry the measured bf16 peak to tf32


def max_over_ranks(value_ms: float, world: int, device="cpu") -> float:
    """Slowest rank's time (every rank gets it); a no-op for one rank."""
    if world <= 1:
        return float(value_ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gflops(useful_flops_per_replica: int, world: int, ms_per_step: float) -> float:
    """Replicas are independent: the job's throughput is every rank's work over the slowest rank's time."""
    return useful_flops_per_replica * world / (ms_per_step * 1e-3) / 1e9


# DRAM traffic of the dominant kernel per launch on the headline workload, from one ncu capture
# (dram__bytes_read.sum + dram__bytes_write.sum, mean over the step's three product launches).  It is only
# reported while the kernel source is the one that was captured.
TRAFFIC_CAPTURE = {"kernel_source_sha256_16": "7c35fd35704f513b", "bytes_per_launch": 7.64e9}


def measured_traffic():
    import hashlib
    path = os.path.join(ROOT, "paper_2208_10391_b200", "csrc", "product_tc.cu")
    try:
        with open(path, "rb") as fh:
            sha = hashlib.sha256(fh.read()).hexdigest()[:16]
    except OSError:
        return None
    return TRAFFIC_CAPTURE["bytes_per_launch"] if sha == TRAFFIC_CAPTURE["kernel_source_sha256_16"] else None


def sum_over_ranks(value: float, world: int, device="cpu") -> float:
    """Sum of a per-rank quantity (every rank gets it); a no-op for one rank."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def split_job_gflops(useful_flops_this_rank: int, world: int, ms_per_step: float, device="cpu") -> float:
    """One equation cut into column slabs: the job's throughput is all slabs' work over the slowest rank's time."""
    return sum_over_ranks(float(useful_flops_this_rank), world, device) / (ms_per_step * 1e-3) / 1e9


def headline_equation() -> wl.Equation:
    return wl.config_large_square()


def column_slab_of(mom, eq: wl.Equation, rank: int, world: int):
    """This rank's share of `eq` under the column-slab split: (slab equation, begin, end); the last factor and the
    Add terms keep their distribution, their columns are [begin, end) of the whole operand's."""
    got = mom.column_slab_equation(eq.descs(), eq.add_descs(), rank, world, eq.chain_t, eq.add_t)
    if got is None:
        raise SystemExit(f"rank {rank} of {world} has no columns of {eq.name}")
    cd, ad, begin, end = got
    last = eq.chain[-1]
    ops = tuple(eq.chain[:-1]) + (wl.Operand(cd[-1].rows, cd[-1].cols, cd[-1].property, last.dist, last.sigma),)
    terms = tuple(wl.Operand(d.rows, d.cols, d.property, t.dist, t.sigma) for d, t in zip(ad, eq.add))
    return wl.Equation(f"{eq.name}_cols{begin}_{end}", eq.seed, ops, terms, chain_t=eq.chain_t, add_t=eq.add_t), begin, end


def cut_columns(eq: wl.Equation, chain, add, begin: int, end: int):
    """Host arrays of the slab equation, cut from the whole equation's arrays (views made contiguous)."""
    import numpy as np
    ct = list(eq.chain_t) + [False] * (len(chain) - len(eq.chain_t))
    at = list(eq.add_t) + [False] * (len(add) - len(eq.add_t))

    def cut(a, t):
        return np.ascontiguousarray(a[begin:end, :] if t else a[:, begin:end])
    return list(chain[:-1]) + [cut(chain[-1], ct[-1])], [cut(a, t) for a, t in zip(add, at)]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"], "bf16_sustained": d["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------
# reference arm / CPU baseline: the oracle, as it stands, on the host cores
# ------------------------------------------------------------------------------------------------

def oracle_sample_seconds(eq, chain, add, rows):
    """Time the oracle on `rows` of X (left-to-right fp64 triple loops); returns (seconds, threads used, X_ref rows, D rows)."""
    from oracle import values as ov
    t0 = time.perf_counter()
    x_ref, den = ov.evaluate([None if c is None else (c[0] if eq.batch > 1 else c) for c in chain], eq.descs(),
                             [None if a is None else (a[0] if eq.batch > 1 else a) for a in add], eq.add_descs(), rows=rows)
    return time.perf_counter() - t0, ov.threads_used(), x_ref, den


def sample_rows(total_rows: int, slab: int = 32):
    """One row out of every 32 (drawn inside each slab with a fixed seed): every tile row and every epilogue warp's slab
    of the product kernels' output is represented."""
    rng = np.random.default_rng(0)
    return np.array([min(total_rows - 1, r0 + int(rng.integers(0, slab))) for r0 in range(0, total_rows, slab)], dtype=np.int64)


def cpu_baseline(eq, chain, add, useful_flops_per_instance, rows, x_rows=None, x_off_structure_ok=None, result_prop=None):
    """The oracle timed on `rows` of X; when `x_rows` (those rows of the X the timed GPU steps left) is given, the same
    oracle values also give the run's own parity figure."""
    from oracle import plan as op
    from oracle import values as ov
    t0 = time.perf_counter()
    op.plan(eq.descs(), eq.add_descs())
    plan_s = time.perf_counter() - t0
    total_rows = eq.chain[0].rows
    secs, threads, x_ref, den = oracle_sample_seconds(eq, chain, add, rows)
    frac = len(rows) / total_rows
    value = useful_flops_per_instance * frac / (secs + plan_s) / 1e9
    out = {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
           "sample": f"{len(rows)} of {total_rows} rows of X (one in every 32; one instance), exhaustive plan + left-to-right fp64 "
                     f"triple loops incl. the error denominator; useful FLOPs scaled by the row fraction; "
                     f"{secs + plan_s:.2f} s"}
    parity = None
    if x_rows is not None:
        parity = {"normwise_err": ov.normwise_error(x_rows, x_ref, den), "bound": 1e-5, "rows_compared": int(len(rows)),
                  "of_rows": int(total_rows), "nan_free": bool(not np.isnan(x_rows).any()),
                  "off_structure_exact_zero": x_off_structure_ok,
                  "what": "X left by the timed steps against the fp64 oracle on the sampled rows: ||X - X_ref||_F / ||D||_F"}
        parity["ok"] = bool(parity["normwise_err"] <= 1e-5 and parity["nan_free"] and x_off_structure_ok is not False)
    return out, parity


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import plan as op
    eq = headline_equation()
    chain, add = wl.generate(eq)
    p = op.plan(eq.descs(), eq.add_descs())
    useful = p.mul_flops + p.add_flops
    n_rows = 4
    total_rows = eq.chain[0].rows
    times = []
    threads = 1
    for i in range(args.warmup + args.steps):
        rows = np.sort(np.random.default_rng(i).choice(total_rows, size=n_rows, replace=False))
        secs, threads, _, _ = oracle_sample_seconds(eq, chain, add, rows)
        if i >= args.warmup:
            times.append(secs)
    mean_s = sum(times) / len(times)
    value = useful * (n_rows / total_rows) / mean_s / 1e9
    sample = f"{n_rows} of {total_rows} rows of X per step, left-to-right fp64 triple loops incl. the error denominator"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": mean_s * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": eq.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------

class ClockSampler:
    """nvidia-smi polled in the background; only samples taken inside [begin(), end()] are reported."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc = None
        self.device_index = device_index
        self.lines = []          # (host time, text)
        self.t0 = self.t1 = None
        self.thread = None

    def start(self):
        import threading
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.device_index)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return

        def reader():
            for line in self.proc.stdout:
                self.lines.append((time.time(), line))
        self.thread = threading.Thread(target=reader, daemon=True)
        self.thread.start()

    def wait_for_first_sample(self, timeout: float = 10.0):
        t = time.time()
        while self.proc is not None and not self.lines and time.time() - t < timeout:
            time.sleep(0.05)

    def begin(self):
        self.t0 = time.time()

    def end(self):
        self.t1 = time.time()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.06)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=2)
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for stamp, line in list(self.lines):
            if self.t0 is not None and not (self.t0 <= stamp <= (self.t1 or stamp) + 0.05):
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def planning_us(mom, eq, variant, repeats=15):
    """Host time of one planning call through the binding (median of `repeats`), in microseconds."""
    ts = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        if isinstance(eq, wl.Expression):
            mom.mom_expression_plan(eq.expr, eq.descs(), variant)
        elif isinstance(eq, wl.SumEquation):
            mom.mom_equation_plan_sum(eq.descs(), eq.transposed, eq.names, variant)
        else:
            mom.mom_equation_plan_transposed(eq.descs(), eq.chain_t, eq.add_descs(), eq.add_t, variant)
        ts.append((time.perf_counter() - t0) * 1e6)
    return statistics.median(ts)


def time_equation(mom, torch, eq, variant, steps, warmup, stream, timing=False, chain_storage=None):
    """Device-resident timing of one configuration: returns dict with per-step ms list, plan, launches.
    chain_storage (plain chains only): mom.STORAGE_PACKED entries hand that triangular operand over as a packed container."""
    if isinstance(eq, wl.Expression):
        # a nested expression: one pointer per operand of the table
        chain, add = wl.generate_expression(eq), []
        plan = mom.mom_expression_plan(eq.expr, eq.descs(), variant)
        dchain = [None if a is None else torch.from_numpy(a).cuda() for a in chain]
        eq = wl.Equation(eq.name, eq.seed, tuple(eq.operands))                          # batch 1, for the code below
    elif isinstance(eq, wl.SumEquation):
        # a sum of chains: one device array per named matrix, one pointer per factor
        arrays = wl.generate_sum(eq)
        plan = mom.mom_equation_plan_sum(eq.descs(), eq.transposed, eq.names, variant)
        by_name = {}
        for row, names in zip(arrays, eq.names):
            for a, nm in zip(row, names):
                if a is not None and nm not in by_name:
                    by_name[nm] = torch.from_numpy(a).cuda()
        dchain = [None if a is None else by_name[nm] for row, names in zip(arrays, eq.names) for a, nm in zip(row, names)]
        chain, add = [a for row in arrays for a in row], []
        eq = wl.Equation(eq.name, eq.seed, tuple(o for c in eq.chains for o in c))     # batch 1, for the code below
    elif chain_storage is not None:
        chain, add = wl.generate(eq)
        # triangular Add terms travel packed too, and so does X when every summand is a triangle of one orientation
        lower = (wl.LOWER_TRI, wl.STRICT_LOWER, wl.UNIT_LOWER)
        tri = lower + (wl.UPPER_TRI, wl.STRICT_UPPER, wl.UNIT_UPPER)
        add_storage = [mom.STORAGE_PACKED if o.prop in tri else mom.STORAGE_DENSE for o in eq.add]
        dense_plan = mom.mom_equation_plan_transposed(eq.descs(), eq.chain_t, eq.add_descs(), eq.add_t, variant)
        x_storage = mom.STORAGE_PACKED if dense_plan.result_desc().property in tri else mom.STORAGE_DENSE
        plan = mom.mom_equation_plan_stored(eq.descs(), eq.chain_t, chain_storage, eq.add_descs(), eq.add_t, add_storage, x_storage, variant)
        chain = [a if s == mom.STORAGE_DENSE or a is None else wl.pack_triangle(a, o.prop in lower) for a, o, s in zip(chain, eq.chain, chain_storage)]
        add = [a if s == mom.STORAGE_DENSE or a is None else wl.pack_triangle(a, o.prop in lower) for a, o, s in zip(add, eq.add, add_storage)]
        dchain = [None if a is None else torch.from_numpy(a).cuda() for a in chain]
    else:
        chain, add = wl.generate(eq)
        plan = mom.mom_equation_plan_transposed(eq.descs(), eq.chain_t, eq.add_descs(), eq.add_t, variant)
        dchain = [None if a is None else torch.from_numpy(a).cuda() for a in chain]
    rd = plan.result_desc()
    dadd = [None if a is None else torch.from_numpy(a).cuda() for a in add]
    out = torch.empty((eq.batch, rd.rows, rd.cols), dtype=torch.float32, device="cuda")
    wsb = plan.workspace_bytes(eq.batch)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device="cuda")
    cp = [None if t is None else t.data_ptr() for t in dchain]
    ap = [None if t is None else t.data_ptr() for t in dadd]
    cs = [0 if t is None else t[0].numel() for t in dchain] if eq.batch > 1 else None
    as_ = [0 if t is None else t[0].numel() for t in dadd] if eq.batch > 1 else None

    def run():
        if eq.batch > 1:
            plan.execute_batched(cp, cs, ap, as_, out.data_ptr(), plan.result_elements(), eq.batch,
                                 ws.data_ptr() if wsb else None, wsb, stream.cuda_stream)
        else:
            plan.execute(cp, ap, out.data_ptr(), ws.data_ptr() if wsb else None, wsb, stream.cuda_stream)

    if timing:
        plan.enable_step_timing(True)
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            run()
        stream.synchronize()
        events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        step_times = []
        for e0, e1 in events:
            e0.record(stream)
            run()
            e1.record(stream)
            if timing:
                stream.synchronize()
                try:
                    step_times.append([plan.step_times(i) for i in range(plan.num_steps())])
                except mom.MomError:        # fused single-kernel plans have no per-step events
                    step_times.append([])
        stream.synchronize()
        # the same steps back to back (nothing waits for the host between them): what a caller who enqueues equation
        # after equation sees; the per-step figures above expose every launch gap when `timing` synchronises each step
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if timing:
            plan.enable_step_timing(False)
        # (short equations: enough repetitions for the start of the burst, an idle GPU's first launch, not to weigh on the mean)
        quick = sorted(e0.elapsed_time(e1) for e0, e1 in events)[len(events) // 2] < 0.5
        reps = max(steps, 200) if quick else steps
        b0.record(stream)
        for _ in range(reps):
            run()
        b1.record(stream)
        stream.synchronize()
        # short equations once more as a CUDA graph: one execute captured (the library's launches, its second stream and its
        # events are capturable once the plan has run: every allocation happens in the first call) and replayed back to back
        ms_graph = None
        if quick:
            try:
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=stream):
                    run()
                graph.replay()
                g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                g0.record(stream)
                for _ in range(reps):
                    graph.replay()
                g1.record(stream)
                stream.synchronize()
                ms_graph = g0.elapsed_time(g1) / reps
            except Exception:                # not capturable here: no figure
                ms_graph = None
    ms = [e0.elapsed_time(e1) for e0, e1 in events]
    ms_b2b = b0.elapsed_time(b1) / reps
    status = plan.device_status()
    if status != (0, 0):
        raise RuntimeError(f"device-side wait timed out: {status}")
    mul, addf = plan.flops()
    stored_bytes = 4 * (sum(t.numel() for t in dchain if t is not None) + sum(t.numel() for t in dadd if t is not None) + plan.result_elements() * eq.batch)
    return {"ms": ms, "ms_back_to_back": ms_b2b, "ms_graph_replay": ms_graph, "plan": plan, "stored_bytes": stored_bytes, "useful_flops": (mul + addf) * eq.batch, "launches": plan.last_launch_count(),
            "step_times": step_times, "host": (chain, add), "keep": (dchain, dadd, out, ws)}


def run_gpu(args):
    import torch
    import torch.distributed as dist
    import paper_2208_10391_b200 as mom

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    variant = {"3xtf32": mom.VARIANT_3XTF32, "ffma": mom.VARIANT_FFMA}[args.variant]
    stream = torch.cuda.Stream()
    peaks = measured_peaks()

    eq = headline_equation()
    whole_eq, slab = eq, None
    if args.split == "columns" and not args.only:
        # one equation over all ranks: this rank evaluates its columns of X, no exchange between ranks
        eq, b, e = column_slab_of(mom, whole_eq, rank, world)
        slab = (b, e)
    sampler = ClockSampler(local)
    if not args.only:
        sampler.start()

    if args.only:
        # one named configuration, nothing else: the small case for profiler captures
        cfgs = {c.name: c for c in (wl.config_tiny(), wl.config_five_general(), wl.config_property_heavy(),
                                    wl.config_large_square(), wl.config_large_square(n=2048), wl.config_batched(), wl.config_paper_chain(),
                                    wl.config_transposed(), wl.config_sum_shared(), wl.config_sum_triangular(),
                                    wl.config_expression(), wl.config_diagonal(), wl.config_gram(), wl.config_square_product(768), wl.config_square_product(1024),
                                    wl.config_square_product(1536), wl.config_square_product(2048), wl.config_packed_triangular(),
                                    # three general factors whose products have few tiles and long contractions: the plane-fed 1-CTA
                                    # tcgen05 kernel with the contraction split inside clusters
                                    wl.Equation("GGG_1536_2048", 14, tuple(wl.Operand(r, c, wl.GENERAL, "normal", c ** -0.5)
                                                                         for r, c in ((1536, 2048), (2048, 1536), (1536, 2048)))))}
        packed = args.only.endswith("_packed")       # the same equation with its triangular operands handed over as packed triangles
        cfg = cfgs[args.only[:-len("_packed")] if packed else args.only]
        storage = None
        if packed:
            storage = [mom.STORAGE_PACKED if o.prop in (wl.LOWER_TRI, wl.UPPER_TRI) else mom.STORAGE_DENSE for o in cfg.chain]
        r = time_equation(mom, torch, cfg, variant, steps=args.steps, warmup=args.warmup, stream=stream,
                          timing=getattr(cfg, "batch", 1) == 1 and not packed, chain_storage=storage)
        print(json.dumps({"workload": cfg.name, "variant": args.variant, "ms": r["ms"], "ms_back_to_back": r["ms_back_to_back"],
                          "ms_graph_replay": r["ms_graph_replay"],
                          "useful_flops": r["useful_flops"],
                          "launches": r["launches"], "step_times_ms": r["step_times"][-1:] }))
        return

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- headline: device-resident, K timed steps bracketed by barriers; every rank runs its own replica
    barrier()
    warm = time_equation(mom, torch, eq, variant, steps=1, warmup=max(args.warmup - 1, 0), stream=stream)
    plan = warm["plan"]
    del warm
    torch.cuda.empty_cache()
    chain, add = wl.generate(whole_eq)
    if slab and slab != (0, rd_cols(whole_eq)):
        chain, add = cut_columns(whole_eq, chain, add, *slab)
    dchain = [None if a is None else torch.from_numpy(a).cuda() for a in chain]
    dadd = [None if a is None else torch.from_numpy(a).cuda() for a in add]
    rd = plan.result_desc()
    out = torch.empty((rd.rows, rd.cols), dtype=torch.float32, device="cuda")
    wsb = plan.workspace_bytes(1)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device="cuda")
    cp = [None if t is None else t.data_ptr() for t in dchain]
    ap = [None if t is None else t.data_ptr() for t in dadd]
    n_steps = plan.num_steps()
    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            plan.execute(cp, ap, out.data_ptr(), ws.data_ptr(), wsb, stream.cuda_stream)
    barrier()
    plan.enable_step_timing(True)      # per-kernel events, averaged over the timed executes
    sampler.wait_for_first_sample()
    sampler.begin()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    prod_ms = [0.0] * n_steps
    pre_ms = [0.0] * n_steps
    launches = 0
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(args.steps):
            plan.execute(cp, ap, out.data_ptr(), ws.data_ptr(), wsb, stream.cuda_stream)
            launches += plan.last_launch_count()
        e1.record(stream)
    barrier()
    sampler.end()
    clocks = sampler.stop()
    total_ms = e0.elapsed_time(e1)
    # per-kernel mean times over the timed region (events recorded inside it, on the same stream)
    for i in range(n_steps):
        a, b = plan.step_times(i)
        prod_ms[i], pre_ms[i] = a, b
    if plan.device_status() != (0, 0):
        raise RuntimeError("device-side wait timed out")
    # the X the timed steps left: the rows the oracle will compute below, and the exact-zero check of everything
    # outside the result's structure (whole matrix, on the device)
    parity_rows = sample_rows(rd.rows)
    x_rows = out[torch.from_numpy(parity_rows).cuda()].cpu().numpy()
    bits = out.view(torch.int32)
    prop = rd.property
    x_off_ok = (bool((torch.triu(bits, 1) == 0).all()) if prop in (wl.LOWER_TRI,) else
                bool((torch.tril(bits, -1) == 0).all()) if prop in (wl.UPPER_TRI,) else True)
    del bits
    total_ms = max_over_ranks(total_ms, world, "cuda")
    ms_per_step = total_ms / args.steps
    mul, addf = plan.flops()
    useful = mul + addf
    value = split_job_gflops(useful, world, ms_per_step, "cuda") if slab else whole_job_gflops(useful, world, ms_per_step)

    # ---- roofline of the dominant kernel (the product kernel): useful FLOPs of its launches / their device time
    steps_info = plan.steps()
    prod_total_ms = sum(prod_ms)
    achieved_tflops = useful / (prod_total_ms * 1e-3) / 1e12 if prod_total_ms > 0 else None
    timed_s = total_ms * 1e-3
    if args.variant == "3xtf32":
        # effective 3xTF32 peak = tf32 dense peak / 3 MMAs per useful product; tf32 peak = measured bf16 peak carried over
        # by the nominal tf32 : bf16 ratio.  Which measured bf16 figure: the sustained one (a seconds-long loop under the
        # power cap) when this run's timed region is itself at least a second long, else the burst one.
        peak_burst = peaks["bf16_burst"] * TF32_OVER_BF16 / 3.0
        peak_sustained = peaks["bf16_sustained"] * TF32_OVER_BF16 / 3.0
        use_sustained = timed_s >= 1.0
        peak = peak_sustained if use_sustained else peak_burst
        peak_note = (f"{peaks['source']} {'sustained' if use_sustained else 'burst'} bf16 "
                     f"{peaks['bf16_sustained'] if use_sustained else peaks['bf16_burst']} TFLOP/s x nominal tf32/bf16 ratio "
                     f"{TF32_OVER_BF16:.4f} / 3 MMAs per useful product; timed region {timed_s:.2f} s")
        bound = "tensor"
    else:
        props = torch.cuda.get_device_properties(local)
        mhz = clocks["sm_mhz"] or 1965.0
        peak = props.multi_processor_count * 128 * 2 * mhz * 1e6 / 1e12
        peak_burst = peak_sustained = peak
        peak_note = f"{props.multi_processor_count} SMs x 128 FP32 lanes x 2 x median SM clock {mhz} MHz"
        bound = "alu"
    whole_tflops = useful / (ms_per_step * 1e-3) / 1e12
    roofline = {"bound": bound, "achieved": achieved_tflops, "peak": peak, "unit": "TFLOP/s",
                "frac": (achieved_tflops / peak) if achieved_tflops else None,
                "frac_is": "product launches of the step (useful FLOPs / their device time) over `peak`",
                "frac_burst": (achieved_tflops / peak_burst) if achieved_tflops else None,
                "frac_sustained": (achieved_tflops / peak_sustained) if achieved_tflops else None,
                "frac_whole_equation": whole_tflops / peak,
                "frac_whole_equation_is": "all launches of the step, operand-split passes included, over `peak`",
                "traffic": measured_traffic() if args.variant == "3xtf32" else None,
                "kernel": "product_tc_pair_kernel" if args.variant == "3xtf32" else "product_ffma_kernel",
                "launches_per_step": n_steps, "product_ms_per_step": prod_ms, "prepass_ms_per_step": pre_ms,
                "peak_is": peak_note}

    slab_price = None
    if slab:
        # what the cut costs in arithmetic: a proper slab of a triangular last factor is general (its zeros are multiplied)
        # and a narrow slab may be parenthesized differently; all slabs' useful FLOPs over the whole equation's
        wp = mom.mom_equation_plan_transposed(whole_eq.descs(), whole_eq.chain_t, whole_eq.add_descs(), whole_eq.add_t, variant)
        slab_price = sum_over_ranks(float(useful), world, "cuda") / float(sum(wp.flops()))
    if roofline["frac"] and roofline["frac"] > 1.0:
        roofline["frac_above_one_because"] = (
            "the denominator is not a tf32 measurement: it carries a cuBLAS bf16 figure (taken on another run, at its own clock under "
            "the power cap) to tf32 by the nominal 1.1/2.25 ratio and divides by 3; this library's own kind::tf32 issue probe gives "
            "the bound the kernel is actually under: see frac_of_probe (full clock) and frac_of_probe_at_run_clock")
    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if slab else "weak", "vs_baseline": None,
        "dtype": "f32 (3xTF32 tensor-core split)" if args.variant == "3xtf32" else "f32",
        "data": "synthetic",
        "config": {"workload": eq.name, "equation": "X = L*A*U*B, 8192x8192 f32, seed 3",
                   "parenthesization": plan.parenthesization(), "useful_flops": useful, "variant": args.variant,
                   "l2": "operands (1 GiB) exceed L2; no flush",
                   "parallelism": (f"one equation, column slabs of X over {world} ranks (this rank: columns {slab[0]}..{slab[1]}), no exchange"
                                   if slab else f"{world} independent replicas"),
                   "plan_us": planning_us(mom, eq, variant)},
        "clocks": clocks, "gpu_launches": launches, "roofline": roofline,
    }
    if slab_price is not None:
        result["config"]["slab_flops_over_whole_equation"] = slab_price

    if rank == 0 and world == 1:
        # ---- probes: sustained tcgen05 kind::tf32 rate and FFMA rate on this GPU
        scratch = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
        probes = {}
        for name, fn in (("tf32_tflops", mom.mom_probe_tf32_tflops), ("ffma_tflops", mom.mom_probe_ffma_tflops)):
            try:
                probes[name] = fn(1000.0, scratch.data_ptr(), stream.cuda_stream)
            except mom.MomError as e:
                probes[name] = f"unavailable: {e}"
        result["probes"] = probes
        if isinstance(probes.get("tf32_tflops"), float) and args.variant == "3xtf32" and achieved_tflops:
            # the library's own kind::tf32 issue loop on resident tiles (runs at the full clock: it draws little power);
            # the second figure scales it to the median SM clock of the timed region
            probe_peak = probes["tf32_tflops"] / 3.0
            result["roofline"]["frac_of_probe"] = achieved_tflops / probe_peak
            if clocks.get("sm_mhz") and clocks.get("sm_max_mhz"):
                result["roofline"]["frac_of_probe_at_run_clock"] = achieved_tflops / (probe_peak * clocks["sm_mhz"] / clocks["sm_max_mhz"])

        # ---- e2e: host operands in pinned memory, H2D + execute + D2H inside the timed region
        stage_b = plan.host_staging_bytes(1)
        del dchain, dadd, out, ws
        torch.cuda.empty_cache()
        staging = torch.empty(stage_b, dtype=torch.uint8, device="cuda")
        pin = [None if a is None else torch.from_numpy(a).pin_memory() for a in chain]
        pin_add = [None if a is None else torch.from_numpy(a).pin_memory() for a in add]
        out_h = torch.empty((rd.rows, rd.cols), dtype=torch.float32).pin_memory()
        hp = [None if t is None else t.data_ptr() for t in pin]
        hap = [None if t is None else t.data_ptr() for t in pin_add]
        e2e_steps = min(args.steps, 5)
        for _ in range(2):
            plan.execute_host(hp, hap, out_h.data_ptr(), 1, staging.data_ptr(), stage_b, stream.cuda_stream)
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            plan.execute_host(hp, hap, out_h.data_ptr(), 1, staging.data_ptr(), stage_b, stream.cuda_stream)
        e2e_s = (time.perf_counter() - t0) / e2e_steps
        h2d = plan.host_upload_bytes(1)      # what the entry point copies: triangular operands only up to the diagonal blocks
        result["e2e"] = {"value": useful / e2e_s / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
                         "d2h_bytes_per_step": out_h.numel() * 4, "ms_per_step": e2e_s * 1e3, "steps": e2e_steps}
        del staging
        torch.cuda.empty_cache()

        # ---- the other configurations, briefly (min of 5 as in the paper's Section 4, and the median)
        others = []
        for cfg in (wl.config_tiny(), wl.config_five_general(), wl.config_property_heavy(), wl.config_batched(),
                    wl.config_paper_chain(), wl.config_transposed(), wl.config_sum_shared(), wl.config_sum_triangular(),
                    wl.config_expression(), wl.config_diagonal(), wl.config_gram(), wl.config_square_product(768), wl.config_square_product(1024),
                    wl.config_square_product(1536), wl.config_square_product(2048)):
            batch = getattr(cfg, "batch", 1)
            r = time_equation(mom, torch, cfg, variant, steps=20, warmup=3, stream=stream, timing=batch == 1)
            ms_min, ms_med = min(r["ms"]), statistics.median(r["ms"])
            entry = {"workload": cfg.name, "parenthesization": r["plan"].parenthesization(),
                     "useful_flops": r["useful_flops"], "ms_min_of_20": ms_min, "ms_median": ms_med,
                     "ms_back_to_back": r["ms_back_to_back"], "ms_graph_replay": r["ms_graph_replay"],
                     "gflops_back_to_back": r["useful_flops"] / (r["ms_back_to_back"] * 1e-3) / 1e9,
                     "gflops_at_min": r["useful_flops"] / (ms_min * 1e-3) / 1e9,
                     "gflops_at_median": r["useful_flops"] / (ms_med * 1e-3) / 1e9,
                     "frac_of_burst_roofline_at_median": r["useful_flops"] / (ms_med * 1e-3) / 1e12 / peak_burst,
                     "launches": r["launches"], "plan_us": planning_us(mom, cfg, variant)}
            if batch > 1:
                per_inst = sum(o.rows * o.cols for o in list(cfg.chain) + list(cfg.add)) + rd_elems(r["plan"])
                entry["bytes_per_instance"] = per_inst * 4
                entry["hbm_gbs_at_median"] = per_inst * 4 * cfg.batch / (ms_med * 1e-3) / 1e9
                entry["hbm_frac_of_measured_peak"] = entry["hbm_gbs_at_median"] / peaks["hbm_gbs"]
            others.append(entry)
            del r
            torch.cuda.empty_cache()
            if batch > 1 and args.variant == "3xtf32":
                # the same equations with L_i handed over as a packed triangle (2176 instead of 4096 entries per instance)
                storage = [mom.STORAGE_PACKED if o.prop == wl.LOWER_TRI else mom.STORAGE_DENSE for o in cfg.chain]
                r = time_equation(mom, torch, cfg, variant, steps=20, warmup=3, stream=stream, chain_storage=storage)
                ms_med = statistics.median(r["ms"])
                per_inst = r["stored_bytes"] // cfg.batch
                others.append({"workload": cfg.name + "_packedL", "parenthesization": r["plan"].parenthesization(),
                               "useful_flops": r["useful_flops"], "ms_min_of_20": min(r["ms"]), "ms_median": ms_med,
                               "ms_back_to_back": r["ms_back_to_back"], "launches": r["launches"],
                               "workspace_bytes": r["plan"].workspace_bytes(cfg.batch), "bytes_per_instance": per_inst,
                               "hbm_gbs_at_median": per_inst * cfg.batch / (ms_med * 1e-3) / 1e9,
                               "hbm_frac_of_measured_peak": per_inst * cfg.batch / (ms_med * 1e-3) / 1e9 / peaks["hbm_gbs"],
                               "dense_bytes_frac_of_measured_peak": entry["bytes_per_instance"] * cfg.batch / (ms_med * 1e-3) / 1e9 / peaks["hbm_gbs"]})
                del r
                torch.cuda.empty_cache()
        result["all_configs"] = others

        # ---- the FFMA comparison variant on the property-heavy configuration, against the FP32 FMA peak
        if args.variant == "3xtf32":
            cfg = wl.config_property_heavy()
            r = time_equation(mom, torch, cfg, mom.VARIANT_FFMA, steps=10, warmup=3, stream=stream, timing=False)
            ms_med = statistics.median(r["ms"])
            clock_mhz = result.get("clocks", {}).get("sm_max_mhz") or 1965.0
            ffma_peak = torch.cuda.get_device_properties(local).multi_processor_count * 128 * 2 * clock_mhz * 1e6 / 1e12
            tf = r["useful_flops"] / (ms_med * 1e-3) / 1e12
            result["ffma_variant"] = {"workload": cfg.name, "ms_median": ms_med, "tflops_useful": tf,
                                      "peak_tflops": ffma_peak, "peak_is": "SMs x 128 lanes x 2 x max SM clock",
                                      "frac": tf / ffma_peak, "frac_of_probe": (tf / probes["ffma_tflops"]) if isinstance(probes.get("ffma_tflops"), float) else None}
            del r
            torch.cuda.empty_cache()

        # ---- CPU baseline: the oracle on a bounded sample of the same workload
        result["cpu_baseline"], result["parity"] = cpu_baseline(eq, chain, add, useful, parity_rows, x_rows, x_off_ok)

    if rank == 0:
        print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


def launcher_command(argv, gpus: int, port: int):
    """The command that starts `gpus` ranks of this script on one node (one process per GPU)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def free_port() -> int:
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def run_check_launch(args):
    """Start-up and bookkeeping only, no GPU and no measurement: every rank joins a gloo group, plans its share of the
    headline equation (planning is host-only) and the ranks agree on the slowest rank's (made-up) time and on the summed
    work; rank 0 prints one JSON line.  This is what a machine without GPUs can check of the multi-rank path."""
    import torch.distributed as dist
    import paper_2208_10391_b200 as mom
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    variant = {"3xtf32": mom.VARIANT_3XTF32, "ffma": mom.VARIANT_FFMA}[args.variant]
    whole = headline_equation()
    whole_plan = mom.mom_equation_plan_transposed(whole.descs(), whole.chain_t, whole.add_descs(), whole.add_t, variant)
    whole_useful = sum(whole_plan.flops())
    eq, slab = whole, None
    if args.split == "columns":
        eq, b, e = column_slab_of(mom, whole, rank, world)
        slab = (b, e)
    plan = mom.mom_equation_plan_transposed(eq.descs(), eq.chain_t, eq.add_descs(), eq.add_t, variant)
    useful = sum(plan.flops())
    ms = max_over_ranks(10.0 + rank, world)                       # a made-up per-rank time: the slowest rank's counts
    total = sum_over_ranks(float(useful), world)
    value = split_job_gflops(useful, world, ms) if slab else whole_job_gflops(useful, world, ms)
    cols = sum_over_ranks(float(slab[1] - slab[0]) if slab else 0.0, world)
    if rank == 0:
        print(json.dumps({"check_launch": True, "n_gpus": world, "gpus_asked": args.gpus, "split": args.split,
                          "ms_slowest_rank": ms, "value": value, "useful_flops_all_ranks": total,
                          "useful_flops_whole_equation": whole_useful, "columns_all_ranks": cols,
                          "slab_flops_over_whole": total / whole_useful if slab else None,
                          "rank0_parenthesization": plan.parenthesization()}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def rd_cols(eq: wl.Equation) -> int:
    """Columns of the equation's result: those of its last factor as used."""
    t = list(eq.chain_t) + [False] * (len(eq.chain) - len(eq.chain_t))
    return eq.chain[-1].rows if t[-1] else eq.chain[-1].cols


def rd_elems(plan):
    d = plan.result_desc()
    return d.rows * d.cols


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=250,
                    help="timed steps of the headline equation (250 steps are about 2.3 s: long enough for the power-capped "
                         "steady state, so that the sustained measured peak is the right roofline denominator)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--variant", default="3xtf32", choices=["3xtf32", "ffma"])
    ap.add_argument("--split", default="none", choices=["none", "columns"],
                    help="columns: the ranks share ONE headline equation, each evaluating a column slab of X (strong scaling); "
                         "none: every rank evaluates its own replica (weak scaling)")
    ap.add_argument("--only", default=None, help="time just this workload (by name) and print a short JSON line")
    ap.add_argument("--check-launch", action="store_true",
                    help="start the ranks, join a gloo group, plan each rank's share and report the bookkeeping; no GPU, no timing")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not (args.impl == "reference"):
        # started as a plain script: start one rank per GPU ourselves and hand over
        cmd = launcher_command(sys.argv[1:], args.gpus, free_port())
        raise SystemExit(subprocess.call(cmd))
    if args.impl == "reference":
        run_reference(args)
    elif args.check_launch:
        run_check_launch(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
