#!/usr/bin/env python
"""RegTop-k step benchmark: one step = regtopk_worker_step (all N workers) + regtopk_aggregate.

    python bench.py [--gpus N] [--steps K] [--warmup W]
        times the headline workload (1.3e9 coordinates, N = 4, k = 1.3e6: the largest single-GPU configuration)
        and, under config.sweep, every other benchmark variant (four model shapes x their k values, plus the
        accumulate-in-place calls), all with the gradients resident in HBM
    python bench.py --workload resnet18 --sparsity-index 0 [--api inplace]
        one variant only (what the profiler commands under profiles/ run)
    python bench.py --impl reference ...
        times the CPU oracle on a bounded sample of the headline workload instead

Prints ONE JSON line.  `value` is G coords/s (N*d coordinates per step, all replicas) with the gradients
already resident in HBM; `e2e` is the same metric through regtopk_round_host with pinned host buffers (H2D of
the gradients and D2H of the pairs and of g inside the timed region).  The path does not shard across GPUs
inside one context: --gpus N runs N independent replicas.
"""
import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "RegTop-k step throughput (G coords/s, all N workers) and achieved HBM GB/s vs peak"
UNIT = "G coords/s"
VARIANTS = [("resnet18", 0), ("resnet18", 1), ("resnet50", 0), ("gpt2", 0), ("gpt2", 1),
            ("flat1p3b", 0), ("flat1p3b", 1), ("flat1p3b", 2)]
HEADLINE = ("flat1p3b", 1)
STREAM_SECTION = ("// k_stream: a = eps + g", "// k_post: one thread-block cluster per worker")


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=["resnet18", "resnet50", "gpt2", "flat1p3b"],
                    help="time this workload only (no sweep); default: the headline workload plus the sweep")
    ap.add_argument("--sparsity-index", type=int, default=None)
    ap.add_argument("--ring", type=int, default=0, help="distinct gradient batches kept in HBM (0 = the workload's step count, capped by memory)")
    ap.add_argument("--scale-to", type=int, default=0,
                    help="with --workload: the same tensor table and value recipe scaled down to about this many "
                         "coordinates (k scales with it); what the profiler captures of the larger shapes use")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--sweep-steps", type=int, default=0, help="timed steps per sweep variant (0 = chosen per workload, about 0.3 s each)")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--select", default="global", choices=["global", "layerwise", "dense"],
                    help="layerwise: every tensor of the workload keeps its own share (one Top-k per layer); dense: the "
                         "exact full-grid selection from the rows is forced every round (the path a missed cutoff takes)")
    ap.add_argument("--parallel", default="replicas", choices=["replicas", "by-worker"],
                    help="by-worker: the workload's N workers are dealt to the ranks in contiguous blocks (N must be at least "
                         "the number of ranks), one NCCL all-gather of the k pairs of every worker per round, every rank "
                         "aggregates all N in worker order; total work is fixed as ranks are added (strong scaling)")
    ap.add_argument("--api", default="plain", choices=["plain", "inplace"],
                    help="inplace: the step is the caller's accumulate (torch add_ into the library's rows) + "
                         "regtopk_worker_step_inplace + regtopk_aggregate; the library's share is reported beside it")
    return ap.parse_args()


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def stream_section_hash():
    """SHA-256 of the streaming kernel's part of the CUDA source (from its heading comment to the next kernel's)."""
    src = open(os.path.join(ROOT, "paper_2501_05633_b200", "csrc", "regtopk.cu")).read()
    a, b = src.find(STREAM_SECTION[0]), src.find(STREAM_SECTION[1])
    if a < 0 or b < a:
        return None
    return hashlib.sha256(src[a:b].encode()).hexdigest()


def recorded_traffic(workload_name, grad_dtype, api, coords):
    """DRAM bytes of one k_stream launch over `coords` coordinates, from the profiler capture summarised under
    profiles/ (taken on the same workload scaled down where the full size is too large to capture: the kernel's
    traffic is proportional to the coordinates it streams, so the capture's bytes per coordinate are scaled up), or
    None when there is no capture for this workload or the kernel's source has changed since it was taken."""
    try:
        rec = json.load(open(os.path.join(ROOT, "profiles", "k_stream_traffic.json")))
    except Exception:
        return None
    now = stream_section_hash()
    for r in rec.get("captures", []):
        if (r.get("workload") == workload_name and r.get("grad_dtype") == grad_dtype and r.get("api", "plain") == api
                and now is not None and r.get("stream_section_sha256") == now):
            return r["dram_bytes_per_launch"] / r["coordinates_per_launch"] * coords
    return None


class ClockSampler:
    """nvidia-smi clock and throttle-reason samples while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
                for nm, v in zip(names, r[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            except Exception:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def workload_label(w, k, sparsity):
    return (f"{w.name}-shaped gradient d={w.d} N={w.N} k={k} ({sparsity:g} of d) mu={w.mu} "
            f"grads={w.grad_dtype}")


def max_over_ranks(values, device, world):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank sets the time)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


# ---- the CPU oracle on a bounded sample (the reference arm, and the cpu_baseline of the GPU arm) -------------------
def oracle_sample(name, sparsity_index, seed, steps, warmup, seconds_per_step):
    """Times the oracle, as it stands, on a sample of workload `name`: the first `ds` coordinates of the tensor table
    scaled down (same value recipe, k scaled with it) for as many of the N workers as fit `seconds_per_step`.
    Returns (G coords/s, ms per step, text describing the sample)."""
    import copy
    from paper_2501_05633_b200 import synth
    from oracle.oracle import OracleRegTopK
    from oracle.oracle import grads_view as to_oracle_view
    w = synth.workload(name)
    s = w.sparsity[sparsity_index]
    dcal = 200_000  # calibrate the oracle's rate on a small slice
    wc = synth.workload(name, scale_to=dcal)
    gs = synth.GradientStream(wc, device="cpu", seed=seed)
    o = OracleRegTopK(wc.d, 1, max(1, int(s * wc.d + 0.5)), w.mu)
    g = gs.next()[:1]
    t0 = time.perf_counter()
    o.worker_step(to_oracle_view(g, wc.d)); o.aggregate()
    rate = wc.d / (time.perf_counter() - t0)
    ds = int(min(w.d, max(50_000, rate * seconds_per_step * 0.8)))
    workers = 1
    if ds == w.d:
        workers = int(max(1, min(w.N, seconds_per_step * rate / w.d)))
    ws_ = copy.deepcopy(synth.workload(name, scale_to=ds) if ds < w.d else w)  # the label keeps the full workload's N
    k = max(1, int(s * ws_.d + 0.5))
    ws_.N = workers
    stream = synth.GradientStream(ws_, device="cpu", seed=seed)
    ring = [to_oracle_view(stream.next(), ws_.d) for _ in range(min(4, ws_.steps))]
    ora = OracleRegTopK(ws_.d, workers, k, w.mu)
    for i in range(warmup):
        ora.worker_step(ring[i % len(ring)]); ora.aggregate()
    t0 = time.perf_counter()
    for i in range(steps):
        ora.worker_step(ring[i % len(ring)]); ora.aggregate()
    el = time.perf_counter() - t0
    val = workers * ws_.d * steps / el / 1e9
    sample = (f"{workers} of {w.N} workers x {ws_.d} of {w.d} coordinates per step (tensor table scaled down, same value "
              f"recipe), k={k}, selection by full sort (std::sort) per worker, 1 thread")
    return val, el / steps * 1e3, sample


def run_reference(args, rank, world):
    """The CPU oracle, as it stands, on a bounded sample of the workload (rank 0 only)."""
    if rank != 0:
        return
    from paper_2501_05633_b200 import synth
    name, ki = (args.workload, args.sparsity_index or 0) if args.workload else HEADLINE
    w = synth.workload(name)
    s = w.sparsity[ki]
    total_steps = args.steps + args.warmup
    budget = min(4.0, 150.0 / max(1, total_steps))  # seconds of oracle work per step
    val, ms, sample = oracle_sample(name, ki, args.seed, args.steps, args.warmup, budget)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": w.grad_dtype, "data": "synthetic",
            "config": {"workload": workload_label(w, w.k_values()[ki], s), "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---- the GPU arm --------------------------------------------------------------------------------------------------
class Bench:
    """One workload's gradient ring in HBM and the timing of its variants."""

    def __init__(self, name, dev, seed, ring_arg, reserve_bytes=0, scale_to=0):
        import torch
        from paper_2501_05633_b200 import synth
        self.torch, self.dev = torch, dev
        self.w = synth.workload(name, scale_to=scale_to or None)
        self.bpe = 2 if self.w.grad_dtype == "bf16" else 4
        self.tdt = torch.bfloat16 if self.w.grad_dtype == "bf16" else torch.float32
        self.stream = synth.GradientStream(self.w, device=dev, seed=seed, pad_to=32)
        self.per_batch = self.w.N * self.stream.ld * self.bpe
        free = torch.cuda.mem_get_info()[0] - reserve_bytes
        n = ring_arg or self.w.steps
        self.ring_n = int(max(2, min(n, (free * 0.45) // self.per_batch)))
        self.ring = [self.stream.next() for _ in range(self.ring_n)]

    def close(self):
        self.ring = None
        self.torch.cuda.empty_cache()

    def layers(self, ki):
        """Every tensor of the workload as a layer that keeps the workload's share of its entries (at least one)."""
        import itertools
        frac = self.w.sparsity[ki]
        ends = list(itertools.accumulate(self.w.shapes))
        ks = [int(min(n, max(1, int(frac * n + 0.5)))) for n in self.w.shapes]
        return ends, ks

    def variant(self, ki, steps, warmup, api="plain", flags=0, per_step_events=False, sampler=None, barrier=None,
                select="global"):
        """Times `steps` rounds after `warmup` (at least 3) with CUDA events on the library's stream (torch's current
        stream); then the same rounds again with an event pair around the streaming kernel.  Returns a dict."""
        torch = self.torch
        import paper_2501_05633_b200 as pkg
        w, ring, ring_n = self.w, self.ring, self.ring_n
        k = w.k_values()[ki]
        layers = self.layers(ki) if select == "layerwise" else None
        if layers is not None:
            k = int(sum(layers[1]))
        if select == "dense":
            flags |= binding_flags("dense")
        lib = pkg.RegTopK(w.d, w.N, k, mu=w.mu, grad_dtype=self.tdt, flags=flags, layers=layers)
        out_idx = torch.empty((w.N, k), dtype=torch.int32, device=self.dev)
        out_val = torch.empty((w.N, k), dtype=torch.float32, device=self.dev)
        inplace = api == "inplace"
        acc = lib.accumulator() if inplace else None

        def step(i):
            if inplace:
                acc.add_(ring[i % ring_n][:, : w.d])  # stands in for a backward pass that accumulates
                lib.worker_step_inplace(out_idx, out_val)
            else:
                lib.worker_step(ring[i % ring_n], out_idx, out_val)
            lib.aggregate()

        sync = barrier or torch.cuda.synchronize
        warmup = max(3, warmup)
        for i in range(warmup):
            step(i)
        lib.status()
        if sampler is not None:
            sampler.start()
        l0 = lib.stats()["kernel_launches"]
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)] if per_step_events else None
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sync()
        e0.record()
        for i in range(steps):
            if marks:
                marks[i].record()
            step(warmup + i)
        if marks:
            marks[steps].record()
        e1.record()
        sync()
        ms = e0.elapsed_time(e1)
        clocks = sampler.stop() if sampler is not None else None
        st = lib.stats()
        launches = st["kernel_launches"] - l0
        lib.status()
        per_step = [marks[i].elapsed_time(marks[i + 1]) for i in range(steps)] if marks else None
        # the streaming kernel alone: an event pair around it inside the library
        lib.profile_enable(True)
        nprof = min(steps, 1000)
        torch.cuda.synchronize()
        for i in range(nprof):
            step(warmup + steps + i)
        torch.cuda.synchronize()
        kern_ms, calls = lib.profile_read()
        lib.profile_enable(False)
        lib_only_ms = None
        if inplace:  # the library's calls alone, one event pair per step
            nlib = min(steps, 200)
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(nlib)]
            for i, (a0, a1) in enumerate(evs):
                acc.add_(ring[i % ring_n][:, : w.d])
                a0.record()
                lib.worker_step_inplace(out_idx, out_val)
                lib.aggregate()
                a1.record()
            torch.cuda.synchronize()
            lib_only_ms = sum(a0.elapsed_time(a1) for a0, a1 in evs) / nlib
        lib.status()
        stats_end = lib.stats()
        coords = w.N * w.d
        alg_bytes = coords * (self.bpe + 8)
        kern_alg_bytes = coords * 4 if inplace else alg_bytes  # in place, the library only reads the rows
        kern_avg_ms = kern_ms / max(1, calls)
        return {"lib": lib, "k": k, "ms_total": ms, "steps": steps, "launches": launches, "clocks": clocks,
                "per_step": per_step, "kern_avg_ms": kern_avg_ms, "kern_alg_bytes": kern_alg_bytes,
                "alg_bytes": alg_bytes, "coords": coords, "lib_only_ms": lib_only_ms,
                "dense_select_workers": stats_end["dense_select_workers"],
                "candidates_last": stats_end["candidates_last"], "step": step}


def binding_flags(select):
    from paper_2501_05633_b200 import binding
    return (binding.FLAG_FORCE_DENSE_SELECT | binding.FLAG_GRID_DENSE_SELECT) if select == "dense" else 0


def sweep_entry(b, r, ki, api, peak, select="global"):
    w = b.w
    ms_step = r["ms_total"] / r["steps"]
    step_gbs = r["alg_bytes"] / (ms_step * 1e-3) / 1e9
    kern_gbs = r["kern_alg_bytes"] / (r["kern_avg_ms"] * 1e-3) / 1e9 if r["kern_avg_ms"] > 0 else None
    e = {"workload": workload_label(w, r["k"], w.sparsity[ki]), "api": api, "select": select, "steps": r["steps"], "ms_per_step": ms_step,
         "g_coords_per_s": r["coords"] / (ms_step * 1e-3) / 1e9, "step_hbm_gbs": step_gbs,
         "step_frac_of_8TBs": step_gbs / 8000.0, "step_frac_of_measured_peak": step_gbs / peak,
         "k_stream_ms": r["kern_avg_ms"], "k_stream_gbs": kern_gbs,
         "k_stream_frac_of_measured_peak": kern_gbs / peak if kern_gbs else None,
         "dense_select_workers": r["dense_select_workers"], "gpu_launches_per_step": r["launches"] / r["steps"]}
    if api == "inplace":
        e["ms_library_only"] = r["lib_only_ms"]
        e["note"] = ("ms_per_step includes the caller's torch add_ of the gradients into the library's rows; "
                     "ms_library_only is worker_step_inplace + aggregate alone; k_stream bytes are 4 per coordinate")
    return e


def sweep_steps(w, arg):
    if arg > 0:
        return arg
    est_ms = w.N * w.d * 12 / 5.0e9  # about 5 TB/s
    return int(max(10, min(1000, 300.0 / est_ms)))


def run_by_worker(args, rank, world, local):
    """The headline workload with its N workers spread over the ranks (paper_2501_05633_b200/sharded.py)."""
    import copy
    import torch
    import torch.distributed as dist
    import paper_2501_05633_b200 as pkg
    from paper_2501_05633_b200 import synth
    from paper_2501_05633_b200.sharded import ShardedRegTopK, worker_block
    pkg.build()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29655")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    name, ki = (args.workload, args.sparsity_index or 0) if args.workload else HEADLINE
    w = synth.workload(name)
    k = w.k_values()[ki]
    first, n_local = worker_block(w.N, rank, world)
    wl = copy.deepcopy(w)
    wl.N = n_local  # this rank generates its own block of the workers only (seeded per rank)
    tdt = torch.bfloat16 if w.grad_dtype == "bf16" else torch.float32
    stream = synth.GradientStream(wl, device=dev, seed=args.seed + 1000 * rank, pad_to=32)
    bpe = 2 if w.grad_dtype == "bf16" else 4
    per_batch = n_local * stream.ld * bpe
    ring_n = int(max(2, min(args.ring or w.steps, (torch.cuda.mem_get_info()[0] * 0.45) // per_batch)))
    ring = [stream.next() for _ in range(ring_n)]
    lib = ShardedRegTopK(w.d, w.N, k, mu=w.mu, grad_dtype=tdt)
    warmup = max(3, args.warmup)
    for i in range(warmup):
        lib.step(ring[i % ring_n])
    lib.lib.status()
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
    l0 = lib.lib.stats()["kernel_launches"]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dist.barrier(); torch.cuda.synchronize()
    e0.record()
    for i in range(args.steps):
        lib.step(ring[(warmup + i) % ring_n])
    e1.record()
    dist.barrier(); torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if sampler else None
    launches = lib.lib.stats()["kernel_launches"] - l0
    lib.lib.status()
    ms_all = max_over_ranks([ms], dev, world)[0]
    if rank == 0:
        coords = w.N * w.d
        ms_step = ms_all / args.steps
        alg_bytes = coords * (bpe + 8)
        step_gbs = alg_bytes / (ms_step * 1e-3) / 1e9
        peak, peak_kind = measured_peak()
        line = {"metric": METRIC, "value": coords * args.steps / (ms_all * 1e-3) / 1e9, "unit": UNIT, "n_gpus": world,
                "steps": args.steps, "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True,
                "scaling": "strong", "vs_baseline": None, "dtype": w.grad_dtype, "data": "synthetic",
                "config": {"workload": workload_label(w, k, w.sparsity[ki]),
                           "parallelism": f"workers sharded over {world} GPUs (blocks of {n_local} on rank 0), one NCCL "
                                          f"all-gather of {8 * w.N * k} bytes of pairs per round, every rank aggregates all {w.N}",
                           "l2": f"inputs larger than L2 ({per_batch / 1e6:.0f} MB per rank and step, ring of {ring_n} batches)",
                           "step_hbm_gbs_all_ranks": step_gbs, "step_frac_of_measured_peak_per_gpu": step_gbs / peak / world,
                           "peak_kind": f"of {peak_kind}"},
                "clocks": clocks, "gpu_launches": launches}
        print(json.dumps(line), flush=True)
    dist.destroy_process_group()


def main():
    args = parse()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.parallel == "by-worker":
        run_by_worker(args, rank, world, local)
        return
    import torch
    import torch.distributed as dist
    import paper_2501_05633_b200 as pkg
    from paper_2501_05633_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    pkg.build()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    peak, peak_kind = measured_peak()
    single = args.workload is not None
    head_name, head_ki = (args.workload, args.sparsity_index or 0) if single else HEADLINE
    do_sweep = not single and not args.no_sweep

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sweep = []
    # ---- the sweep: every other variant, device-resident, one workload's ring in HBM at a time ----
    if do_sweep:
        for name in ("resnet18", "resnet50", "gpt2", "flat1p3b"):
            b = Bench(name, dev, args.seed + rank, args.ring)
            n_steps = sweep_steps(b.w, args.sweep_steps)
            for ki in range(len(b.w.sparsity)):
                if (name, ki) == HEADLINE:
                    continue
                r = b.variant(ki, n_steps, args.warmup)
                sweep.append(sweep_entry(b, r, ki, "plain", peak))
                r["lib"].close()
                del r
                torch.cuda.empty_cache()
            if name in ("resnet18", "flat1p3b"):  # the accumulate-in-place calls on the smallest and the largest rows
                ki = 0 if name == "resnet18" else 1
                r = b.variant(ki, n_steps, args.warmup, api="inplace")
                sweep.append(sweep_entry(b, r, ki, "inplace", peak))
                r["lib"].close()
                del r
                torch.cuda.empty_cache()
            if name in ("resnet18", "gpt2"):  # layer-wise selection, and the forced dense exact path, on two shapes
                for sel in ("layerwise", "dense"):
                    r = b.variant(0, max(10, n_steps // 4), args.warmup, select=sel)
                    sweep.append(sweep_entry(b, r, 0, "plain", peak, select=sel))
                    r["lib"].close()
                    del r
                    torch.cuda.empty_cache()
            if name != head_name:
                b.close()
                del b
        head = b  # the headline workload's ring is the last one built
    else:
        head = Bench(head_name, dev, args.seed + rank, args.ring, scale_to=args.scale_to if single else 0)

    # ---- the headline: timed region with per-step events, clocks sampled meanwhile ----
    w = head.w
    sampler = ClockSampler(local) if rank == 0 else None
    flags = binding.FLAG_HOST_STAGING if (args.e2e_steps > 0 and args.api == "plain") else 0
    r = head.variant(head_ki, args.steps, args.warmup, api=args.api, flags=flags, per_step_events=True,
                     sampler=sampler, barrier=barrier, select=args.select)
    lib, k, step = r["lib"], r["k"], r["step"]
    inplace = args.api == "inplace"
    # round 0 (no previous support: Algorithm 1) on its own
    r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    round0 = []
    for _ in range(3):
        lib.state_reset()
        torch.cuda.synchronize()
        r0.record()
        step(0)
        r1.record()
        torch.cuda.synchronize()
        round0.append(r0.elapsed_time(r1))
    round0_ms = statistics.median(round0)
    # end to end through host buffers
    e2e_s = float("nan")
    if args.e2e_steps > 0 and not inplace:
        h_g = torch.empty(head.ring[0].shape, dtype=head.ring[0].dtype, pin_memory=True)
        h_g.copy_(head.ring[0])
        h_idx = torch.empty((w.N, k), dtype=torch.int32, pin_memory=True)
        h_val = torch.empty((w.N, k), dtype=torch.float32, pin_memory=True)
        h_agg = torch.empty(w.d, dtype=torch.float32, pin_memory=True)
        for i in range(2):
            lib.round_host(h_g, h_idx, h_val, h_agg)
        barrier()
        t0 = time.perf_counter()
        for i in range(args.e2e_steps):
            lib.round_host(h_g, h_idx, h_val, h_agg)  # synchronises each step
        barrier()
        e2e_s = time.perf_counter() - t0
        del h_g, h_agg
    lib.status()

    ms_all, e2e_all = max_over_ranks([r["ms_total"], e2e_s], dev, world)
    if rank == 0:
        coords = r["coords"]
        value = world * coords * args.steps / (ms_all * 1e-3) / 1e9
        ms_step = ms_all / args.steps
        step_gbs = r["alg_bytes"] / (ms_step * 1e-3) / 1e9
        achieved = r["kern_alg_bytes"] / (r["kern_avg_ms"] * 1e-3) / 1e9
        ps = sorted(r["per_step"])
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": w.grad_dtype, "data": "synthetic",
            "config": {"workload": workload_label(w, k, w.sparsity[head_ki]),
                       "select": args.select, "replicas": world, "parallelism": "replicas only (one context runs on one GPU)",
                       "l2": f"inputs larger than L2 ({head.per_batch / 1e6:.0f} MB per step, ring of {head.ring_n} batches)",
                       "step_hbm_gbs": step_gbs, "step_frac_of_measured_peak": step_gbs / peak,
                       "step_frac_of_8TBs": step_gbs / 8000.0,
                       "ms_per_step_max": ps[-1], "ms_per_step_p99": ps[min(len(ps) - 1, int(0.99 * len(ps)))],
                       "ms_per_step_median": statistics.median(ps),
                       "dense_select_workers": r["dense_select_workers"],
                       "candidates_last": r["candidates_last"],
                       "round0_ms": round0_ms},
            "clocks": r["clocks"],
            "e2e": {"value": (world * coords * args.e2e_steps / e2e_all / 1e9) if (args.e2e_steps > 0 and not inplace) else None,
                    "unit": UNIT, "h2d_bytes_per_step": w.N * head.stream.ld * head.bpe,
                    "d2h_bytes_per_step": 2 * w.N * k * 4 + w.d * 4},
            "gpu_launches": r["launches"],
            "roofline": {"bound": "hbm", "kernel": "k_stream", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                         "traffic": recorded_traffic(w.name, w.grad_dtype, args.api, coords),
                         "algorithmic_bytes_per_launch": r["kern_alg_bytes"], "avg_launch_ms": r["kern_avg_ms"]},
        }
        if inplace:
            line["config"]["api"] = ("accumulate in place: ms_per_step includes the caller's torch add_ of the gradients "
                                     "into the library's rows; ms_library_only is worker_step_inplace + aggregate alone")
            line["config"]["ms_library_only"] = r["lib_only_ms"]
        if do_sweep:
            line["config"]["sweep"] = sweep
        if world == 1 and not args.no_cpu_baseline:
            lib.close()
            head.close()
            val, ms, sample = oracle_sample(head_name, head_ki, args.seed, 1, 1, 12.0)
            line["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
