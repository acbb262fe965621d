#!/usr/bin/env python
"""RegTop-k step benchmark: one step = regtopk_worker_step (all N workers) + regtopk_aggregate.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet18] [--sparsity-index 0]
    python bench.py --impl reference ...      # times the CPU oracle on a bounded sample instead

Prints ONE JSON line.  `value` is G coords/s (N*d coordinates per step, all replicas) with the
gradients already resident in HBM; `e2e` is the same metric through regtopk_round_host with pinned
host buffers (H2D of the gradients and D2H of the pairs and of g inside the timed region).
The path does not shard (one GPU by design): --gpus N runs N independent replicas.
"""
import argparse
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

# dram__bytes_read.sum + dram__bytes_write.sum of one k_stream launch from the ncu capture summarised in
# profiles/k_stream_resnet18_fp32_full.md; valid for that workload and the kernel as captured.
NCU_STREAM_TRAFFIC = {"resnet18": 1027.1e6}

METRIC = "RegTop-k step throughput (G coords/s, all N workers) and achieved HBM GB/s vs peak"
UNIT = "G coords/s"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18", choices=["resnet18", "resnet50", "gpt2", "flat1p3b"])
    ap.add_argument("--sparsity-index", type=int, default=0)
    ap.add_argument("--ring", type=int, default=0, help="distinct gradient batches kept in HBM (0 = the workload's step count, capped by memory)")
    ap.add_argument("--e2e-steps", type=int, default=8)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--seed", type=int, default=0)
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


def run_reference(args, rank, world):
    """The CPU oracle, as it stands, on a bounded sample of the workload (rank 0 only)."""
    if rank != 0:
        return
    import numpy as np
    import torch
    from paper_2501_05633_b200 import synth
    from oracle.oracle import OracleRegTopK
    w = synth.workload(args.workload)
    s = w.sparsity[args.sparsity_index]
    total_steps = args.steps + args.warmup
    budget = min(4.0, 150.0 / max(1, total_steps))  # seconds of oracle work per step
    # calibrate the oracle's rate on a small slice
    dcal = 200_000
    wc = synth.workload(args.workload, scale_to=dcal)
    gs = synth.GradientStream(wc, device="cpu", seed=args.seed)
    o = OracleRegTopK(wc.d, 1, max(1, int(s * wc.d + 0.5)), w.mu)
    g = gs.next()[:1]
    from oracle.oracle import grads_view as to_oracle_view
    t0 = time.perf_counter()
    o.worker_step(to_oracle_view(g, wc.d)); o.aggregate()
    rate = wc.d / (time.perf_counter() - t0)
    ds = int(min(w.d, max(50_000, rate * budget * 0.8)))
    workers = 1
    if ds == w.d:
        workers = int(max(1, min(w.N, budget * rate / w.d)))
    ws_ = synth.workload(args.workload, scale_to=ds) if ds < w.d else w
    k = max(1, int(s * ws_.d + 0.5))
    ws_.N = workers
    stream = synth.GradientStream(ws_, device="cpu", seed=args.seed)
    ring = [to_oracle_view(stream.next(), ws_.d) for _ in range(min(4, ws_.steps))]
    ora = OracleRegTopK(ws_.d, workers, k, w.mu)
    for i in range(args.warmup):
        ora.worker_step(ring[i % len(ring)]); ora.aggregate()
    t0 = time.perf_counter()
    for i in range(args.steps):
        ora.worker_step(ring[i % len(ring)]); ora.aggregate()
    el = time.perf_counter() - t0
    val = workers * ws_.d * args.steps / el / 1e9
    sample = f"{workers} of {w.N} workers x first-scaled {ws_.d} of {w.d} coordinates per step, k={k}, full sort per worker"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": el / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_label(w, int(s * w.d + 0.5), s), "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def cpu_baseline(w, k, seed):
    """One round (round 1, after a round 0 that sets the state) of the full workload on the oracle."""
    import torch
    from paper_2501_05633_b200 import synth
    from oracle.oracle import OracleRegTopK
    from oracle.oracle import grads_view as to_oracle_view
    nw = min(w.N, 8)  # bounded: a full sort of d entries per worker costs about a second per 10M
    wsamp = synth.workload(w.name)
    wsamp.N = nw
    stream = synth.GradientStream(wsamp, device="cuda", seed=seed)
    ora = OracleRegTopK(w.d, nw, k, w.mu)
    g0 = to_oracle_view(stream.next().cpu(), w.d)
    g1 = to_oracle_view(stream.next().cpu(), w.d)
    ora.worker_step(g0); ora.aggregate()
    t0 = time.perf_counter()
    ora.worker_step(g1); ora.aggregate()
    el = time.perf_counter() - t0
    out = {"value": nw * w.d / el / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"one round (round 1) of {nw} of the {w.N} workers at full d={w.d}, k={k}, {el:.1f} s"}
    # second figure: the same oracle with its workers (they are independent) spread over the host's cores
    cores = min(nw, os.cpu_count() or 1)
    if cores > 1 and el < 60.0:
        par = OracleRegTopK(w.d, nw, k, w.mu, threads=cores)
        par.worker_step(g0); par.aggregate()
        t0 = time.perf_counter()
        par.worker_step(g1); par.aggregate()
        el2 = time.perf_counter() - t0
        out["workers_in_parallel"] = {"value": nw * w.d / el2 / 1e9, "unit": UNIT, "cores": cores}
    return out


def main():
    args = parse()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    import torch
    import torch.distributed as dist
    import paper_2501_05633_b200 as pkg
    from paper_2501_05633_b200 import synth, binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    pkg.build()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    w = synth.workload(args.workload)
    k = w.k_values()[args.sparsity_index]
    bpe = 2 if w.grad_dtype == "bf16" else 4
    tdt = torch.bfloat16 if w.grad_dtype == "bf16" else torch.float32
    stream = synth.GradientStream(w, device=dev, seed=args.seed + rank, pad_to=32)
    per_batch = w.N * stream.ld * bpe
    free = torch.cuda.mem_get_info()[0]
    ring_n = args.ring or w.steps
    ring_n = int(max(2, min(ring_n, (free * 0.5) // per_batch)))
    ring = [stream.next() for _ in range(ring_n)]
    lib = pkg.RegTopK(w.d, w.N, k, mu=w.mu, grad_dtype=tdt,
                      flags=binding.FLAG_HOST_STAGING if args.e2e_steps > 0 else 0)
    out_idx = torch.empty((w.N, k), dtype=torch.int32, device=dev)
    out_val = torch.empty((w.N, k), dtype=torch.float32, device=dev)

    inplace = args.api == "inplace"
    acc = lib.accumulator() if inplace else None

    def step(i):
        if inplace:
            acc.add_(ring[i % ring_n][:, : w.d])  # stands in for a backward pass that accumulates
            lib.worker_step_inplace(out_idx, out_val)
        else:
            lib.worker_step(ring[i % ring_n], out_idx, out_val)
        lib.aggregate()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        step(i)
    lib.status()
    # ---- timed region: device-resident inputs ----
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    l0 = lib.stats()["kernel_launches"]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for i in range(args.steps):
        step(args.warmup + i)
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    st = lib.stats()
    launches = st["kernel_launches"] - l0
    lib.status()
    # ---- same steps again with an event pair around the streaming kernel (roofline of the dominant kernel) ----
    lib.profile_enable(True)
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    nprof = min(args.steps, 1000)
    torch.cuda.synchronize()
    p0.record()
    for i in range(nprof):
        step(args.warmup + args.steps + i)
    p1.record()
    torch.cuda.synchronize()
    ms_prof = p0.elapsed_time(p1)
    kern_ms, calls = lib.profile_read()
    lib.profile_enable(False)
    lib_only_ms = None
    if inplace:  # the library's calls alone, one event pair per step
        nlib = min(args.steps, 200)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(nlib)]
        for i, (a0, a1) in enumerate(evs):
            acc.add_(ring[i % ring_n][:, : w.d])
            a0.record()
            lib.worker_step_inplace(out_idx, out_val)
            lib.aggregate()
            a1.record()
        torch.cuda.synchronize()
        lib_only_ms = sum(a0.elapsed_time(a1) for a0, a1 in evs) / nlib
    # ---- round 0 (no previous support: Algorithm 1) on its own ----
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
    # ---- end to end through host buffers ----
    e2e_s = float("nan")
    if args.e2e_steps > 0 and not inplace:
        h_g = [ring[i].cpu().pin_memory() for i in range(min(2, ring_n))]
        h_idx = torch.empty((w.N, k), dtype=torch.int32).pin_memory()
        h_val = torch.empty((w.N, k), dtype=torch.float32).pin_memory()
        h_agg = torch.empty(w.d, dtype=torch.float32).pin_memory()
        for i in range(2):
            lib.round_host(h_g[i % len(h_g)], h_idx, h_val, h_agg)
        barrier()
        t0 = time.perf_counter()
        for i in range(args.e2e_steps):
            lib.round_host(h_g[i % len(h_g)], h_idx, h_val, h_agg)  # synchronises each step
        barrier()
        e2e_s = time.perf_counter() - t0
    lib.status()
    stats_end = lib.stats()

    ms_all, e2e_all = max_over_ranks([ms, e2e_s], dev, world)
    if rank == 0:
        coords = w.N * w.d
        value = world * coords * args.steps / (ms_all * 1e-3) / 1e9
        peak, peak_kind = measured_peak()
        alg_bytes = coords * (bpe + 8)
        kern_alg_bytes = coords * 4 if inplace else alg_bytes  # in place, the library only reads the rows
        kern_avg_ms = kern_ms / max(1, calls)
        achieved = kern_alg_bytes / (kern_avg_ms * 1e-3) / 1e9
        step_gbs = alg_bytes / (ms_all / args.steps * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_all / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_label(w, k, w.sparsity[args.sparsity_index]),
                       "replicas": world, "parallelism": "replicas only (the path runs on one GPU)",
                       "l2": f"inputs larger than L2 ({per_batch / 1e6:.0f} MB per step, ring of {ring_n} batches)",
                       "step_hbm_gbs": step_gbs, "step_frac_of_measured_peak": step_gbs / peak,
                       "step_frac_of_8TBs": step_gbs / 8000.0,
                       "dense_select_workers": stats_end["dense_select_workers"],
                       "candidates_last": stats_end["candidates_last"],
                       "ms_per_step_with_kernel_events": ms_prof / nprof,
                       "round0_ms": round0_ms},
            "clocks": clocks,
            "e2e": {"value": (world * coords * args.e2e_steps / e2e_all / 1e9) if (args.e2e_steps > 0 and not inplace) else None, "unit": UNIT,
                    "h2d_bytes_per_step": w.N * stream.ld * bpe, "d2h_bytes_per_step": 2 * w.N * k * 4 + w.d * 4},
            "gpu_launches": launches,
            "roofline": {"bound": "hbm", "kernel": "k_stream", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                         "traffic": NCU_STREAM_TRAFFIC.get(w.name) if w.grad_dtype == "f32" else None,
                         "algorithmic_bytes_per_launch": kern_alg_bytes, "avg_launch_ms": kern_avg_ms},
        }
        if inplace:
            line["config"]["api"] = ("accumulate in place: ms_per_step includes the caller's torch add_ of the gradients "
                                     "into the library's rows; ms_library_only is worker_step_inplace + aggregate alone")
            line["config"]["ms_library_only"] = lib_only_ms
        if world == 1 and not args.no_cpu_baseline:
            del ring
            torch.cuda.empty_cache()
            line["cpu_baseline"] = cpu_baseline(w, k, args.seed)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
