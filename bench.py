#!/usr/bin/env python
"""Benchmark of the activation-sparse gated FFN library on B200.

One "step" is one pass of the whole hot path (gate, activation, compaction, up, scale, down,
reduction) over one batch of synthetic decode tokens: CALLS_PER_STEP single-token FFN calls, each with
its own token, rotating over several independent weight sets so that every call finds its weights in
HBM and not in L2.  The headline value is microseconds per FFN call at 90 % sparsity on the
4096 x 14336 bf16 decode shape; the line also carries the achieved HBM rate over the bytes a call
must touch, the same through the host-buffer entry point, the dense comparator, the roofline
fraction against the measured copy peak and the CPU oracle timed on this machine's host cores.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
    python bench.py --report out.json      # the wider matrix (other sparsities, LoPA, batches)
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import torch  # noqa: E402

import synthetic_inputs as syn  # noqa: E402
from bench_report import measured_hbm_peak  # noqa: E402

D_MODEL, D_FF, SPARSITY, ACT = 4096, 14336, 0.9, "relu"
CALLS_PER_STEP = 1000
WEIGHT_SETS = 4
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the main kernel at this workload: kept beside the
# ncu summary it comes from and rewritten whenever that summary is refreshed
NCU_TRAFFIC_FILE = ROOT / "profiles" / "fused_ffn_kernel_decode_4096x14336_s090.json"
WORKLOAD = "llama-style standard-gated FFN decode, d_model=4096 d_ff=14336 bf16 batch=1 RELU, sparsity 0.9"


def ncu_traffic_per_launch():
    """DRAM bytes per launch of the dominant kernel from the kept ncu summary, or None if there is none."""
    try:
        return float(json.loads(NCU_TRAFFIC_FILE.read_text())["dram_bytes_per_launch"])
    except Exception:
        return None


def extra_points(m, dev):
    """Headline points of the other configurations (LoPA gate, batched decode, the 8192 x 28672 shape), short runs
    of the measurement matrix's own routine, so that a default bench run observes them too."""
    import bench_report as rep

    D, H = D_MODEL, D_FF
    base = [syn.standard_ffn(D, H, torch.bfloat16, 2, dev, sparsity=0.9, extra=i) for i in range(WEIGHT_SETS)]
    std = lambda w: {"W_g": w["W_g"]}  # noqa: E731
    rows = []
    gi = m.g_diagonal(H, D, dev)
    lsets = []
    for i, w in enumerate(base):
        lw = syn.lopa_ffn(D, H, 512, torch.bfloat16, 3, dev, sparsity=0.9, extra=i)
        lw["W_up"], lw["W_down"] = w["W_up"], w["W_down"]
        lsets.append(lw)
    lg = lambda w: {"V": w["V"], "U": w["U"], "g_idx": gi, "use_rmsnorm": True, "rms_eps": 1e-5}  # noqa: E731
    rows.append(rep.measure("lopa r=512 relu", D, H, 1, lsets, lg, "relu", r=512, n_calls=120))
    del lsets
    p = syn.zipf_firing_profile(H, 1.1, 0.1, 0.99, seed=4)
    zb = syn.bias_from_firing_profile(p).to(dev)
    rows.append(rep.measure("batched zipf B=16", D, H, 16, [dict(w, b_g=zb) for w in base], std, "relu", n_calls=80))
    del base
    torch.cuda.empty_cache()
    D, H = 8192, 28672
    layers = [syn.standard_ffn(D, H, torch.bfloat16, 5, dev, sparsity=0.9, extra=i) for i in range(4)]
    rows.append(rep.measure("stress 8192x28672 s=0.9 B=1", D, H, 1, layers, std, "sqrelu", n_calls=48))
    keep = ("name", "B", "fired_rows", "us_per_call", "touched_mb", "gbs", "frac_measured_peak", "dense_us",
            "speedup_vs_dense", "dense_library_us", "speedup_vs_best_dense", "device_status")
    return [{k: r[k] for k in keep} for r in rows]


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 6 and r[2 + i].lower() == "active" for r in self.rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def dist_setup(n_gpus: int, backend: str = "nccl"):
    """One process per GPU under torchrun; rank 0 alone when launched plainly.  `backend` is "nccl" on
    GPUs and "gloo" in the CPU tests of this plumbing."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist

        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if backend == "nccl":
            torch.cuda.set_device(local)
            dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
        else:
            dist.init_process_group(backend)
    return rank, world, local


def max_over_ranks(ms: float, world: int, dev) -> float:
    """Slowest rank's time: the job is as fast as its slowest replica."""
    if world == 1:
        return ms
    import torch.distributed as dist

    t = torch.tensor([ms], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier(world: int, cuda: bool = True):
    if world > 1:
        import torch.distributed as dist

        dist.barrier()
    if cuda:
        torch.cuda.synchronize()


def whole_job_us_per_call(ms_max: float, steps: int, calls_per_step: int, world: int) -> float:
    """Microseconds per FFN call of the whole job: `world` replicas each made steps * calls_per_step
    calls in ms_max milliseconds (weak scaling, no data-path collective)."""
    return ms_max * 1e3 / (steps * calls_per_step * world)


class Workload:
    """Config 2 decode point: WEIGHT_SETS independent standard-gated FFNs and CALLS_PER_STEP tokens."""

    def __init__(self, m, dev, seed=2, sparsity=SPARSITY, sets=WEIGHT_SETS, tokens=CALLS_PER_STEP):
        self.m, self.dev = m, dev
        self.sets = [syn.standard_ffn(D_MODEL, D_FF, torch.bfloat16, seed, dev, sparsity=sparsity, extra=i)
                     for i in range(sets)]
        self.gates = [{"W_g": w["W_g"]} for w in self.sets]
        self.x = syn.tokens(tokens, D_MODEL, torch.bfloat16, seed, dev)
        self.y = torch.empty((tokens, D_MODEL), dtype=torch.float32, device=dev)
        self.ffn = m.SparseFFN(D_MODEL, D_FF, torch.bfloat16, B_max=1, device=dev)
        self.x_host = self.x.cpu().pin_memory()
        self.y_host = torch.empty((tokens, D_MODEL), dtype=torch.float32).pin_memory()
        self.n_act = None

    def prepare(self, stream):
        """Marshal every call of a step once: sparse, dense comparator and host-buffer variants."""
        self.calls = {"sparse": [], "dense": [], "host": []}
        for t in range(self.x.shape[0]):
            w, g = self.sets[t % len(self.sets)], self.gates[t % len(self.sets)]
            a = (g, w["b_g"], w["W_up"], w["W_down"], ACT)
            self.calls["sparse"].append(self.ffn.prepared(self.x[t], *a, self.y[t], stream=stream))
            self.calls["dense"].append(self.ffn.prepared(self.x[t], *a, self.y[t], dense=True, stream=stream))
            self.calls["host"].append(self.ffn.prepared(self.x_host[t], *a, self.y_host[t], host=True, stream=stream))

    def step(self, kind="sparse"):
        for c in self.calls[kind]:
            c()

    def count_active(self):
        """Fired neurons per token (outside any timed region): sets the algorithmic byte count."""
        n = []
        for t in range(self.x.shape[0]):
            w = self.sets[t % len(self.sets)]
            self.ffn.sparse_ffn_forward(self.x[t], self.gates[t % len(self.sets)], w["b_g"], w["W_up"], w["W_down"],
                                        ACT, self.y[t])
            n.append(int(self.ffn.last_active().numel()))
        self.n_act = n
        return n


def time_steps(fn, steps, warmup, world, dev, stream):
    """Device time of `steps` calls of fn, CUDA events on the launching stream, max over ranks."""
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            fn()
        barrier(world)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        barrier(world)
    return max_over_ranks(e0.elapsed_time(e1), world, dev)


def cpu_baseline(sample_tokens=96, sparsity=SPARSITY, seed=2):
    """The CPU oracle as it stands (plain C++, double accumulation), sparse route, on a bounded sample
    of the same workload: `sample_tokens` tokens against one weight set, OpenMP over tokens."""
    import oracle

    cores = os.cpu_count() or 1
    w = syn.standard_ffn(D_MODEL, D_FF, torch.bfloat16, seed, "cpu", sparsity=sparsity)
    x = syn.tokens(sample_tokens, D_MODEL, torch.bfloat16, seed, "cpu")
    oracle.ffn(x[:1], w["W_up"], w["W_down"], ACT, W_g=w["W_g"], b_g=w["b_g"])  # load + warm
    t0 = time.perf_counter()
    oracle.ffn(x, w["W_up"], w["W_down"], ACT, W_g=w["W_g"], b_g=w["b_g"], route="sparse", threads=cores)
    dt = time.perf_counter() - t0
    # one thread, sparse and dense route, on a few tokens: what one host core does per call
    n1 = min(4, sample_tokens)
    t1 = time.perf_counter()
    oracle.ffn(x[:n1], w["W_up"], w["W_down"], ACT, W_g=w["W_g"], b_g=w["b_g"], route="sparse", threads=1)
    t2 = time.perf_counter()
    oracle.ffn(x[:n1], w["W_up"], w["W_down"], ACT, W_g=w["W_g"], b_g=w["b_g"], route="dense", threads=1)
    t3 = time.perf_counter()
    return {"value": dt / sample_tokens * 1e6, "unit": "us/FFN-call", "cores": min(cores, sample_tokens),
            "kind": "oracle", "sample": f"{sample_tokens} tokens of the same workload, one weight set, sparse route, "
                                        f"OpenMP over tokens ({dt:.1f} s wall)",
            "single_thread_us": {"sparse": (t2 - t1) / n1 * 1e6, "dense": (t3 - t2) / n1 * 1e6, "tokens": n1}}


def run_reference(args, rank):
    if rank != 0:
        return
    sample = 48
    base = None
    for _ in range(args.warmup):
        cpu_baseline(8)
    vals = []
    for _ in range(args.steps):
        base = cpu_baseline(sample)
        vals.append(base["value"])
    v = statistics.mean(vals)
    base["value"] = v
    print(json.dumps({
        "impl": "reference", "metric": "us_per_ffn_call", "value": v, "unit": "us/FFN-call", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": v * sample / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "step": f"{sample} FFN calls on the host cores (bounded sample)"},
        "cpu_baseline": base, "gpu_launches": 0,
        "e2e": {"value": v, "unit": "us/FFN-call", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def run_ours(args, rank, world, local):
    import paper_2609_31975_b200 as m

    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)
    wl = Workload(m, dev, tokens=args.calls)
    wl.ffn.set_gate_engine(args.engine)
    n_act = wl.count_active()
    mean_rows = statistics.mean(n_act)
    bytes_per_call = statistics.mean(m.touched_bytes(D_MODEL, D_FF, n, 2) for n in n_act)
    dense_bytes = m.dense_bytes(D_MODEL, D_FF, 2)

    stream = torch.cuda.Stream(dev)
    wl.prepare(stream)
    l0 = wl.ffn.launch_count()
    with ClockSampler(local) as clk:
        ms = time_steps(wl.step, args.steps, args.warmup, world, dev, stream)
    launches = (wl.ffn.launch_count() - l0) * args.steps // (args.steps + args.warmup)
    calls = args.steps * args.calls
    us_call = ms * 1e3 / calls
    assert abs(us_call / world - whole_job_us_per_call(ms, args.steps, args.calls, world)) < 1e-9
    if args.skip_extras:
        if rank == 0:
            print(json.dumps({"metric": "us_per_ffn_call", "value": us_call / world, "unit": "us/FFN-call",
                              "note": "sparse path only (profiling run, not a bench line)"}))
        return
    dsteps = max(1, args.steps // 2)
    ms_dense = time_steps(lambda: wl.step("dense"), dsteps, 1, world, dev, stream)
    us_dense = ms_dense * 1e3 / (dsteps * args.calls)
    ms_e2e = time_steps(lambda: wl.step("host"), args.steps, 1, world, dev, stream)
    us_e2e = ms_e2e * 1e3 / calls
    status = wl.ffn.device_status()
    if status != 0:
        raise RuntimeError(f"device status {status} after the timed region")
    if rank != 0:
        return
    peak, peak_kind = measured_hbm_peak()
    achieved = bytes_per_call / (us_call * 1e-6) / 1e9
    line = {
        "metric": "us_per_ffn_call", "value": us_call / world, "unit": "us/FFN-call", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "step": f"{args.calls} single-token FFN calls, one token each",
                   "l2": f"rotating over {WEIGHT_SETS} independent weight sets ({WEIGHT_SETS * dense_bytes / 1e9:.2f} GB) "
                         "so inputs exceed L2", "storage": "bf16 weights and tokens, fp32 accumulation and output",
                   "measured_sparsity": 1.0 - mean_rows / D_FF, "gate_engine": args.engine, "parallelism": f"{world} independent replicas"},
        "tokens_per_s": world * 1e6 / us_call,
        "touched_bytes_per_call": bytes_per_call,
        "achieved_gbs": achieved, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
        "dense_us_per_call": us_dense, "dense_gbs": dense_bytes / (us_dense * 1e-6) / 1e9,
        "speedup_vs_dense": us_dense / us_call,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"{peak_kind} copy bandwidth", "traffic": ncu_traffic_per_launch(),
                     "algorithmic_bytes_per_launch": bytes_per_call,
                     "kernel": "fused_ffn_kernel (one launch per FFN call: gate stream on the CUDA cores, rows of fired "
                               "neurons, cross-CTA sum in the first CTAs to finish)"},
        "e2e": {"value": us_e2e / world, "unit": "us/FFN-call", "h2d_bytes_per_step": args.calls * D_MODEL * 2,
                "d2h_bytes_per_step": args.calls * D_MODEL * 4},
        "gpu_launches": launches, "clocks": clk.summary(),
        "cpu_baseline": cpu_baseline() if world == 1 else None,
        "extra": extra_points(m, dev) if world == 1 and not args.no_extra else None,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--report", default=None, help="write the wider measurement matrix to this JSON file")
    ap.add_argument("--quick", action="store_true", help="with --report: one point per family")
    ap.add_argument("--only", default=None, help="with --report: only the cases whose name contains this")
    ap.add_argument("--report-calls", type=int, default=None, help="with --report: calls per case")
    ap.add_argument("--calls", type=int, default=CALLS_PER_STEP, help="FFN calls (tokens) per step")
    ap.add_argument("--engine", default="auto", choices=["auto", "cuda_core", "tensor_core"],
                    help="gate engine of the single-token calls (the handle's default is auto)")
    ap.add_argument("--no-extra", action="store_true", help="leave out the other configurations' headline points")
    ap.add_argument("--skip-extras", action="store_true",
                    help="time the sparse path only (no dense comparator, host-buffer or CPU legs): for profiler runs")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank, world, local = dist_setup(args.gpus)
    try:
        if args.impl == "reference":
            run_reference(args, rank)
        elif args.report:
            import bench_report as report

            if rank == 0:
                report.run(args.report, quick=args.quick, only=args.only, n_calls=args.report_calls)
        else:
            run_ours(args, rank, world, local)
    finally:
        if world > 1:
            import torch.distributed as dist

            if dist.is_initialized():
                dist.destroy_process_group()


if __name__ == "__main__":
    main()
