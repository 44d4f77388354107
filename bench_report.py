"""Wider measurement matrix behind `bench.py --report`: the sparsity sweep of the decode shape, the LoPA
gates, batched decode under Zipf firing and the 8192 x 28672 stress shape.  Every row times K back-to-back
calls with CUDA events on the launching stream, rotating over enough independent weight sets that the
weights of a call are never L2-resident, and reports microseconds per call, the bytes the call must touch
(from the measured number of fired rows) and the achieved rate."""
from __future__ import annotations

import json
import math
import statistics
import sys
from pathlib import Path

import torch

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import synthetic_inputs as syn  # noqa: E402
from paper_2609_31975_b200 import SparseFFN, g_diagonal, touched_bytes, dense_bytes  # noqa: E402

DEV = "cuda:0"
NOMINAL = 8000.0
FALLBACK_HBM_GBS = 6650.0  # an earlier copy measurement on this machine, used only when MEASURED_PEAKS.json is absent


def measured_hbm_peak():
    """(GB/s, "measured" | "fallback"): the copy bandwidth every roofline fraction is quoted against."""
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def _time(calls, stream, reps=3):
    with torch.cuda.stream(stream):
        for c in calls[: min(len(calls), 16)]:
            c()
        torch.cuda.synchronize()
        best = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for c in calls:
                c()
            e1.record(stream)
            torch.cuda.synchronize()
            best.append(e0.elapsed_time(e1) * 1e3 / len(calls))
    return statistics.median(best), min(best)


def _call_intervals(calls, stream):
    """Spacing of consecutive calls with an event recorded after every call: median and 95th percentile in
    microseconds.  The event records keep consecutive calls from overlapping (no dependent-launch overlap across an
    event), so these intervals are those of isolated calls, longer than the back-to-back figure."""
    with torch.cuda.stream(stream):
        for c in calls[: min(len(calls), 16)]:
            c()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(len(calls) + 1)]
        ev[0].record(stream)
        for i, c in enumerate(calls):
            c()
            ev[i + 1].record(stream)
        torch.cuda.synchronize()
    d = sorted(ev[i].elapsed_time(ev[i + 1]) * 1e3 for i in range(len(calls)))
    return d[len(d) // 2], d[min(len(d) - 1, int(0.95 * len(d)))]


def _time_graph(calls, stream, replays=5):
    """The same sequence of calls captured once in a CUDA graph and replayed: no host work between the calls."""
    with torch.cuda.stream(stream):
        for c in calls[: min(len(calls), 16)]:
            c()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for c in calls:
                c()
        graph.replay()
        stream.synchronize()
        times = []
        for _ in range(replays):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            graph.replay()
            e1.record(stream)
            e1.synchronize()
            times.append(e0.elapsed_time(e1) * 1e3 / len(calls))
        del graph
    return statistics.median(times), min(times)


def _is_q8(w):
    """0 for fp32 / bf16 weights, 8 for int8 codes, 4 for packed 4-bit codes."""
    if not isinstance(w["W_up"], dict):
        return 0
    return 4 if w["W_up"]["q"].dtype == torch.uint8 else 8


def _library_dense_calls(sets, x, act, n):
    """A second dense comparator: the same FFN as three library matrix products (cuBLAS through torch, bf16 in and out)
    and two elementwise kernels per call, outputs preallocated.  Only its time is used; standard gate on bf16 weights."""
    H, D = sets[0]["W_up"].shape
    B = 1 if x.dim() == 2 else x.shape[1]
    z = torch.empty((B, H), dtype=torch.bfloat16, device=DEV)
    u = torch.empty((B, H), dtype=torch.bfloat16, device=DEV)
    yb = torch.empty((B, D), dtype=torch.bfloat16, device=DEV)
    biases = [w["b_g"].to(torch.bfloat16) for w in sets]
    fn = {"relu": torch.relu_, "sqrelu": lambda t: torch.relu_(t).square_(), "rsplus": torch.nn.functional.silu}[act]

    def one(t):
        w, b = sets[t % len(sets)], biases[t % len(sets)]
        xt = x[t].view(B, D)

        def call():
            torch.addmm(b, xt, w["W_g"].t(), out=z)
            fn(z)
            torch.matmul(xt, w["W_up"].t(), out=u)
            z.mul_(u)
            torch.matmul(z, w["W_down"], out=yb)
        return call
    return [one(t) for t in range(n)]


def _bytes(D, H, n_rows, esz, B, r, q8):
    """Algorithmic bytes of one call; int8 weights: one byte per weight, bf16 tokens, and the fp32 row scales of
    the gate matrix and of the fired W_up / W_down rows."""
    if not q8:
        return touched_bytes(D, H, n_rows, esz, B, r)
    if q8 == 4:  # 4-bit codes: half a byte per weight
        weights = touched_bytes(D, H, n_rows, 1, 0, r) - H * 4
        return weights // 2 + H * 4 + B * D * 2 + B * D * 4 + 4 * (H + 2 * n_rows + (r or 0))
    return touched_bytes(D, H, n_rows, 1, B, r) + B * D + 4 * (H + 2 * n_rows + (r or 0))


def measure(name, D, H, B, sets, gate_of, act, r=None, n_calls=200, peak=None, act_up=None, graph=False):
    """sets: list of weight dicts; gate_of(w) -> gate dict; act_up: activation on the up projection (double
    activation) or None.  Returns one result row."""
    peak = peak or measured_hbm_peak()[0]
    ffn = SparseFFN(D, H, torch.bfloat16, r_max=r or 0, B_max=B, device=DEV)
    ffn.set_up_activation(act_up)
    stream = torch.cuda.Stream(DEV)
    x = syn.tokens(n_calls * B, D, torch.bfloat16, 99, DEV).view(n_calls, B, D)
    y = torch.empty((n_calls, B, D), dtype=torch.float32, device=DEV)
    rows, sparse_calls, dense_calls = [], [], []
    for t in range(n_calls):
        w = sets[t % len(sets)]
        xt = x[t, 0] if B == 1 else x[t]
        yt = y[t, 0] if B == 1 else y[t]
        if t < 24:  # fired rows per call (union for B > 1), outside the timed region
            fwd = {0: ffn.sparse_ffn_forward, 8: ffn.sparse_ffn_forward_q8, 4: ffn.sparse_ffn_forward_q4}[_is_q8(w)]
            fwd(xt, gate_of(w), w["b_g"], w["W_up"], w["W_down"], act, yt)
            rows.append(int(ffn.last_active().numel()))
        sparse_calls.append(ffn.prepared(xt, gate_of(w), w["b_g"], w["W_up"], w["W_down"], act, yt, stream=stream))
        dense_calls.append(ffn.prepared(xt, gate_of(w), w["b_g"], w["W_up"], w["W_down"], act, yt, dense=True,
                                        stream=stream))
    n_rows = statistics.mean(rows)
    us, us_min = _time_graph(sparse_calls, stream) if graph else _time(sparse_calls, stream)
    us_dense, _ = _time(dense_calls[: max(16, n_calls // 4)], stream, reps=2)
    iv_med, iv_p95 = _call_intervals(sparse_calls, stream)
    us_lib = None
    if not _is_q8(sets[0]) and "W_g" in gate_of(sets[0]):
        us_lib, _ = _time(_library_dense_calls(sets, x, act, max(16, n_calls // 4)), stream, reps=2)
    status = ffn.device_status()
    q8 = _is_q8(sets[0])
    nbytes = _bytes(D, H, round(n_rows), 2, B, r, q8)
    row = dict(name=name, D=D, H=H, B=B, r=r, act=act, fired_rows=n_rows, fired_frac=n_rows / H,
               us_per_call=us, us_min=us_min, us_interval_median=iv_med, us_interval_p95=iv_p95,
               tokens_per_s=B * 1e6 / us, touched_mb=nbytes / 1e6,
               gbs=nbytes / us / 1e3, frac_measured_peak=nbytes / us / 1e3 / peak,
               frac_nominal=nbytes / us / 1e3 / NOMINAL, dense_us=us_dense,
               dense_gbs=_bytes(D, H, H, 2, B, r, q8) / us_dense / 1e3, speedup_vs_dense=us_dense / us,
               dense_library_us=us_lib, speedup_vs_best_dense=min(us_dense, us_lib or us_dense) / us,
               device_status=status)
    del ffn, sparse_calls, dense_calls
    torch.cuda.empty_cache()
    return row


def measure_chain(name, D, H, layers, gate_of, act, r=None, dtype=torch.bfloat16, replays=20, peak=None):
    """One token through ``len(layers)`` dependent FFN layers (x_{l+1} = dtype(x_pre[l+1] + 0 * y_l): a true
    dependency with fresh N(0,1) inputs, so the sparsity of every layer stays calibrated), captured once in a
    CUDA graph and replayed.  Returns microseconds per layer for the sparse and the dense route."""
    from paper_2609_31975_b200 import residual_cast
    peak = peak or measured_hbm_peak()[0]
    L = len(layers)
    ffn = SparseFFN(D, H, dtype, r_max=r or 0, B_max=1, device=DEV)
    stream = torch.cuda.Stream(DEV)
    x_pre = syn.tokens(L + 1, D, dtype, 77, DEV)
    xs = torch.empty((L + 1, D), dtype=dtype, device=DEV)
    ys = torch.empty((L, D), dtype=torch.float32, device=DEV)
    out = {}
    esz = 2 if dtype == torch.bfloat16 else 4
    q8 = _is_q8(layers[0])
    sparse_fwd = ffn.sparse_ffn_forward_q8 if q8 else ffn.sparse_ffn_forward
    dense_fwd = ffn.dense_ffn_forward_q8 if q8 else ffn.dense_ffn_forward
    for route in ("sparse", "dense"):
        def body():
            xs[0].copy_(x_pre[0])
            for l, w in enumerate(layers):
                fwd = dense_fwd if route == "dense" else sparse_fwd
                fwd(xs[l], gate_of(w), w["b_g"], w["W_up"], w["W_down"], act, ys[l], stream=stream)
                residual_cast(ys[l], x_pre[l + 1], 0.0, xs[l + 1], stream=stream)
        with torch.cuda.stream(stream):
            body()                      # warm-up outside the capture (one-time kernel attribute calls)
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                body()
            for _ in range(3):
                graph.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(replays):
                graph.replay()
            e1.record(stream)
            e1.synchronize()
        out[route] = e0.elapsed_time(e1) * 1e3 / (replays * L)
        del graph
    rows = []
    for l, w in enumerate(layers[:8]):
        sparse_fwd(xs[l], gate_of(w), w["b_g"], w["W_up"], w["W_down"], act, ys[l])
        rows.append(int(ffn.last_active().numel()))
    n_rows = statistics.mean(rows)
    status = ffn.device_status()
    nbytes = _bytes(D, H, round(n_rows), esz, 1, r, q8)
    us = out["sparse"]
    row = dict(name=name, D=D, H=H, B=1, r=r, act=act, fired_rows=n_rows, fired_frac=n_rows / H,
               us_per_call=us, us_min=us, tokens_per_s=1e6 / (us * L), touched_mb=nbytes / 1e6,
               gbs=nbytes / us / 1e3, frac_measured_peak=nbytes / us / 1e3 / peak,
               frac_nominal=nbytes / us / 1e3 / NOMINAL, dense_us=out["dense"],
               dense_gbs=_bytes(D, H, H, esz, 1, r, q8) / out["dense"] / 1e3, speedup_vs_dense=out["dense"] / us,
               device_status=status, layers=L)
    del ffn
    torch.cuda.empty_cache()
    return row


def run(out_path, quick=False, only=None, n_calls=None):
    """only: substring filter on the case names (for profiler runs); n_calls: calls per case."""
    peak = measured_hbm_peak()[0]
    rows = []

    def want(name):
        return only is None or only in name

    def add(name, *a, **k):
        if not want(name):
            return
        if n_calls:
            k["n_calls"] = n_calls
        rows.append(measure(name, *a, **k))
        print(json.dumps(rows[-1]), flush=True)

    D, H = 4096, 14336
    std = lambda w: {"W_g": w["W_g"]}
    # decode shape: sparsity sweep
    base = [syn.standard_ffn(D, H, torch.bfloat16, 2, DEV, sparsity=0.9, extra=i) for i in range(4)]
    for s in ((0.9,) if quick else (0.5, 0.7, 0.8, 0.9, 0.95)):
        b = syn.gate_bias_for_sparsity(s)
        sets = [dict(w, b_g=torch.full((H,), b, device=DEV)) for w in base]
        add(f"decode 4096x14336 s={s}", D, H, 1, sets, std, "relu", peak=peak)
        if s == 0.9:  # double activation (RELU on the up projection as well): same rows read, one more epilogue op
            add(f"decode 4096x14336 s={s} double activation", D, H, 1, sets, std, "relu", peak=peak, act_up="relu")
            # the same 200 calls captured in one CUDA graph and replayed (no host work between calls), and the warm
            # figure: one weight set only, so part of every call's bytes comes from L2 (not a roofline number)
            add(f"decode 4096x14336 s={s} (one CUDA graph of the calls)", D, H, 1, sets, std, "relu", peak=peak, graph=True)
            add(f"decode 4096x14336 s={s} warm (a single weight set, L2 hits)", D, H, 1, sets[:1], std, "relu", peak=peak)
    # batched decode under Zipf firing
    p = syn.zipf_firing_profile(H, 1.1, 0.1, 0.99, seed=4)
    zb = syn.bias_from_firing_profile(p).to(DEV)
    zsets = [dict(w, b_g=zb) for w in base]
    for B in ((16,) if quick else (4, 16, 64)):
        add(f"batched zipf B={B}", D, H, B, zsets, std, "relu", n_calls=100, peak=peak)
        if B == 16:
            add(f"batched zipf B={B} double activation", D, H, B, zsets, std, "relu", n_calls=100, peak=peak,
                act_up="relu")
    # LoPA gates (up/down weights shared with the standard sets)
    gi = g_diagonal(H, D, DEV)
    for r in ((512,) if quick else (256, 512, 1024)):
        lsets = []
        for i, w in enumerate(base):
            lw = syn.lopa_ffn(D, H, r, torch.bfloat16, 3, DEV, sparsity=0.9, extra=i)
            lw["W_up"], lw["W_down"] = w["W_up"], w["W_down"]
            lsets.append(lw)
        lg = lambda w: {"V": w["V"], "U": w["U"], "g_idx": gi, "use_rmsnorm": True, "rms_eps": 1e-5}
        for act in ("relu", "sqrelu"):
            add(f"lopa r={r} {act}", D, H, 1, lsets, lg, act, r=r, peak=peak)
        del lsets
    del base, zsets
    torch.cuda.empty_cache()
    # weight-only int8 (codes + one fp32 scale per row): the decode shape and one LoPA gate
    if only is None or "int8" in only:
        qsets = [syn.standard_ffn_q8(D, H, 6, DEV, sparsity=0.9, extra=i) for i in range(8)]
        for s in ((0.9,) if quick else (0.8, 0.9, 0.95)):
            b = syn.gate_bias_for_sparsity(s)
            sets = [dict(w, b_g=torch.full((H,), b, device=DEV)) for w in qsets]
            add(f"decode 4096x14336 s={s} int8", D, H, 1, sets, std, "relu", peak=peak)
        lsets = []
        for i, w in enumerate(qsets):
            lw = syn.lopa_ffn_q8(D, H, 512, 7, DEV, sparsity=0.9, extra=i)
            lw["W_up"], lw["W_down"] = w["W_up"], w["W_down"]
            lsets.append(lw)
        lg = lambda w: {"V": w["V"], "U": w["U"], "g_idx": gi, "use_rmsnorm": True, "rms_eps": 1e-5}
        add("lopa r=512 relu int8", D, H, 1, lsets, lg, "relu", r=512, peak=peak)
        if not quick:  # batches on the tcgen05 kernels, which expand the codes to bf16 on the way to the tensor cores
            zq = [dict(w, b_g=zb) for w in qsets]
            for B in (4, 16, 64):
                add(f"batched zipf B={B} int8", D, H, B, zq, std, "relu", n_calls=100, peak=peak)
            del zq
        del qsets, lsets
        torch.cuda.empty_cache()
    # weight-only int4 (packed 4-bit codes + one fp32 scale per row)
    if only is None or "int4" in only:
        qsets = [syn.standard_ffn_q4(D, H, 8, DEV, sparsity=0.9, extra=i) for i in range(8)]
        for s in ((0.9,) if quick else (0.8, 0.9, 0.95)):
            b = syn.gate_bias_for_sparsity(s)
            sets = [dict(w, b_g=torch.full((H,), b, device=DEV)) for w in qsets]
            add(f"decode 4096x14336 s={s} int4", D, H, 1, sets, std, "relu", peak=peak)
        if not quick:
            zq = [dict(w, b_g=zb) for w in qsets]
            for B in (4, 16, 64):
                add(f"batched zipf B={B} int4", D, H, B, zq, std, "relu", n_calls=100, peak=peak)
            del zq
        del qsets
        torch.cuda.empty_cache()
    if not quick and (only is None or "stress" in only):
        # stress shape: 8 independent layers per step
        D, H = 8192, 28672
        layers = [syn.standard_ffn(D, H, torch.bfloat16, 5, DEV, sparsity=0.9, extra=i) for i in range(8)]
        for s in (0.8, 0.9, 0.95):
            b = syn.gate_bias_for_sparsity(s)
            sets = [dict(w, b_g=torch.full((H,), b, device=DEV)) for w in layers]
            for B in (1, 8):
                add(f"stress 8192x28672 s={s} B={B}", D, H, B, sets, std, "sqrelu", n_calls=64, peak=peak)
        gi = g_diagonal(H, D, DEV)
        lsets = []
        for i, w in enumerate(layers):
            lw = {k: syn.normal_tensor(shape, std_, torch.bfloat16, 5, k, DEV, i)
                  for k, shape, std_ in (("V", (1024, D), 1 / math.sqrt(D)), ("U", (H, 1024), 1 / 32.0))}
            lw["W_up"], lw["W_down"] = w["W_up"], w["W_down"]
            lsets.append(lw)
        lg = lambda w: {"V": w["V"], "U": w["U"], "g_idx": gi, "use_rmsnorm": True, "rms_eps": 1e-5}
        for s in (0.8, 0.9, 0.95):
            b = syn.gate_bias_for_sparsity(s, math.sqrt(2.0))
            sets = [dict(w, b_g=torch.full((H,), b, device=DEV)) for w in lsets]
            for B in (1, 8):
                add(f"stress lopa r=1024 s={s} B={B}", D, H, B, sets, lg, "sqrelu", r=1024, n_calls=64, peak=peak)
    if not quick and (only is None or "paper shape" in only):
        # The paper's wall-clock shape (scaling-ladder level 13: D = 3840, H = 10240, 38 layers), one token through
        # all layers in one CUDA graph; LoPA with r = D/8 and the adaptive hidden dimension H' (Sec. 3.3).
        D, H, L = 3840, 10240, 38
        r = D // 8
        Hp = D * (3 * H - r) // (r + 2 * D)
        for dtype, tag in ((torch.bfloat16, "bf16"), (torch.float32, "fp32")):
            for s_ in (0.9,):
                layers = [syn.standard_ffn(D, H, dtype, 13, DEV, sparsity=s_, extra=i) for i in range(L)]
                name = f"paper shape 3840x10240 x{L} layers {tag} s={s_} standard (graph)"
                if want(name):
                    rows.append(measure_chain(name, D, H, layers, std, "relu", dtype=dtype, peak=peak))
                    print(json.dumps(rows[-1]), flush=True)
                del layers
                torch.cuda.empty_cache()
                gi = g_diagonal(Hp, D, DEV)
                layers = []
                for i in range(L):
                    lw = syn.lopa_ffn(D, Hp, r, dtype, 14, DEV, sparsity=s_, extra=i)
                    layers.append(lw)
                lg = lambda w: {"V": w["V"], "U": w["U"], "g_idx": gi, "use_rmsnorm": True, "rms_eps": 1e-5}
                name = f"paper shape 3840x{Hp} x{L} layers {tag} s={s_} LoPA r={r} (graph)"
                if want(name):
                    rows.append(measure_chain(name, D, Hp, layers, lg, "relu", r=r, dtype=dtype, peak=peak))
                    print(json.dumps(rows[-1]), flush=True)
                del layers
                torch.cuda.empty_cache()
        # the same two chains on int8 weights (bf16 tokens)
        layers = [syn.standard_ffn_q8(D, H, 15, DEV, sparsity=0.9, extra=i) for i in range(L)]
        name = f"paper shape 3840x10240 x{L} layers int8 s=0.9 standard (graph)"
        if want(name):
            rows.append(measure_chain(name, D, H, layers, std, "relu", peak=peak))
            print(json.dumps(rows[-1]), flush=True)
        del layers
        torch.cuda.empty_cache()
        gi = g_diagonal(Hp, D, DEV)
        layers = [syn.lopa_ffn_q8(D, Hp, r, 16, DEV, sparsity=0.9, extra=i) for i in range(L)]
        lg = lambda w: {"V": w["V"], "U": w["U"], "g_idx": gi, "use_rmsnorm": True, "rms_eps": 1e-5}
        name = f"paper shape 3840x{Hp} x{L} layers int8 s=0.9 LoPA r={r} (graph)"
        if want(name):
            rows.append(measure_chain(name, D, Hp, layers, lg, "relu", r=r, peak=peak))
            print(json.dumps(rows[-1]), flush=True)
        del layers
        torch.cuda.empty_cache()
    Path(out_path).parent.mkdir(parents=True, exist_ok=True)
    Path(out_path).write_text(json.dumps(rows, indent=1))
    md = ["| case | B | fired rows | us/call | touched MB | GB/s | % of measured peak | % of 8 TB/s | dense us | speedup | "
          "library dense us |",
          "|---|---|---|---|---|---|---|---|---|---|---|"]
    for r_ in rows:
        md.append(f"| {r_['name']} | {r_['B']} | {r_['fired_rows']:.0f} ({100 * r_['fired_frac']:.1f} %) | "
                  f"{r_['us_per_call']:.1f} | {r_['touched_mb']:.1f} | {r_['gbs']:.0f} | "
                  f"{100 * r_['frac_measured_peak']:.1f} | {100 * r_['frac_nominal']:.1f} | {r_['dense_us']:.1f} | "
                  f"{r_['speedup_vs_dense']:.2f}x | "
                  + (f"{r_['dense_library_us']:.1f} |" if r_.get("dense_library_us") else "- |"))
    Path(out_path).with_suffix(".md").write_text("\n".join(md) + "\n")
    return rows
