#!/usr/bin/env python
"""Benchmark of the CompAct compressed linear layer on B200.

One "step" is one pass of the whole hot path -- forward [Y|Z] = X[W|P], backward
dX = dY W^T and Gc = Z^T dY, Adam update W <- W - lr*alpha*P N, refresh -- over
every layer of the LLaMA-7B-shaped layer set (16384 tokens, hidden 4096) with
synthetic inputs.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c5|c4|c3|c2]

With --gpus N > 1 and no launcher around it, the script starts N ranks of itself
(one per GPU, torch.distributed.run on 127.0.0.1); under a launcher it reads
RANK / LOCAL_RANK / WORLD_SIZE from the environment.  Tokens shard across the
ranks and the only exchange is the all-reduce of each layer's r x m gradient.

Timing: W warm-up steps, then untimed steps until the part has been under load
for --preheat-seconds (a power-capped B200 settles to its sustained clocks in
about two seconds), then EXACTLY K timed steps between CUDA events.  The clock
samples reported are those that fall inside the timed window.

`--impl reference` times the CPU oracle (oracle/) as it stands on the host cores,
on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2410_15352_b200 import workloads as wlm  # noqa: E402

METRIC = "CompAct linear fwd+bwd+update TFLOP/s"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

WORKLOADS = {"c5": wlm.config5, "c4": wlm.config4, "c3": wlm.config3, "c2": wlm.config2}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def layer_flops(wl: wlm.Workload, tokens: int) -> float:
    return sum(wlm.algorithmic_flops(tokens, L.n, L.m, L.r) for L in wl.layers)


# ----------------------------------------------------------------------------------------
# clock sampling during the timed region
# ----------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi in a side process, one line every 10 ms with its own timestamp; stop(t0, t1) keeps the
    samples whose timestamp lies between the two wall-clock times (the timed window)."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "10"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    @staticmethod
    def _stamp(text: str):
        try:
            return datetime.datetime.strptime(text.strip(), "%Y/%m/%d %H:%M:%S.%f").timestamp()
        except ValueError:
            return None

    def stop(self, t0: float, t1: float):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "window": "timed region only"}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    rows.append((self._stamp(f[0]), float(f[1]), float(f[2]), float(f[3]),
                                 [nm for nm, v in zip(names, f[5:9]) if v.lower().startswith("active")]))
                except ValueError:
                    continue
            os.unlink(self.path)
        except Exception:
            pass
        inside = [r for r in rows if r[0] is not None and t0 <= r[0] <= t1]
        if not inside and rows:
            # the window was shorter than the sampling period: take the samples nearest to it
            mid = 0.5 * (t0 + t1)
            inside = sorted((r for r in rows if r[0] is not None), key=lambda r: abs(r[0] - mid))[:3]
            out["window"] = "nearest samples (window shorter than the sampling period)"
        if inside:
            out.update(sm_mhz=statistics.median(r[1] for r in inside), sm_max_mhz=max(r[2] for r in inside),
                       reasons=sorted({nm for r in inside for nm in r[4]}), samples=len(inside),
                       power_w_max=max(r[3] for r in inside), power_w_median=statistics.median(r[3] for r in inside))
        return out


# ----------------------------------------------------------------------------------------
# the CPU oracle leg (reported baseline; also `--impl reference`)
# ----------------------------------------------------------------------------------------
def distinct_shapes(wl: wlm.Workload):
    """[(first layer index of the shape, how many layers have it)] in layer order."""
    seen = {}
    for li, L in enumerate(wl.layers):
        key = (L.n, L.m, L.r, L.x_dist)
        if key not in seen:
            seen[key] = [li, 0]
        seen[key][1] += 1
    return [tuple(v) for v in seen.values()]


def oracle_sample(wl: wlm.Workload, sample_tokens: int, steps: int = 1):
    """fwd+bwd+update of one layer of each distinct shape of the set on `sample_tokens` tokens with the oracle as it
    stands.  The forward and the backward are proportional to the token count, the update does not depend on it,
    so the set's full-size step is extrapolated as sum_shape count * (t_update + t_tokens * tokens / sample).
    Returns a dict with the measured and the extrapolated seconds per step."""
    from oracle import compact_oracle as co
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    mode = "exact" if wl.dtype == "f32" else "bf16"
    shapes = distinct_shapes(wl)
    layers = {}
    for li, _ in shapes:
        L = wl.layers[li]
        W0 = wlm.draw_W(wl, li).to(torch.float64).numpy()
        layers[li] = co.CompActLayerOracle(W0, L.n, L.m, L.r, wl.seed, li, wl.refresh_T, wl.lr, wl.beta1, wl.beta2,
                                           wl.eps, wl.alpha, mode)
    measured, extrapolated = [], []
    scale = wl.tokens / sample_tokens
    for s in range(steps):
        t_meas = t_full = 0.0
        for li, count in shapes:
            lay = layers[li]
            X = wlm.draw_X(wl, li, s, sample_tokens).to(torch.float64).numpy()
            dY = wlm.draw_dY(wl, li, s, sample_tokens).to(torch.float64).numpy()
            t0 = time.perf_counter()
            Y, Z = lay.forward(X)
            dX, Gc = lay.backward(dY, Z)
            t1 = time.perf_counter()
            lay.update(Gc)
            t2 = time.perf_counter()
            t_meas += (t2 - t0)
            t_full += count * ((t2 - t1) + (t1 - t0) * scale)
        measured.append(t_meas)
        extrapolated.append(t_full)
    sample_flops = sum(wlm.algorithmic_flops(sample_tokens, wl.layers[li].n, wl.layers[li].m, wl.layers[li].r) for li, _ in shapes)
    names = ", ".join(f"{wl.layers[li].name} {wl.layers[li].n}x{wl.layers[li].m} r={wl.layers[li].r} (x{c})" for li, c in shapes)
    return {
        "seconds_measured": statistics.median(measured), "flops_measured": sample_flops,
        "seconds_full_step_extrapolated": statistics.median(extrapolated), "flops_full_step": layer_flops(wl, wl.tokens),
        "threads": threads,
        "sample": (f"one layer of each distinct shape [{names}] of {wl.name} at {sample_tokens} of {wl.tokens} tokens with the "
                   f"full update; whole-set step extrapolated: token-proportional time x{scale:g}, update time as measured, "
                   "times the number of layers of the shape"),
    }


def cpu_baseline_entry(r):
    return {"value": r["flops_full_step"] / r["seconds_full_step_extrapolated"] / 1e12, "unit": UNIT, "cores": r["threads"],
            "kind": "oracle", "sample": r["sample"], "extrapolated": True,
            "seconds_full_step_extrapolated": r["seconds_full_step_extrapolated"],
            "measured_on_sample": {"seconds": r["seconds_measured"], "value": r["flops_measured"] / r["seconds_measured"] / 1e12}}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = WORKLOADS[args.workload]()
    sample_tokens = min(wl.tokens, 256)
    for _ in range(min(args.warmup, 1)):
        oracle_sample(wl, sample_tokens, steps=1)
    r = oracle_sample(wl, sample_tokens, steps=max(1, args.steps))
    cpu = cpu_baseline_entry(r)
    val = cpu["value"]
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": r["seconds_full_step_extrapolated"] * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "tokens": wl.tokens, "sample": r["sample"]},
        "tokens_per_s": wl.tokens / r["seconds_full_step_extrapolated"],
        "cpu_baseline": cpu,
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------
# the CUDA path
# ----------------------------------------------------------------------------------------
class LayerBuffers:
    def __init__(self, wl, li, tokens, dev, gen):
        from paper_2410_15352_b200 import binding as cb
        L = wl.layers[li]
        dt = wlm.torch_dtype(wl.dtype)
        self.L = L
        self.lay = cb.CompactLinear(L.n, L.m, L.r, dtype=dt, seed=wl.seed, layer_id=li, refresh_T=wl.refresh_T, lr=wl.lr,
                                    beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps, alpha=wl.alpha)
        xs = (1.0 / L.n ** 0.5) if wl.x_scale_inv_sqrt_n else 1.0
        X = torch.randn((tokens, L.n), device=dev, generator=gen, dtype=torch.float32)
        if L.x_dist == "outlier":
            X[:, 37::100] *= 20.0
        elif L.x_dist == "gelu":
            X = torch.nn.functional.gelu(X)
        self.X = (X * xs).to(dt)
        del X
        dys = wl.dy_std if wl.dy_std is not None else 1.0 / L.n ** 0.5
        self.dY = (torch.randn((tokens, L.m), device=dev, generator=gen, dtype=torch.float32) * dys).to(dt)
        self.W = (torch.randn((L.n, L.m), device=dev, generator=gen, dtype=torch.float32) * 0.02).to(dt)
        self.Y = torch.empty((tokens, L.m), device=dev, dtype=dt)
        self.Z = torch.empty((tokens, self.lay.ldz), device=dev, dtype=dt)
        self.dX = torch.empty((tokens, L.n), device=dev, dtype=dt)
        self.Gc = torch.empty((L.r, L.m), device=dev, dtype=torch.float32)
        self.M = torch.zeros_like(self.Gc)
        self.V = torch.zeros_like(self.Gc)
        self.lay.workspace(tokens)


# DRAM traffic from the committed ncu captures (profiles/compact_gemm2_kernel_c5_*.md): dram__bytes_read.sum +
# dram__bytes_write.sum of all launches of one forward call (expansion of P, product), one backward call (product,
# reduction of the Gc partials) and one update call (Adam + expansion, product) of the three distinct C5 shapes,
# every launch from cold caches.  Other shapes are scaled from the q_proj figures by flops (forward, backward) and by
# algorithmic bytes (update).  The update's reduce-adds leave W dirty in the L2: its write-back happens after the
# kernel and is not in these figures.
NCU_DRAM_BYTES_PER_CALL = {
    (4096, 4096, 512): (399.6e6, 604.0e6, 67.2e6),
    (4096, 11008, 512): (1367.5e6, 2629.5e6, 212.3e6),
    (11008, 4096, 1376): (3038.0e6, 1683.9e6, 267.6e6),
}


def ncu_dram_bytes(L, tokens: int, eb: int):
    """(forward, backward, update) DRAM bytes of one layer's calls, from the captures or scaled from q_proj's."""
    key = (L.n, L.m, L.r)
    if key in NCU_DRAM_BYTES_PER_CALL and tokens == 16384:
        return NCU_DRAM_BYTES_PER_CALL[key]
    f0, b0, u0 = NCU_DRAM_BYTES_PER_CALL[(4096, 4096, 512)]
    qn, qm, qr, qt = 4096, 4096, 512, 16384
    return (f0 * (tokens * L.n * (L.m + L.r)) / (qt * qn * (qm + qr)),
            b0 * (tokens * L.m * (L.n + L.r)) / (qt * qm * (qn + qr)),
            u0 * wlm.update_bytes(L.n, L.m, L.r, eb) / wlm.update_bytes(qn, qm, qr, 2))


def must_spawn(gpus: int, environ) -> bool:
    """--gpus N > 1 with no launcher's environment around: this process starts the ranks itself."""
    return gpus > 1 and "WORLD_SIZE" not in environ


def run_ours(args):
    import torch.distributed as dist
    from paper_2410_15352_b200 import binding as cb
    from paper_2410_15352_b200 import dp
    from paper_2410_15352_b200.build import build_library

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "INFO")          # the communicator's topology lines go to stderr
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build_library()
    if world > 1:
        dist.barrier()
    cb.lib()

    wl = WORKLOADS[args.workload]()
    if args.layers:
        keep = [int(x) for x in args.layers.split(",")]
        wl = wlm.Workload(**{**wl.__dict__, "layers": [wl.layers[i] for i in keep], "name": wl.name + "[" + args.layers + "]"})
    tokens = wl.tokens                     # per GPU: weak scaling, ranks hold different token shards
    gen = torch.Generator(device=dev)
    gen.manual_seed(1234 + rank)
    layers = [LayerBuffers(wl, li, tokens, dev, gen) for li in range(len(wl.layers))]
    if world > 1:                          # replicas start from identical weights
        for lb in layers:
            dist.broadcast(lb.W, 0)
    stream = torch.cuda.current_stream()

    def step(record=None):
        for i, lb in enumerate(layers):
            if record is None:
                dp.layer_step(lb.lay, lb.X, lb.dY, lb.W, lb.Y, lb.Z, lb.dX, lb.Gc, lb.M, lb.V)
                continue
            # the same calls as dp.layer_step, with an event between them
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            ev[0].record(stream)
            _, _, ep = lb.lay.forward(lb.X, lb.W, lb.Y, lb.Z)
            ev[1].record(stream)
            lb.lay.backward(lb.dY, lb.Z, lb.W, lb.Gc, lb.dX)
            ev[2].record(stream)
            dp.allreduce_compressed_grad(lb.Gc)
            lb.lay.adam_update(lb.W, lb.Gc, lb.M, lb.V, ep)
            ev[3].record(stream)
            lb.lay.refresh_projection()
            record.append((i, ev))

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    warm = max(args.warmup, 3)
    for _ in range(warm):
        step()
    sync_all()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    # bring the part to its sustained state: untimed steps for --preheat-seconds
    preheat_steps = 0
    t_pre = time.perf_counter()
    while time.perf_counter() - t_pre < args.preheat_seconds:
        for _ in range(4):
            step()
        torch.cuda.synchronize()
        preheat_steps += 4
    records = []
    launches0 = cb.kernel_launch_count()
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.time()
    e0.record(stream)
    for _ in range(args.steps):
        step(records)
    e1.record(stream)
    sync_all()
    wall1 = time.time()
    total_ms = e0.elapsed_time(e1)
    launches = cb.kernel_launch_count() - launches0
    clocks = sampler.stop(wall0, wall1) if rank == 0 else None
    if world > 1:
        t = torch.tensor([total_ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    flops_step = layer_flops(wl, tokens) * world
    value = flops_step / (ms_per_step * 1e-3) / 1e12

    # Secondary measurement (1 GPU): the same layers with q/k/v and gate/up run as groups that share one input,
    # as they do in a transformer block (compact_group_fwd / compact_group_bwd); same flops, fewer launches,
    # dX summed in the kernel.  The headline above keeps the per-layer calls.
    grouped = None
    if world == 1 and not args.no_groups:
        sets, i = [], 0
        fam_of = {"q": "qkv", "k": "qkv", "v": "qkv", "gate": "gu", "up": "gu"}
        names = [lb.L.name.split("_")[0] for lb in layers]
        while i < len(layers):
            j = i + 1
            fam = fam_of.get(names[i])
            while fam and j < len(layers) and j - i < 3 and fam_of.get(names[j]) == fam and layers[j].L.n == layers[i].L.n:
                j += 1
            sets.append(list(range(i, j)))
            i = j
        if any(len(g) > 1 for g in sets):
            groups = [(cb.CompactGroup([layers[k].lay for k in g]), g) for g in sets]

            def gstep():
                for grp, g in groups:
                    lbs = [layers[k] for k in g]
                    _, _, eps = grp.forward(lbs[0].X, [b.W for b in lbs], [b.Y for b in lbs], [b.Z for b in lbs])
                    grp.backward([b.dY for b in lbs], [b.Z for b in lbs], [b.W for b in lbs], [b.Gc for b in lbs], lbs[0].dX)
                    for b, ep in zip(lbs, eps):
                        b.lay.adam_update(b.W, b.Gc, b.M, b.V, ep)
                        b.lay.refresh_projection()

            for _ in range(3):
                gstep()
            torch.cuda.synchronize()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record(stream)
            for _ in range(args.steps):
                gstep()
            g1.record(stream)
            torch.cuda.synchronize()
            gms = g0.elapsed_time(g1) / args.steps
            grouped = {"ms_per_step": gms, "value": flops_step / (gms * 1e-3) / 1e12, "unit": UNIT,
                       "groups": [[layers[k].L.name for k in g] for g in sets],
                       "note": "same layers and flops, timed right after the headline in the same sustained state; "
                               "q/k/v and gate/up read one input each (compact_group_fwd/bwd)"}

    # per-call device times (CUDA events on the launching stream, inside the timed region)
    t_fwd = t_bwd = t_upd = 0.0
    per_layer = {}
    for i, ev in records:
        f, b, u = ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2]), ev[2].elapsed_time(ev[3])
        t_fwd += f; t_bwd += b; t_upd += u
        d = per_layer.setdefault(i, [0.0, 0.0, 0.0]); d[0] += f; d[1] += b; d[2] += u
    nrec = args.steps
    eb = 2 if wl.dtype == "bf16" else 4
    gemm_flops = sum(2.0 * tokens * (L.n * L.m + L.n * L.r + L.m * L.n + L.r * L.m) for L in wl.layers)
    upd_bytes = sum(wlm.update_bytes(L.n, L.m, L.r, eb) for L in wl.layers)
    peaks, peak_kind = measured_peaks()
    tens_peak = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
    tens_burst = float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
    hbm_peak = float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))
    gemm_ms = (t_fwd + t_bwd) / nrec
    gemm_tflops = gemm_flops / (gemm_ms * 1e-3) / 1e12
    upd_ms = t_upd / nrec
    upd_gbs = upd_bytes / (upd_ms * 1e-3) / 1e9
    gemm_launches = 2 * len(wl.layers)
    dram = [ncu_dram_bytes(L, tokens, eb) for L in wl.layers]
    traffic_gemm = sum(d[0] + d[1] for d in dram) / gemm_launches
    traffic_upd = sum(d[2] for d in dram) / len(wl.layers)
    roofline = {"kernel": "compact_gemm2_kernel (the forward and backward calls: Z, Y, Gc, dX on pairs of SMs; with them the expansion of P "
                          "and the reduction of the Gc partials, 2 % of their time)", "bound": "tensor",
                "achieved": gemm_tflops, "peak": tens_peak, "unit": "TFLOP/s", "frac": gemm_tflops / tens_peak,
                "peak_kind": f"{peak_kind} bf16 sustained (the kernel is timed inside a long step)",
                "frac_of_measured_burst": gemm_tflops / tens_burst, "frac_of_nominal_2250": gemm_tflops / NOMINAL_BF16_TFLOPS,
                "avg_launch_ms": gemm_ms / gemm_launches, "calls_per_step": gemm_launches,
                "algorithmic_flops_per_launch": gemm_flops / gemm_launches, "traffic": traffic_gemm,
                "traffic_note": "DRAM bytes per forward or backward call: the ncu captures of the three C5 shapes, averaged over the step's 14 calls"}
    # each layer's update against the roofline that bounds it: HBM below the ridge n r / (2 n + 10 r) flop/byte, tensor above
    ridge = tens_peak * 1e12 / (hbm_peak * 1e9)
    upd_layers = {}
    for i, v in per_layer.items():
        L = wl.layers[i]
        ms = v[2] / nrec
        by, fl = wlm.update_bytes(L.n, L.m, L.r, eb), 2.0 * L.n * L.r * L.m
        ent = {"ms": ms, "GB/s": by / (ms * 1e-3) / 1e9, "frac_of_measured_hbm": by / (ms * 1e-3) / 1e9 / hbm_peak,
               "TFLOP/s": fl / (ms * 1e-3) / 1e12, "flop_per_byte": fl / by, "bound": "tensor" if fl / by > ridge else "hbm"}
        if ent["bound"] == "tensor":
            ent["frac_of_measured_bf16_sustained"] = ent["TFLOP/s"] / tens_peak
        upd_layers[f"{L.name}#{i}"] = ent
    roofline_update = {"kernel": "update calls (adam_and_expand_kernel, compact_gemm2_kernel with W -= lr alpha P N in its epilogue)", "bound": "hbm",
                       "achieved": upd_gbs, "peak": hbm_peak, "unit": "GB/s", "frac": upd_gbs / hbm_peak,
                       "peak_kind": f"{peak_kind} copy", "frac_of_nominal_8000": upd_gbs / NOMINAL_HBM_GBS,
                       "avg_launch_ms": upd_ms / len(wl.layers), "algorithmic_bytes_per_launch": upd_bytes / len(wl.layers),
                       "traffic": traffic_upd, "per_layer": upd_layers, "ridge_flop_per_byte": ridge}

    # End to end through the public API with HOST inputs: every step copies each layer's X and dY from pinned host
    # memory and reads the step's Gc back.  The copies run on a stream of their own, a layer ahead of the compute.
    e2e = None
    if not args.no_e2e:
        hX = [torch.empty(lb.X.shape, dtype=lb.X.dtype, pin_memory=True).copy_(lb.X) for lb in layers]
        hdY = [torch.empty(lb.dY.shape, dtype=lb.dY.dtype, pin_memory=True).copy_(lb.dY) for lb in layers]
        hG = [torch.empty(lb.Gc.shape, dtype=lb.Gc.dtype, pin_memory=True) for lb in layers]
        h2d = sum(t.numel() * t.element_size() for t in hX + hdY)
        d2h = sum(t.numel() * t.element_size() for t in hG)
        up, down = torch.cuda.Stream(), torch.cuda.Stream()
        ready = [torch.cuda.Event() for _ in layers]
        consumed = [torch.cuda.Event() for _ in layers]
        reduced = [torch.cuda.Event() for _ in layers]
        for ev in consumed:
            ev.record(stream)

        def e2e_step():
            for i, (lb, x, dy) in enumerate(zip(layers, hX, hdY)):
                up.wait_event(consumed[i])             # the previous step has finished with this layer's inputs
                with torch.cuda.stream(up):
                    lb.X.copy_(x, non_blocking=True)
                    lb.dY.copy_(dy, non_blocking=True)
                    ready[i].record(up)
            for i, (lb, g) in enumerate(zip(layers, hG)):
                stream.wait_event(ready[i])
                _, _, ep = lb.lay.forward(lb.X, lb.W, lb.Y, lb.Z)
                lb.lay.backward(lb.dY, lb.Z, lb.W, lb.Gc, lb.dX)
                consumed[i].record(stream)
                dp.allreduce_compressed_grad(lb.Gc)
                reduced[i].record(stream)
                down.wait_event(reduced[i])
                with torch.cuda.stream(down):
                    g.copy_(lb.Gc, non_blocking=True)
                lb.lay.adam_update(lb.W, lb.Gc, lb.M, lb.V, ep)
                lb.lay.refresh_projection()
            stream.wait_stream(down)

        e2e_steps = max(1, min(args.steps, 5))
        e2e_step()
        sync_all()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        b.record(stream)
        sync_all()
        e2e_ms = a.elapsed_time(b) / e2e_steps
        if world > 1:
            t = torch.tensor([e2e_ms], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e_ms = float(t.item())
        e2e = {"value": flops_step / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d * world,
               "d2h_bytes_per_step": d2h * world, "ms_per_step": e2e_ms, "steps": e2e_steps,
               "h2d_gbs_per_gpu": h2d / (e2e_ms * 1e-3) / 1e9,
               "note": "copies on their own streams, overlapped with the compute of other layers; bound by the host link"}
        del hX, hdY, hG

    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            cpu = cpu_baseline_entry(oracle_sample(wl, max(1, wl.tokens // 16), steps=1))
        mhz = clocks.get("sm_mhz") if clocks else None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": wl.dtype, "data": "synthetic",
            "config": {"workload": wl.name, "tokens_per_gpu": tokens, "layers": [f"{L.name}:{L.n}x{L.m},r={L.r}" for L in wl.layers],
                       "refresh_T": wl.refresh_T, "l2": "inputs larger than L2 (layer set holds several GB)",
                       "parallelism": f"dp{world}" if world > 1 else "single",
                       "preheat_seconds": args.preheat_seconds, "preheat_steps": preheat_steps},
            "tokens_per_s": tokens * world / (ms_per_step * 1e-3),
            "pct_of_nominal_bf16_peak": 100.0 * value / (NOMINAL_BF16_TFLOPS * world),
            "pct_of_measured_bf16_sustained": 100.0 * value / (tens_peak * world),
            "pct_of_measured_bf16_burst": 100.0 * value / (tens_burst * world),
            "ms_times_mhz_per_step": (ms_per_step * mhz) if mhz else None,
            "per_call_ms": {"fwd": t_fwd / nrec, "bwd": t_bwd / nrec, "update": t_upd / nrec},
            "per_layer_ms": {wl.layers[i].name + f"#{i}": [x / nrec for x in v] for i, v in per_layer.items()},
            "roofline": roofline, "roofline_update": roofline_update, "cpu_baseline": cpu, "e2e": e2e, "grouped": grouped,
            "gpu_launches": int(launches), "clocks": clocks,
        }
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", choices=sorted(WORKLOADS))
    ap.add_argument("--preheat-seconds", type=float, default=2.0,
                    help="untimed steps under load before the timed ones, so that the clocks are the sustained ones")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-groups", action="store_true", help="skip the secondary measurement with q/k/v and gate/up as groups")
    ap.add_argument("--layers", default="", help="comma-separated layer indices of the workload (default: all)")
    args = ap.parse_args()
    if must_spawn(args.gpus, os.environ):
        from paper_2410_15352_b200 import dp
        sys.exit(dp.spawn_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
