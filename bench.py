#!/usr/bin/env python
"""Benchmark of the CompAct compressed linear layer on B200.

One "step" is one pass of the whole hot path -- forward [Y|Z] = X[W|P], backward
dX = dY W^T and Gc = Z^T dY, Adam update W <- W - lr*alpha*P N, refresh -- over
every layer of the LLaMA-7B-shaped layer set (16384 tokens, hidden 4096) with
synthetic inputs.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c5|c4|c3|c2]

`--impl reference` times the CPU oracle (oracle/) as it stands on the host cores,
on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
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
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
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
                 "-lms", "20"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, pw = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 8:
                    continue
                try:
                    sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
                except ValueError:
                    continue
                for nm, v in zip(names, f[4:8]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm),
                       power_w_max=max(pw))
        return out


# ----------------------------------------------------------------------------------------
# the CPU oracle leg (reported baseline; also `--impl reference`)
# ----------------------------------------------------------------------------------------
def oracle_sample(wl: wlm.Workload, sample_tokens: int, steps: int = 1, layer_ids=(0,)):
    """fwd+bwd+update of the layers `layer_ids` on `sample_tokens` tokens with the
    oracle as it stands.  Returns (seconds per step, flops per step, threads)."""
    import numpy as np
    from oracle import compact_oracle as co
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    mode = "exact" if wl.dtype == "f32" else "bf16"
    layers = []
    for li in layer_ids:
        L = wl.layers[li]
        W0 = wlm.draw_W(wl, li).to(torch.float64).numpy()
        layers.append(co.CompActLayerOracle(W0, L.n, L.m, L.r, wl.seed, li, wl.refresh_T, wl.lr, wl.beta1, wl.beta2,
                                            wl.eps, wl.alpha, mode))
    times = []
    for s in range(steps):
        ins = [(wlm.draw_X(wl, li, s, sample_tokens).to(torch.float64).numpy(),
                wlm.draw_dY(wl, li, s, sample_tokens).to(torch.float64).numpy()) for li in layer_ids]
        t0 = time.perf_counter()
        for lay, (X, dY) in zip(layers, ins):
            Y, Z = lay.forward(X)
            dX, Gc = lay.backward(dY, Z)
            lay.update(Gc)
        times.append(time.perf_counter() - t0)
    flops = sum(wlm.algorithmic_flops(sample_tokens, wl.layers[li].n, wl.layers[li].m, wl.layers[li].r) for li in layer_ids)
    return statistics.median(times), flops, threads


def sample_description(wl: wlm.Workload, sample_tokens: int, layer_ids=(0,)) -> str:
    names = ", ".join(f"{wl.layers[li].name} {wl.layers[li].n}x{wl.layers[li].m} r={wl.layers[li].r}" for li in layer_ids)
    return f"layer(s) [{names}] of {wl.name}, {sample_tokens} of {wl.tokens} tokens, full update, per step"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = WORKLOADS[args.workload]()
    sample_tokens = 256
    sec, flops, threads = oracle_sample(wl, sample_tokens, steps=max(1, args.steps))
    val = flops / sec / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "tokens": wl.tokens, "sample": sample_description(wl, sample_tokens)},
        "tokens_per_s": sample_tokens / sec,
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": sample_description(wl, sample_tokens)},
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
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)] if record is not None else None
            if ev: ev[0].record(stream)
            _, _, ep = lb.lay.forward(lb.X, lb.W, lb.Y, lb.Z)
            if ev: ev[1].record(stream)
            lb.lay.backward(lb.dY, lb.Z, lb.W, lb.Gc, lb.dX)
            if ev: ev[2].record(stream)
            if world > 1:                  # data parallel: the only exchange is the r x m compressed gradient
                dp.allreduce_compressed_grad(lb.Gc)
            lb.lay.adam_update(lb.W, lb.Gc, lb.M, lb.V, ep)
            if ev: ev[3].record(stream)
            lb.lay.refresh_projection()
            if ev: record.append((i, ev))

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    sync_all()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    records = []
    launches0 = cb.kernel_launch_count()
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step(records)
    e1.record(stream)
    sync_all()
    total_ms = e0.elapsed_time(e1)
    launches = cb.kernel_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
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
        names = [lb.L.name.split("_")[0] for lb in layers]
        while i < len(layers):
            j = i + 1
            fam = {"q": "qkv", "k": "qkv", "v": "qkv", "gate": "gu", "up": "gu"}.get(names[i])
            while fam and j < len(layers) and j - i < 3 and {"q": "qkv", "k": "qkv", "v": "qkv", "gate": "gu", "up": "gu"}.get(names[j]) == fam \
                    and layers[j].L.n == layers[i].L.n:
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
            # the per-layer step again, right after: the part is power-capped and slows down over a long run, so
            # only numbers taken next to each other compare
            g0.record(stream)
            for _ in range(args.steps):
                step()
            g1.record(stream)
            torch.cuda.synchronize()
            pms = g0.elapsed_time(g1) / args.steps
            grouped = {"ms_per_step": gms, "value": flops_step / (gms * 1e-3) / 1e12, "unit": UNIT,
                       "per_layer_ms_per_step_right_after": pms,
                       "groups": [[layers[k].L.name for k in g] for g in sets],
                       "note": "same layers and flops; q/k/v and gate/up read one input each (compact_group_fwd/bwd)"}

    # per-call device times (CUDA events on the launching stream, inside the timed region)
    t_fwd = t_bwd = t_upd = 0.0
    per_layer = {}
    for i, ev in records:
        f, b, u = ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2]), ev[2].elapsed_time(ev[3])
        t_fwd += f; t_bwd += b; t_upd += u
        d = per_layer.setdefault(i, [0.0, 0.0, 0.0]); d[0] += f; d[1] += b; d[2] += u
    nrec = args.steps
    gemm_flops = sum(2.0 * tokens * (L.n * L.m + L.n * L.r + L.m * L.n + L.r * L.m) for L in wl.layers)
    upd_bytes = sum(wlm.update_bytes(L.n, L.m, L.r, 2 if wl.dtype == "bf16" else 4) for L in wl.layers)
    peaks, peak_kind = measured_peaks()
    tens_peak = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
    hbm_peak = float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))
    gemm_ms = (t_fwd + t_bwd) / nrec
    gemm_tflops = gemm_flops / (gemm_ms * 1e-3) / 1e12
    upd_ms = t_upd / nrec
    upd_gbs = upd_bytes / (upd_ms * 1e-3) / 1e9
    gemm_launches = 2 * len(wl.layers)
    # DRAM traffic from the committed ncu capture of the C5 q_proj launches
    # (profiles/compact_gemm_kernel_c5_qproj_full.md): forward 578.9 MB, backward 629.6 MB for
    # 1236.95 algorithmic GFLOP; update 37.9 MB for 109.1 MB of algorithmic bytes (W stays in L2
    # at that size).  Scaled to this workload's launches in proportion to the algorithmic work.
    traffic_gemm = (578.9e6 + 629.6e6) / 1236.95e9 * gemm_flops / gemm_launches
    traffic_upd = None
    roofline = {"kernel": "compact_gemm_kernel (forward and backward launches)", "bound": "tensor",
                "achieved": gemm_tflops, "peak": tens_peak, "unit": "TFLOP/s", "frac": gemm_tflops / tens_peak,
                "peak_kind": f"{peak_kind} bf16 sustained", "frac_of_nominal_2250": gemm_tflops / NOMINAL_BF16_TFLOPS,
                "avg_launch_ms": gemm_ms / gemm_launches, "launches_per_step": gemm_launches,
                "algorithmic_flops_per_launch": gemm_flops / gemm_launches, "traffic": traffic_gemm,
                "traffic_note": "bytes per launch, scaled by flops from the ncu capture of the C5 q_proj forward+backward launches"}
    roofline_update = {"kernel": "adam_moments + compact_gemm_kernel (update launches)", "bound": "hbm",
                       "achieved": upd_gbs, "peak": hbm_peak, "unit": "GB/s", "frac": upd_gbs / hbm_peak,
                       "peak_kind": f"{peak_kind} copy", "frac_of_nominal_8000": upd_gbs / NOMINAL_HBM_GBS,
                       "avg_launch_ms": upd_ms / len(wl.layers), "algorithmic_bytes_per_launch": upd_bytes / len(wl.layers),
                       "traffic": traffic_upd}

    # end to end through the public API with HOST inputs: H2D of X, dY every step, D2H of the step's Gc
    e2e = None
    if (rank == 0 or world > 1) and not args.no_e2e:
        hX = [torch.empty(lb.X.shape, dtype=lb.X.dtype, pin_memory=True).copy_(lb.X) for lb in layers]
        hdY = [torch.empty(lb.dY.shape, dtype=lb.dY.dtype, pin_memory=True).copy_(lb.dY) for lb in layers]
        hG = [torch.empty(lb.Gc.shape, dtype=lb.Gc.dtype, pin_memory=True) for lb in layers]
        h2d = sum(t.numel() * t.element_size() for t in hX + hdY)
        d2h = sum(t.numel() * t.element_size() for t in hG)

        def e2e_step():
            for lb, x, dy, g in zip(layers, hX, hdY, hG):
                lb.X.copy_(x, non_blocking=True)
                lb.dY.copy_(dy, non_blocking=True)
                _, _, ep = lb.lay.forward(lb.X, lb.W, lb.Y, lb.Z)
                lb.lay.backward(lb.dY, lb.Z, lb.W, lb.Gc, lb.dX)
                if world > 1:
                    dp.allreduce_compressed_grad(lb.Gc)
                lb.lay.adam_update(lb.W, lb.Gc, lb.M, lb.V, ep)
                lb.lay.refresh_projection()
                g.copy_(lb.Gc, non_blocking=True)

        e2e_steps = max(1, min(args.steps, 3))
        e2e_step()
        sync_all()
        t0 = time.perf_counter()
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
        e2e = {"value": flops_step / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps}
        del hX, hdY, hG

    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            sample_tokens = 256
            sec, fl, threads = oracle_sample(wl, sample_tokens, steps=5)
            cpu = {"value": fl / sec / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle",
                   "sample": sample_description(wl, sample_tokens),
                   "seconds": sec}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": wl.dtype, "data": "synthetic",
            "config": {"workload": wl.name, "tokens_per_gpu": tokens, "layers": [f"{L.name}:{L.n}x{L.m},r={L.r}" for L in wl.layers],
                       "refresh_T": wl.refresh_T, "l2": "inputs larger than L2 (layer set holds several GB)",
                       "parallelism": f"dp{world}" if world > 1 else "single"},
            "tokens_per_s": tokens * world / (ms_per_step * 1e-3),
            "pct_of_nominal_bf16_peak": 100.0 * value / (NOMINAL_BF16_TFLOPS * world),
            "pct_of_measured_bf16_sustained": 100.0 * value / (tens_peak * world),
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
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-groups", action="store_true", help="skip the secondary measurement with q/k/v and gate/up as groups")
    ap.add_argument("--layers", default="", help="comma-separated layer indices of the workload (default: all)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
