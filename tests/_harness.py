"""Shared parity harness: steps one layer through the CUDA path and the CPU
oracle on the same seeded inputs and returns relative Frobenius errors."""
from __future__ import annotations

import numpy as np
import torch

from oracle import compact_oracle as co
from paper_2410_15352_b200 import binding as cb
from paper_2410_15352_b200 import workloads as wlm

TOL = {"f32": 1e-5, "bf16": 2e-2}     # relative Frobenius error (fp32; bf16 with fp32 accumulation)


def f32(x: float) -> float:
    """The value the C ABI receives when a Python float is passed as a C float."""
    return float(np.float32(x))


def to64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def make_pair(wl: wlm.Workload, li: int):
    """(CUDA layer handle, oracle layer) for layer `li` of a workload."""
    L = wl.layers[li]
    dt = wlm.torch_dtype(wl.dtype)
    W0 = wlm.draw_W(wl, li)
    gpu = cb.CompactLinear(L.n, L.m, L.r, dtype=dt, seed=wl.seed, layer_id=li, refresh_T=wl.refresh_T,
                           lr=wl.lr, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps, alpha=wl.alpha)
    ora = co.CompActLayerOracle(to64(W0), L.n, L.m, L.r, seed=wl.seed, layer_id=li, refresh_T=wl.refresh_T,
                                lr=f32(wl.lr), beta1=f32(wl.beta1), beta2=f32(wl.beta2), eps=f32(wl.eps),
                                alpha=f32(wl.alpha), mode="exact" if wl.dtype == "f32" else "bf16")
    return gpu, ora, W0


def run_layer_trajectory(wl: wlm.Workload, li: int, steps: int, tokens: int | None = None,
                         check_every_step: bool = True):
    """Runs `steps` fwd+bwd+update+refresh on both sides; returns {name: max rel error}."""
    tokens = wl.tokens if tokens is None else tokens
    L = wl.layers[li]
    gpu, ora, W0 = make_pair(wl, li)
    W = W0.cuda()
    M = torch.zeros((L.r, L.m), dtype=torch.float32, device="cuda")
    V = torch.zeros_like(M)
    errs = {k: 0.0 for k in ("Y", "Z", "dX", "Gc", "W", "M", "V")}
    epochs = []
    for s in range(steps):
        X = wlm.draw_X(wl, li, s, tokens)
        dY = wlm.draw_dY(wl, li, s, tokens)
        Y, Z, ep = gpu.forward(X.cuda(), W)
        assert ep == ora.state.epoch
        epochs.append(ep)
        dX, Gc = gpu.backward(dY.cuda(), Z, W)
        Yo, Zo = ora.forward(to64(X))
        dXo, Gco = ora.backward(to64(dY), Zo)
        gpu.adam_update(W, Gc, M, V, ep)
        gpu.refresh_projection()
        ora.update(Gco)
        if check_every_step or s == steps - 1:
            assert not Z[:, L.r:].any(), "pad columns of Z must be exact zeros"
            for k, a, b in (("Y", Y, Yo), ("Z", Z[:, :L.r], Zo), ("dX", dX, dXo), ("Gc", Gc, Gco),
                            ("W", W, ora.W), ("M", M, ora.M), ("V", V, ora.V)):
                errs[k] = max(errs[k], co.rel_frobenius(to64(a), b))
        assert gpu.epoch == ora.state.epoch and gpu.step == ora.state.step
    dW = co.rel_frobenius(to64(W) - to64(W0), ora.W - to64(W0))
    return errs, epochs, dW
