"""Shared parity harness: steps one layer through the CUDA path and the CPU
oracle on the same seeded inputs and returns relative Frobenius errors --
of whole tensors, and the worst one over tiles of each tensor."""
from __future__ import annotations

import numpy as np
import torch

from oracle import compact_oracle as co
from paper_2410_15352_b200 import binding as cb
from paper_2410_15352_b200 import workloads as wlm

TOL = {"f32": 1e-5, "bf16": 2e-2}     # relative Frobenius error (fp32; bf16 with fp32 accumulation)

# Bounds on the accumulated update, ||dW_gpu - dW_oracle|| / ||dW_oracle|| with dW = W_k - W_0.
# bf16: both sides store W in bf16, whose spacing near |W| ~ 0.02 is 2^-13 = 1.2e-4, while one step moves an
# entry by about lr * |P N| ~ 1e-3.  Where the two pre-rounding sums straddle a rounding boundary the stored
# values differ by one spacing; the pre-rounding sums differ by the bf16 rounding of the increment in the
# tensor-core update (2^-9 * 1e-3), by one-ulp differences in < 0.5 % of the entries of P, and, at step 1
# where N = sign(Gc), by sign flips of entries of Gc that are zero to rounding.  That is a few percent of the
# entries off by 12 % of a step: at most 0.03-0.05 after one step, and less, relative to the accumulated
# update, after several.  An update that applies a wrong tile of P, a wrong scale (alpha, lr, bias
# correction) or skips a tile is off by 0.3 or more.
TOL_DW = {"f32": 1e-4, "bf16": 6e-2}
# The worst tile may carry a few more flipped roundings than the average one.
TOL_DW_TILE = {"f32": 2e-4, "bf16": 1.5e-1}

TILE = (128, 64)          # tiles of Y, Z, dX, W: one epilogue warp-set block by one staged chunk
TILE_GC = (32, 32)        # tiles of Gc, M, V: one staged fp32 chunk


def f32(x: float) -> float:
    """The value the C ABI receives when a Python float is passed as a C float."""
    return float(np.float32(x))


def to64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def tile_sq_norms(a: np.ndarray, th: int, tw: int) -> np.ndarray:
    """Sum of squares over th x tw tiles (ragged edge tiles included) of a 2-D array."""
    a = np.asarray(a, dtype=np.float64)
    R, C = a.shape
    Rp, Cp = -(-R // th) * th, -(-C // tw) * tw
    sq = np.zeros((Rp, Cp))
    sq[:R, :C] = a * a
    return sq.reshape(Rp // th, th, Cp // tw, tw).sum(axis=(1, 3))


def worst_tile(a, b, tile=TILE) -> float:
    """max over tiles of ||a - b||_F / ||b||_F (b the oracle's tensor).  A tile whose oracle norm is below
    1e-3 of the average tile's is measured against the average instead (it holds almost nothing)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    if a.size == 0:
        return 0.0
    num = tile_sq_norms(a - b, *tile)
    den = tile_sq_norms(b, *tile)
    floor = 1e-6 * den.mean()
    if floor == 0.0:
        return float(np.sqrt(num.max()))
    return float(np.sqrt((num / np.maximum(den, floor)).max()))


def make_pair(wl: wlm.Workload, li: int):
    """(CUDA layer handle, oracle layer) for layer `li` of a workload."""
    L = wl.layers[li]
    dt = wlm.torch_dtype(wl.dtype)
    W0 = wlm.draw_W(wl, li)
    gpu = cb.CompactLinear(L.n, L.m, L.r, dtype=dt, seed=wl.seed, layer_id=li, refresh_T=wl.refresh_T,
                           lr=wl.lr, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps, alpha=wl.alpha, sparse_s=wl.sparse_s)
    ora = co.CompActLayerOracle(to64(W0), L.n, L.m, L.r, seed=wl.seed, layer_id=li, refresh_T=wl.refresh_T,
                                lr=f32(wl.lr), beta1=f32(wl.beta1), beta2=f32(wl.beta2), eps=f32(wl.eps),
                                alpha=f32(wl.alpha), mode="exact" if wl.dtype == "f32" else "bf16", sparse_s=wl.sparse_s)
    return gpu, ora, W0


def _record(errs, key, a, b, tile):
    errs[key] = max(errs.get(key, 0.0), co.rel_frobenius(a, b))
    errs[key + "_tile"] = max(errs.get(key + "_tile", 0.0), worst_tile(a, b, tile))


def run_layer_trajectory(wl: wlm.Workload, li: int, steps: int, tokens: int | None = None,
                         check_every_step: bool = True, lr_call=None):
    """Runs `steps` fwd+bwd+update+refresh on both sides.

    Returns (errs, epochs, dW, dW_tile): errs maps a tensor's name to its largest relative Frobenius error over
    the checked steps and name + "_tile" to the largest error of any tile; dW and dW_tile are the same two
    figures for the accumulated update W_k - W_0 (the largest over the checked steps).  lr_call: a learning
    rate handed to every update call instead of the layer configuration's."""
    tokens = wl.tokens if tokens is None else tokens
    L = wl.layers[li]
    gpu, ora, W0 = make_pair(wl, li)
    W = W0.cuda()
    W064 = to64(W0)
    M = torch.zeros((L.r, L.m), dtype=torch.float32, device="cuda")
    V = torch.zeros_like(M)
    errs, epochs = {}, []
    dW = dW_tile = 0.0
    for s in range(steps):
        X = wlm.draw_X(wl, li, s, tokens)
        dY = wlm.draw_dY(wl, li, s, tokens)
        Y, Z, ep = gpu.forward(X.cuda(), W)
        assert ep == ora.state.epoch
        epochs.append(ep)
        dX, Gc = gpu.backward(dY.cuda(), Z, W)
        Yo, Zo = ora.forward(to64(X))
        dXo, Gco = ora.backward(to64(dY), Zo)
        if lr_call is None:
            gpu.adam_update(W, Gc, M, V, ep)
            ora.update(Gco)
        else:
            gpu.adam_update(W, Gc, M, V, ep, lr=lr_call)
            ora.update(Gco, lr=f32(lr_call))
        gpu.refresh_projection()
        if check_every_step or s == steps - 1:
            assert not Z[:, L.r:].any(), "pad columns of Z must be exact zeros"
            for k, a, b, tile in (("Y", Y, Yo, TILE), ("Z", Z[:, :L.r], Zo, TILE), ("dX", dX, dXo, TILE),
                                  ("Gc", Gc, Gco, TILE_GC), ("W", W, ora.W, TILE), ("M", M, ora.M, TILE_GC),
                                  ("V", V, ora.V, TILE_GC)):
                _record(errs, k, to64(a), b, tile)
            dg, do = to64(W) - W064, ora.W - W064
            dW = max(dW, co.rel_frobenius(dg, do))
            dW_tile = max(dW_tile, worst_tile(dg, do, TILE))
        assert gpu.epoch == ora.state.epoch and gpu.step == ora.state.step
    assert gpu.status() == cb.OK
    return errs, epochs, dW, dW_tile


def assert_parity(errs, dW, dW_tile, dtype: str, what=""):
    """Every whole-tensor error and every worst-tile error within the tolerance of `dtype`, and the accumulated
    update within its own bounds."""
    for k, v in errs.items():
        assert v <= TOL[dtype], (what, k, v)
    assert dW <= TOL_DW[dtype], (what, "dW", dW)
    assert dW_tile <= TOL_DW_TILE[dtype], (what, "dW_tile", dW_tile)


def run_compressed_trajectory(wl: wlm.Workload, li: int, steps: int, tokens: int, yx_steps=(), n_rows: int = 256):
    """A whole trajectory at a large shape: the CUDA path runs every call in full; the oracle runs what the
    weight trajectory needs -- z = x P, G_hat = z^T dL/do and Algorithm 3, none of which reads W -- every step,
    and o = x W, dL/dx = dL/do W^T on `n_rows` sampled token rows at the steps listed in `yx_steps` (0-based).
    Returns (errs, epochs, dW, dW_tile) as run_layer_trajectory does."""
    L = wl.layers[li]
    gpu, ora, W0 = make_pair(wl, li)
    W = W0.cuda()
    W064 = to64(W0)
    M = torch.zeros((L.r, L.m), dtype=torch.float32, device="cuda")
    V = torch.zeros_like(M)
    errs, epochs = {}, []
    dW = dW_tile = 0.0
    rng = np.random.default_rng(1000 + li)
    P, P_epoch = None, -1
    for s in range(steps):
        X = wlm.draw_X(wl, li, s, tokens)
        dY = wlm.draw_dY(wl, li, s, tokens)
        Y, Z, ep = gpu.forward(X.cuda(), W)
        assert ep == ora.state.epoch
        epochs.append(ep)
        dX, Gc = gpu.backward(dY.cuda(), Z, W)
        X64, dY64 = to64(X), to64(dY)
        if P_epoch != ora.state.epoch:           # one projection per epoch on the oracle side too
            P, P_epoch = ora.P(), ora.state.epoch
        if s in yx_steps:
            rows = np.sort(rng.choice(tokens, size=min(n_rows, tokens), replace=False))
            rows[0], rows[-1] = 0, tokens - 1
            Yo, _ = co.linear_fwd(X64[rows], ora.W, P, ora.mode)
            dXo = co.round_bf16(dY64[rows] @ ora.W.T)
            _record(errs, "Y", to64(Y)[rows], Yo, (n_rows, 64))
            _record(errs, "dX", to64(dX)[rows], dXo, (n_rows, 64))
        Zo = co.round_bf16(X64 @ P)
        Gco = Zo.T @ dY64
        gpu.adam_update(W, Gc, M, V, ep)
        gpu.refresh_projection()
        ora.W, ora.M, ora.V = co.adam_update(ora.W, Gco, ora.M, ora.V, ora.state.step + 1, P, ora.lr, ora.beta1,
                                             ora.beta2, ora.eps, ora.alpha, ora.mode)
        ora.state.advance()
        assert not Z[:, L.r:].any(), "pad columns of Z must be exact zeros"
        for k, a, b, tile in (("Z", Z[:, :L.r], Zo, TILE), ("Gc", Gc, Gco, TILE_GC), ("W", W, ora.W, TILE),
                              ("M", M, ora.M, TILE_GC), ("V", V, ora.V, TILE_GC)):
            _record(errs, k, to64(a), b, tile)
        dg, do = to64(W) - W064, ora.W - W064
        dW = max(dW, co.rel_frobenius(dg, do))
        dW_tile = max(dW_tile, worst_tile(dg, do, TILE))
        assert gpu.epoch == ora.state.epoch and gpu.step == ora.state.step
    assert gpu.status() == cb.OK
    return errs, epochs, dW, dW_tile
