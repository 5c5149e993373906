"""Parity at the benchmark configurations' full sizes, through the C ABI, in the
launch configuration bench.py times.  Small configurations run whole
trajectories against the oracle; at the large shapes the oracle checks sampled
rows of Y, Z, dX, sampled rows of Gc (reduced over all tokens) and sampled rows
of the updated W (which needs the full Gc), all on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import compact_oracle as co
from paper_2410_15352_b200 import binding as cb
from paper_2410_15352_b200 import workloads as wlm
from paper_2410_15352_b200.build import build_library
from tests._harness import (TILE, TILE_GC, TOL, TOL_DW, TOL_DW_TILE, assert_parity, f32, make_pair,
                            run_compressed_trajectory, run_layer_trajectory, to64, worst_tile)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()
    cb.set_kernel_family(0)


# ---- config 2: whole trajectories with refresh, one layer of each distinct shape ----------
@pytest.mark.parametrize("li", [0, 4, 6])
def test_config2_trajectory(li):
    wl = wlm.config2()
    errs, epochs, dW, dW_tile = run_layer_trajectory(wl, li, steps=wl.steps, check_every_step=True)
    assert epochs == [0] * 10 + [1] * 10
    assert_parity(errs, dW, dW_tile, "bf16", wl.layers[li].name)


FULL_SIZE = [
    ("c5", 0), ("c5", 4), ("c5", 6),          # LLaMA-7B shapes: 4096x4096 r512, 4096x11008 r512, 11008x4096 r1376
    ("c3r8", 6), ("c3r4", 6), ("c3r8", 4),    # ragged ranks 342 and 684, ragged m 2736, outlier channels
    ("c4", 5), ("c4", 4),                      # r = n/2 = 1536 with GELU inputs; 768 -> 3072
]
CONFIGS = {"c5": wlm.config5, "c4": wlm.config4, "c3r8": lambda: wlm.config3(8), "c3r4": lambda: wlm.config3(4)}


@pytest.mark.parametrize("cfg,li", FULL_SIZE)
def test_full_size_two_steps(cfg, li):
    # Two whole steps at the configuration's full token count, in the launch configuration bench.py times.
    # The oracle computes Z, Gc, M, V and W in full (so the second step carries moment history and both bias
    # corrections), Y and dX on sampled token rows; every tensor is also checked tile by tile.
    wl = CONFIGS[cfg]()
    errs, epochs, dW, dW_tile = run_compressed_trajectory(wl, li, steps=2, tokens=wl.tokens, yx_steps=(0, 1), n_rows=48)
    assert epochs == [0, 0]
    assert_parity(errs, dW, dW_tile, "bf16", (cfg, li))


@pytest.mark.parametrize("li", [4, 6])
def test_full_size_tile_orders_same_bits(li):
    # At the LLaMA-7B MLP shapes the pair-of-SMs launches walk operands larger than the L2 in column panels (and the
    # forward numbers Z and Y tiles in its own order).  Every tile of every output against the single-SM family,
    # which numbers its items differently and generates P on chip: all outputs bit for bit, full size.
    wl = wlm.config5()
    X, dY = wlm.draw_X(wl, li, 0).cuda(), wlm.draw_dY(wl, li, 0).cuda()
    out = []
    for fam in (0, 2):
        cb.set_kernel_family(fam)
        gpu, _, W0 = make_pair(wl, li)
        W = W0.cuda()
        Y, Z, _ = gpu.forward(X, W)
        dX, Gc = gpu.backward(dY, Z, W)
        assert gpu.status() == cb.OK
        out.append((Y, Z, dX, Gc))
        del gpu
    cb.set_kernel_family(0)
    for a, b in zip(*out):
        assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a, b.view(torch.int16) if b.dtype == torch.bfloat16 else b)


# ---- configs 3 and 4 at their stated step counts and refresh periods -----------------------------------
# The attention shapes run at the full token count; the wide shapes (whose oracle step costs seconds) at a
# quarter of it, which leaves every tile shape, the ragged ranks and the schedule as they are.
STATED = [
    ("c3r8", 0, 16384), ("c3r4", 0, 16384),            # 1024 -> 1024, r = 128 and 256: 50 steps, T = 25
    ("c3r8", 6, 4096), ("c3r4", 6, 4096),              # 2736 -> 1024, r = 342 and 684 (ragged)
    ("c3r4", 4, 4096),                                 # 1024 -> 2736, r = 256
    ("c4", 0, 16384), ("c4", 4, 4096), ("c4", 5, 4096),  # 768 -> 768, 768 -> 3072, 3072 -> 768 (r = n/2): 30 steps, T = 10
]


@pytest.mark.parametrize("cfg,li,tokens", STATED)
def test_stated_steps_with_refresh(cfg, li, tokens):
    wl = CONFIGS[cfg]()
    T = wl.refresh_T
    # o and dL/dx are checked on sampled rows at the first step, right after each refresh and at the last step
    yx = sorted({0, wl.steps - 1} | {k * T for k in range(1, wl.steps // T + 1) if k * T < wl.steps})
    errs, epochs, dW, dW_tile = run_compressed_trajectory(wl, li, steps=wl.steps, tokens=tokens, yx_steps=yx)
    assert epochs == [s // T for s in range(wl.steps)]
    assert_parity(errs, dW, dW_tile, "bf16", (cfg, li))


def test_config5_reduced_tokens_trajectory():
    # whole-tensor parity over 3 steps at the 7B layer shape with fewer tokens
    wl = wlm.config5().with_tokens(2048)
    errs, epochs, dW, dW_tile = run_layer_trajectory(wl, 0, steps=3)
    assert epochs == [0, 0, 0]
    assert_parity(errs, dW, dW_tile, "bf16")


def test_forced_refresh_changes_projection():
    wl = wlm.config5().with_tokens(512)
    gpu, ora, W0 = make_pair(wl, 0)
    X = wlm.draw_X(wl, 0, 0, 512).cuda()
    W = W0.cuda()
    _, Z0, ep0 = gpu.forward(X, W)
    assert gpu.refresh_projection(force=True) == ep0 + 1
    _, Z1, ep1 = gpu.forward(X, W)
    assert ep1 == ep0 + 1 and not torch.equal(Z0, Z1)
    Zo = co.round_bf16(to64(X) @ co.projection(wl.seed, 0, 1, 4096, 512, "bf16"))
    assert co.rel_frobenius(to64(Z1), Zo) <= TOL["bf16"]
