"""GPU parity of the layer with the sparse Johnson-Lindenstrauss projection (the paper's ablation study and the
"fuse the sampling and multiplication steps" remark of its Limitations section): the hashed terms bit for bit,
the projection's entries, and forward / backward / update trajectories against the oracle, through the C ABI.
On this GPU the tiles of P are still fed to the tensor cores -- as integer counts written straight into
shared memory, which costs a few Philox calls per row instead of a Gaussian per entry."""
import math

import numpy as np
import pytest
import torch

from oracle import compact_oracle as co
from paper_2410_15352_b200 import binding as cb
from paper_2410_15352_b200 import workloads as wlm
from paper_2410_15352_b200.build import build_library
from tests._harness import TOL, assert_parity, make_pair, run_compressed_trajectory, run_layer_trajectory, to64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()
    cb.set_kernel_family(0)
    yield
    cb.set_kernel_family(0)


@pytest.fixture(params=[0, 1, 2], ids=["auto", "simt", "nocluster"])
def family(request):
    cb.set_kernel_family(request.param)
    yield request.param
    cb.set_kernel_family(0)


@pytest.mark.parametrize("seed,layer,epoch,n,r,s", [
    (0, 0, 0, 128, 16, 8), ((9 << 32) | 0xABCDEF01, 6, 3, 400, 342, 6), (2 ** 64 - 1, 0xFFFFFFFF, 0xFFFFFFFF, 64, 7, 3),
    (1, 2, 1, 1376, 344, 1)])
def test_sparse_terms_bit_exact(seed, layer, epoch, n, r, s):
    lay = cb.CompactLinear(n, 64, r, seed=seed, layer_id=layer, sparse_s=s)
    got = lay.debug_sparse_terms(epoch=epoch).cpu().numpy().view(np.uint32)
    cols, signs = co.sparse_jl_terms(seed, layer, epoch, n, r, s)
    want = cols.astype(np.uint32) | np.where(signs < 0, np.uint32(0x80000000), np.uint32(0))
    assert got.shape == want.shape and np.array_equal(got, want)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_sparse_projection_entries(dtype):
    n, r, s = 520, 100, 8
    lay = cb.CompactLinear(n, 64, r, dtype=dtype, seed=3, layer_id=2, sparse_s=s)
    P = to64(lay.debug_projection(epoch=1))
    want = co.projection(3, 2, 1, n, r, sparse_s=s)
    assert np.array_equal(P != 0, want != 0)                                  # the same support
    rel = 2.0 ** -8 if dtype == torch.bfloat16 else 2e-7                       # one rounding of count / sqrt(s)
    assert np.all(np.abs(P - want) <= rel * np.abs(want))


SMALL = [
    # tokens, n, m, r, s
    (384, 512, 512, 128, 8),
    (300, 1376, 512, 344, 8),        # ragged tokens, ragged r
    (130, 264, 72, 50, 3),           # everything ragged, s not a multiple of four
    (1300, 192, 1544, 136, 8),       # several token blocks; m not a multiple of 64: the streaming update
    (700, 1200, 320, 600, 4),        # r beyond the resident panel: the streaming update with a sparse tile
    (640, 320, 512, 320, 16),        # r == n
]


@pytest.mark.parametrize("tokens,n,m,r,s", SMALL)
def test_sparse_bf16_trajectory(family, tokens, n, m, r, s):
    wl = wlm.Workload("sparse", 86, "bf16", tokens, [wlm.LayerShape("l", n, m, r)], steps=3, refresh_T=2,
                      x_scale_inv_sqrt_n=True, sparse_s=s)
    errs, epochs, dW, dW_tile = run_layer_trajectory(wl, 0, 3)
    assert epochs == [0, 0, 1]
    assert_parity(errs, dW, dW_tile, "bf16")


def test_sparse_fp32_trajectory():
    wl = wlm.Workload("sparse32", 85, "f32", 257, [wlm.LayerShape("l", 132, 260, 33)], steps=2, refresh_T=1, sparse_s=5)
    errs, epochs, dW, dW_tile = run_layer_trajectory(wl, 0, 2)
    assert epochs == [0, 1]
    assert_parity(errs, dW, dW_tile, "f32")


def test_sparse_z_rows_are_rows_of_p_bitwise(family):
    n, m, r, tokens, s = 512, 256, 100, 640, 8
    lay = cb.CompactLinear(n, m, r, seed=4, layer_id=1, sparse_s=s)
    Pb = lay.debug_projection()
    rows = np.random.default_rng(0).integers(0, n, size=tokens)
    X = torch.zeros((tokens, n), dtype=torch.bfloat16)
    X[torch.arange(tokens), torch.from_numpy(rows)] = 1.0
    X[::7] = 0.0
    W = torch.zeros((n, m), dtype=torch.bfloat16, device="cuda")
    _, Z, _ = lay.forward(X.cuda(), W)
    want = Pb[torch.from_numpy(rows).cuda()].clone()
    want[::7] = 0
    assert torch.equal(Z[:, :r].view(torch.int16), want.view(torch.int16)) and not Z[:, r:].any()


def test_sparse_config3_down_projection_full_size():
    # LLaMA-350M's 2736 -> 1024 layer at r = n/8 = 342 with outlier channels, 16384 tokens, two steps
    wl = wlm.config3(8)
    wl = wlm.Workload(**{**wl.__dict__, "sparse_s": 8, "name": wl.name + "_sparse"})
    errs, epochs, dW, dW_tile = run_compressed_trajectory(wl, 6, steps=2, tokens=wl.tokens, yx_steps=(0, 1), n_rows=48)
    assert epochs == [0, 0]
    assert_parity(errs, dW, dW_tile, "bf16")


def test_sparse_group_matches_single_layers():
    tokens, n = 700, 256
    shapes = [(512, 72), (512, 72)]
    wl = wlm.Workload("sgrp", 84, "bf16", tokens, [wlm.LayerShape(f"l{g}", n, m, r) for g, (m, r) in enumerate(shapes)],
                      x_scale_inv_sqrt_n=True, sparse_s=8)
    pairs = [make_pair(wl, g) for g in range(2)]
    gpus = [p[0] for p in pairs]
    Ws = [p[2].cuda() for p in pairs]
    X = wlm.draw_X(wl, 0, 0).cuda()
    Ys, Zs, _ = cb.CompactGroup(gpus).forward(X, Ws)
    for g, lay in enumerate(gpus):
        Y1, Z1, _ = lay.forward(X, Ws[g])
        assert torch.equal(Ys[g].view(torch.int16), Y1.view(torch.int16)) and torch.equal(Zs[g].view(torch.int16), Z1.view(torch.int16))
        Zo = co.round_bf16(to64(X) @ pairs[g][1].P())
        assert co.rel_frobenius(to64(Z1[:, :shapes[g][1]]), Zo) <= TOL["bf16"]
