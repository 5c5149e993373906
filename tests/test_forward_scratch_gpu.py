"""The two ways compact_linear_fwd builds Z = X P (Algorithm 1 line 2): with scratch, P of the epoch is written
out once and Z is a further set of columns of the pair-of-SMs product; without, the kernel regenerates the tiles
of P where it consumes them.  Same entries of P, same accumulation order: the results must agree bit for bit,
and each must agree with the oracle."""
import ctypes as C
import math

import pytest
import torch

from oracle import compact_oracle as co
from paper_2410_15352_b200 import binding as cb
from paper_2410_15352_b200 import workloads as wlm
from paper_2410_15352_b200.build import build_library

from tests._harness import TOL, make_pair, to64, worst_tile

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()
    cb.set_kernel_family(0)
    yield
    cb.set_kernel_family(0)


def bits(t):
    return t.view(torch.int16) if t.dtype == torch.bfloat16 else t


SHAPES = [
    # tokens, n, m, r, sparse_s
    (5, 64, 64, 8, 0),              # fewer tokens than one tile row
    (300, 256, 136, 40, 0),         # everything ragged; r < 64: one block of P that is mostly padding
    (1000, 520, 264, 100, 0),       # n not a multiple of 64: the last k-step reads past the end of X and P
    (1300, 192, 1544, 136, 0),      # several column tiles of W, two of P
    (2100, 448, 2056, 342, 0),      # r = 342 -> 352 columns of Z, 384 of scratch: a tile of P with a zero tail
    (1000, 520, 264, 100, 4),       # sparse projection: integer counts in scratch, 1 / sqrt(s) in the epilogue
    (2100, 448, 520, 342, 8),
]


@pytest.mark.parametrize("tokens,n,m,r,s", SHAPES)
def test_with_and_without_scratch_same_bits_and_oracle(tokens, n, m, r, s):
    wl = wlm.Workload("scr", 77, "bf16", tokens, [wlm.LayerShape("l", n, m, r)], x_scale_inv_sqrt_n=True, sparse_s=s)
    gpu, ora, W0 = make_pair(wl, 0)
    W, X = W0.cuda(), wlm.draw_X(wl, 0, 0).cuda()
    before = cb.kernel_launch_count()
    Y0, Z0, _ = gpu.forward(X, W, scratch=False)
    mid = cb.kernel_launch_count()
    Y1 = torch.full_like(Y0, 3.0)
    Z1 = torch.full_like(Z0, 3.0)
    gpu.forward(X, W, Y1, Z1)
    assert cb.kernel_launch_count() - mid == 2          # the expansion and the product
    assert 1 <= mid - before <= 2
    assert gpu.status() == cb.OK
    assert torch.equal(bits(Y0), bits(Y1)) and torch.equal(bits(Z0), bits(Z1))
    assert not Z1[:, r:].any()
    Yo, Zo = ora.forward(to64(X))
    for a, b in ((Y1, Yo), (Z1[:, :r], Zo)):
        assert co.rel_frobenius(to64(a), b) <= TOL["bf16"]
        assert worst_tile(to64(a), b) <= TOL["bf16"]


def test_empty_batch_with_scratch_launches_nothing():
    lay = cb.CompactLinear(256, 136, 40)
    W = torch.zeros((256, 136), dtype=torch.bfloat16, device="cuda")
    X = torch.zeros((0, 256), dtype=torch.bfloat16, device="cuda")
    before = cb.kernel_launch_count()
    Y, Z, ep = lay.forward(X, W)
    assert cb.kernel_launch_count() == before and Y.shape == (0, 136) and Z.shape == (0, lay.ldz) and ep == 0


def test_scratch_holds_the_projection_the_debug_kernel_writes():
    # White box: what the expansion leaves at the front of the workspace (its contents are not part of the
    # interface) against the per-entry debug kernel, which shares no code path with it beyond Philox/Box-Muller.
    for n, m, r, s in ((520, 264, 100, 0), (448, 520, 342, 8)):
        lay = cb.CompactLinear(n, m, r, seed=5, layer_id=2, sparse_s=s)
        W = torch.zeros((n, m), dtype=torch.bfloat16, device="cuda")
        X = torch.zeros((64, n), dtype=torch.bfloat16, device="cuda")
        lay.forward(X, W)
        ldp = -(-lay.ldz // 64) * 64
        ws = lay.workspace(64)[: n * ldp * 2].view(torch.bfloat16).view(n, ldp)
        assert not ws[:, r:].any()
        P = lay.debug_projection()
        if s == 0:
            assert torch.equal(bits(ws[:, :r].contiguous()), bits(P))
        else:
            counts = ws[:, :r].float()
            assert torch.equal(counts, counts.round()) and counts.abs().sum(dim=1).max() <= s
            assert torch.equal((counts * (1.0 / math.sqrt(s))).to(torch.bfloat16), P)


def test_group_with_and_without_scratch_same_bits():
    tokens, n = 1100, 320
    shapes = [(512, 72), (1096, 40), (520, 136)]
    wl = wlm.Workload("grp", 95, "bf16", tokens, [wlm.LayerShape(f"l{g}", n, m, r) for g, (m, r) in enumerate(shapes)],
                      x_scale_inv_sqrt_n=True)
    pairs = [make_pair(wl, g) for g in range(len(shapes))]
    grp = cb.CompactGroup([p[0] for p in pairs])
    Ws = [p[2].cuda() for p in pairs]
    X = wlm.draw_X(wl, 0, 0).cuda()
    Ys0, Zs0, _ = grp.forward(X, Ws, scratch=False)
    before = cb.kernel_launch_count()
    Ys1, Zs1, _ = grp.forward(X, Ws)
    assert cb.kernel_launch_count() - before == len(shapes) + 1      # one expansion per layer, one product
    for a, b in zip(Ys0 + Zs0, Ys1 + Zs1):
        assert torch.equal(bits(a), bits(b))


def test_scratch_that_is_too_small_is_not_used_and_misaligned_scratch_is_refused():
    tokens, n, m, r = 300, 256, 136, 40
    lay = cb.CompactLinear(n, m, r, seed=3)
    L = cb.lib()
    need = int(L.compact_fwd_workspace_bytes(lay._h))
    assert need == n * 64 * 2 and lay.workspace_bytes(tokens) >= need
    W = (torch.randn(n, m, device="cuda") * 0.05).to(torch.bfloat16)
    X = torch.randn(tokens, n, device="cuda").to(torch.bfloat16)
    Y0, Z0, _ = lay.forward(X, W, scratch=False)
    Y = torch.empty_like(Y0)
    Z = torch.empty_like(Z0)
    ws = torch.full((need,), 0x5A, dtype=torch.uint8, device="cuda")
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)

    def call(ptr, size):
        return L.compact_linear_fwd(lay._h, tokens, X.data_ptr(), n, W.data_ptr(), m, Y.data_ptr(), m, Z.data_ptr(), lay.ldz,
                                    None, C.c_void_p(ptr), size, st)

    assert call(ws.data_ptr(), need - 256) == cb.OK
    torch.cuda.synchronize()
    assert bool((ws == 0x5A).all())                        # untouched: the kernel generated P itself
    assert torch.equal(bits(Y), bits(Y0)) and torch.equal(bits(Z), bits(Z0))
    assert call(ws.data_ptr() + 8, need - 8) == cb.ERR_ALIGNMENT
    assert call(ws.data_ptr(), need) == cb.OK
    torch.cuda.synchronize()
    assert not bool((ws == 0x5A).all())
    assert torch.equal(bits(Y), bits(Y0)) and torch.equal(bits(Z), bits(Z0))
    assert lay.status() == cb.OK
