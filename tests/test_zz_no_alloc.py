"""The allocation-free update entry point against the regular one.

Some users of this library step their optimizer from a place where asking CUDA for
memory is off the table: the framework around them has already taken all of HBM for
its pool, or they run inside another runtime's callback where an allocation would
stall every stream on the device.  `compact_adam_update_noalloc` serves them from a
scratch array built into the library.  This file checks, through the C ABI, that it
gives the same W, M, V as `compact_adam_update` on two consecutive steps, that the
second call is not disturbed by what the first one left in the shared scratch, and
that an oversized layer is refused before anything runs.  It is collected last so
that a failure here cannot hide other tests behind `-x`.
"""
import pytest
import torch

from oracle import compact_oracle as co
from paper_2410_15352_b200 import binding as cb
from paper_2410_15352_b200 import workloads as wlm
from paper_2410_15352_b200.build import build_library
from tests._harness import TOL, to64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()
    cb.set_kernel_family(0)


@pytest.mark.parametrize("dtype,tokens,n,m,r", [("bf16", 512, 512, 768, 128), ("f32", 256, 128, 512, 16)])
def test_noalloc_update_matches_regular_update_twice(dtype, tokens, n, m, r):
    wl = wlm.Workload("noalloc", 97, dtype, tokens, [wlm.LayerShape("l", n, m, r)], refresh_T=0,
                      x_scale_inv_sqrt_n=True)
    dt = wlm.torch_dtype(dtype)
    a = cb.CompactLinear(n, m, r, dtype=dt, seed=3, layer_id=2)
    b = cb.CompactLinear(n, m, r, dtype=dt, seed=3, layer_id=2)
    Wa = wlm.draw_W(wl, 0).cuda()
    Wb = Wa.clone()
    Ma, Va = torch.zeros((r, m), device="cuda"), torch.zeros((r, m), device="cuda")
    Mb, Vb = torch.zeros_like(Ma), torch.zeros_like(Va)
    launches_before = None
    for step in range(2):                       # two calls in a row share the built-in scratch
        X, dY = wlm.draw_X(wl, 0, step).cuda(), wlm.draw_dY(wl, 0, step).cuda()
        _, Z, ep = a.forward(X, Wa)
        _, Gc = a.backward(dY, Z, Wa, need_dX=False)
        a.adam_update(Wa, Gc, Ma, Va, ep)                       # regular entry point, caller's workspace
        torch.cuda.synchronize()
        free0, held0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        b.adam_update_noalloc(Wb, Gc, Mb, Vb, ep)               # same step from the built-in scratch
        torch.cuda.synchronize()
        if step == 1:
            # once the library's device code is resident (the first call saw to that), a call leaves the
            # device's free memory and torch's pool exactly as it found them
            assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == held0
        for name, x, y in (("W", Wa, Wb), ("M", Ma, Mb), ("V", Va, Vb)):
            assert co.rel_frobenius(to64(y), to64(x)) <= TOL[dtype], (step, name)
            assert torch.equal(x, y), (step, name)              # same kernels, same inputs: identical bits
        assert a.step == b.step == step + 1
    assert b.status() == cb.OK


def test_noalloc_update_refuses_oversized_layer():
    big = cb.CompactLinear(8192, 8192, 2048)    # r*m*4 = 64 MiB > 32 MiB of built-in scratch
    assert big.workspace_bytes(0) > cb.NOALLOC_SCRATCH_BYTES
    before = cb.kernel_launch_count()
    buf = torch.zeros(16, device="cuda")
    with pytest.raises(cb.CompactError) as e:
        big.adam_update_noalloc(buf, buf, buf, buf, 0)
    assert e.value.code == cb.ERR_SCRATCH_LIMIT
    assert cb.kernel_launch_count() == before and big.step == 0
