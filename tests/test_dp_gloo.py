"""World-size-2 CPU (gloo) test of the data-parallel path: token shards, one
all-reduce of the compressed gradient, identical updates on every rank.  The
per-rank arithmetic is the oracle's (the CUDA path needs a GPU); what is under
test is the sharding and the exchange."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import compact_oracle as co
from paper_2410_15352_b200 import dp
from paper_2410_15352_b200 import workloads as wlm


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = wlm.Workload("dp", 96, "bf16", 640, [wlm.LayerShape("l", 64, 48, 16)], refresh_T=2, x_scale_inv_sqrt_n=True)
        L = wl.layers[0]
        W0 = wlm.draw_W(wl, 0).to(torch.float64).numpy()
        lay = co.CompActLayerOracle(W0, L.n, L.m, L.r, 0, 0, wl.refresh_T, 1e-3, 0.9, 0.999, 1e-8, mode="bf16")
        lo, hi = dp.shard_rows(wl.tokens, rank, world)
        for step in range(3):
            X = wlm.draw_X(wl, 0, step, hi - lo, row_start=lo).to(torch.float64).numpy()
            dY = wlm.draw_dY(wl, 0, step, hi - lo, row_start=lo).to(torch.float64).numpy()
            _, Z = lay.forward(X)
            _, Gc = lay.backward(dY, Z)
            G = torch.from_numpy(Gc.copy())
            dp.allreduce_compressed_grad(G)
            lay.update(G.numpy())
        q.put((rank, lo, hi, lay.W, lay.state.epoch))
    finally:
        dist.destroy_process_group()


def test_shard_rows_cover_and_align():
    for tokens, world in [(16384, 8), (640, 2), (1000, 3), (100, 4)]:
        spans = [dp.shard_rows(tokens, r, world) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == tokens
        for (a, b), (c, d) in zip(spans, spans[1:]):
            assert b == c and a <= b
        assert all(a % 128 == 0 or a == tokens for a, _ in spans)


def test_dp_two_ranks_match_single_rank():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=120) for _ in range(world)), key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # single-rank reference on the whole batch
    wl = wlm.Workload("dp", 96, "bf16", 640, [wlm.LayerShape("l", 64, 48, 16)], refresh_T=2, x_scale_inv_sqrt_n=True)
    W0 = wlm.draw_W(wl, 0).to(torch.float64).numpy()
    lay = co.CompActLayerOracle(W0, 64, 48, 16, 0, 0, 2, 1e-3, 0.9, 0.999, 1e-8, mode="bf16")
    for step in range(3):
        X = wlm.draw_X(wl, 0, step).to(torch.float64).numpy()
        dY = wlm.draw_dY(wl, 0, step).to(torch.float64).numpy()
        _, Z = lay.forward(X)
        _, Gc = lay.backward(dY, Z)
        lay.update(Gc)
    assert res[0][1:3] == (0, 384) and res[1][1:3] == (384, 640)
    assert np.array_equal(res[0][3], res[1][3])                # replicas stay bitwise in sync
    assert res[0][4] == res[1][4] == lay.state.epoch == 1
    assert np.allclose(res[0][3], lay.W, rtol=0, atol=2.0 ** -8 * np.abs(lay.W).max())   # sum order differs by shard
