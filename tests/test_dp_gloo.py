"""World-size-2 CPU (gloo) test of the data-parallel path: token shards, one
all-reduce of the compressed gradient, identical updates on every rank.  The
step function is the one bench.py drives (dp.layer_step); the per-rank
arithmetic behind it is the oracle's, wrapped in the binding's interface (the
CUDA path needs a GPU); what is under test is the sharding, the exchange and
the launcher."""
import os
import socket
import subprocess
import sys
import textwrap

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


class OracleAsLayer:
    """The oracle layer behind the call interface of binding.CompactLinear (tensors are fp64 CPU tensors)."""

    def __init__(self, ora):
        self.ora = ora

    def forward(self, X, W, Y, Z):
        Yo, Zo = self.ora.forward(X.numpy())
        Y.copy_(torch.from_numpy(Yo)); Z.copy_(torch.from_numpy(Zo))
        return Y, Z, self.ora.state.epoch

    def backward(self, dY, Z, W, Gc, dX):
        dXo, Gco = self.ora.backward(dY.numpy(), Z.numpy())
        dX.copy_(torch.from_numpy(dXo)); Gc.copy_(torch.from_numpy(Gco))
        return dX, Gc

    def adam_update(self, W, Gc, M, V, epoch, lr=None):
        assert epoch == self.ora.state.epoch
        self.ora.update(Gc.numpy(), lr=lr)
        W.copy_(torch.from_numpy(self.ora.W))

    def refresh_projection(self):
        return self.ora.state.epoch          # the oracle's update already advanced the schedule


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = wlm.Workload("dp", 96, "bf16", 640, [wlm.LayerShape("l", 64, 48, 16)], refresh_T=2, x_scale_inv_sqrt_n=True)
        L = wl.layers[0]
        W0 = wlm.draw_W(wl, 0).to(torch.float64)
        lay = OracleAsLayer(co.CompActLayerOracle(W0.numpy(), L.n, L.m, L.r, 0, 0, wl.refresh_T, 1e-3, 0.9, 0.999, 1e-8, mode="bf16"))
        lo, hi = dp.shard_rows(wl.tokens, rank, world)
        t = hi - lo
        f64 = lambda *shape: torch.zeros(shape, dtype=torch.float64)
        W, Y, Z, dX, Gc, M, V = W0.clone(), f64(t, L.m), f64(t, L.r), f64(t, L.n), f64(L.r, L.m), f64(L.r, L.m), f64(L.r, L.m)
        epochs = []
        for step in range(3):
            X = wlm.draw_X(wl, 0, step, t, row_start=lo).to(torch.float64)
            dY = wlm.draw_dY(wl, 0, step, t, row_start=lo).to(torch.float64)
            epochs.append(dp.layer_step(lay, X, dY, W, Y, Z, dX, Gc, M, V))
        assert epochs == [0, 0, 1]
        q.put((rank, lo, hi, W.numpy(), lay.ora.state.epoch))
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


def test_launcher_starts_one_rank_per_gpu(tmp_path):
    # `bench.py --gpus N` outside a launcher re-runs itself through dp.spawn_ranks; here a stand-in script
    # takes the place of the benchmark and records what each rank was given
    worker = tmp_path / "fake_worker.py"
    worker.write_text(textwrap.dedent("""
        import os, sys
        e = os.environ
        open(os.path.join(sys.argv[1], "rank%s.txt" % e["RANK"]), "w").write(
            " ".join([e["RANK"], e["LOCAL_RANK"], e["WORLD_SIZE"], e["MASTER_ADDR"], e["MASTER_PORT"]] + sys.argv[2:]))
    """))
    port = dp.free_port()
    env = dict(os.environ, RANK="7", WORLD_SIZE="9")          # leftovers of an outer launcher must not leak in
    rc = dp.spawn_ranks(2, str(worker), [str(tmp_path), "--gpus", "2"], port=port, env=env)
    assert rc == 0
    got = sorted((tmp_path / f"rank{r}.txt").read_text().split() for r in range(2))
    assert got == [[str(r), str(r), "2", "127.0.0.1", str(port), "--gpus", "2"] for r in range(2)]


def test_bench_decides_when_to_spawn():
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    assert bench.must_spawn(gpus=2, environ={}) and bench.must_spawn(gpus=8, environ={"HOME": "/"})
    assert not bench.must_spawn(gpus=1, environ={})
    assert not bench.must_spawn(gpus=2, environ={"WORLD_SIZE": "2", "RANK": "0"})     # already under a launcher
    cmd = dp.rank_launch_command(4, "bench.py", ["--gpus", "4", "--steps", "3"], port=29999)
    assert cmd[1:] == ["-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=4", "--master-addr", "127.0.0.1",
                       "--master-port", "29999", "bench.py", "--gpus", "4", "--steps", "3"]
