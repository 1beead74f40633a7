"""The N > 1 path on CPU: two `gloo` ranks. The quantized linear shards by rows with replicated
parameters and has no exchange step, so what needs checking is the host logic around it: each
rank draws its own batch, the shards together are the global batch, results need no collective,
the step time is the maximum over ranks and only rank 0 reports."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _layer():
    import workloads as wl
    return wl.scaled(wl.config_layers(2)[2], batch=3, P=21, K=64, N=48)     # fc1 + GELU, tiny


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import oracle
    import workloads as wl
    from layer_setup import prepare
    L = _layer()
    par = prepare(L, samples=4, gps_n=32)                       # replicated parameters: same on every rank
    step = bench.rank_step(rank, 0, world)
    X, pos = wl.activations(L, step), wl.positions(L, step)
    ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], L.bits, L.act)
    # a rank-dependent fake step time: the job's time must be the slowest rank's
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
    # gather only to let the test compare; the benchmark itself gathers nothing
    ys = [torch.empty(L.M, L.N, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(ys, torch.from_numpy(ref["Y"]))
    xs = [torch.empty(L.M, L.K, dtype=torch.float32) for _ in range(world)]
    dist.all_gather(xs, torch.from_numpy(np.ascontiguousarray(X)))
    if rank == 0:
        np.savez(os.path.join(out_dir, "r0.npz"), ms=ms, Y=torch.cat(ys).numpy(), X=torch.cat(xs).numpy(),
                 tops=bench.whole_job_tops(world, L.ops, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_rows_without_a_collective(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    got = np.load(tmp_path / "r0.npz")
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import bench
    import oracle
    import workloads as wl
    from layer_setup import prepare
    L = _layer()
    par = prepare(L, samples=4, gps_n=32)
    # the global batch in one process: the ranks' batches stacked
    Xg = np.concatenate([wl.activations(L, bench.rank_step(r, 0, world)) for r in range(world)])
    pg = np.concatenate([wl.positions(L, bench.rank_step(r, 0, world)) for r in range(world)])
    np.testing.assert_array_equal(got["X"], Xg)
    assert not np.array_equal(Xg[:L.M], Xg[L.M:])                # the ranks drew different batches
    ref = oracle.qlinear(Xg, pg, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], L.bits, L.act)
    np.testing.assert_array_equal(got["Y"], ref["Y"])            # rows are independent: shards == whole
    assert float(got["ms"]) == 15.0                              # max over ranks
    assert float(got["tops"]) == pytest.approx(world * L.ops / 15e-3 / 1e12)


def test_rank_steps_partition_the_global_batches():
    import bench
    for world in (1, 2, 4, 8):
        seen = [bench.rank_step(r, s, world) for s in range(3) for r in range(world)]
        assert sorted(seen) == list(range(3 * world))
