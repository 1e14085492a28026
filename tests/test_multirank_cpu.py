"""World-size-2 run of the benchmark's multi-rank host logic on CPU (gloo): the path shards token rows
across ranks with replicated weights and no collective on the data path, and the slowest rank decides
the reported time.  Two processes each take their shard of a small batch through the CPU oracle; the
shards put together must equal the oracle on the whole batch, and the time reduction must be the maximum."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

ROWS_PER_RANK = 96


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import oracle
    import workload

    spec = workload.LinearSpec("mr", 1024, 128, workload.DIST_NORMAL, 21, 0)
    W, b = spec.weight(), spec.bias()                            # replicated: every rank derives the same weights
    prep = oracle.prepare_weights(W, oracle.smooth_factors(spec.x_calib(64), W), None)
    row0 = bench.rank_row0(rank, ROWS_PER_RANK)
    y = oracle.w4a4_linear(spec.x_rows(row0, ROWS_PER_RANK), prep, b, 0)["y"]
    np.save(os.path.join(out_dir, f"y{rank}.npy"), y)
    # the slowest rank decides: rank r pretends to have taken 10 + 5 r milliseconds
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")
    np.save(os.path.join(out_dir, f"ms{rank}.npy"), np.array([ms, row0]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_rows_and_take_the_slowest_time(tmp_path):
    import bench
    import oracle
    import workload

    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    spec = workload.LinearSpec("mr", 1024, 128, workload.DIST_NORMAL, 21, 0)
    W, b = spec.weight(), spec.bias()
    prep = oracle.prepare_weights(W, oracle.smooth_factors(spec.x_calib(64), W), None)
    whole = oracle.w4a4_linear(spec.x_rows(0, world * ROWS_PER_RANK), prep, b, 0)["y"]
    parts = [np.load(tmp_path / f"y{r}.npy") for r in range(world)]
    assert np.array_equal(np.concatenate(parts, axis=0), whole)         # row sharding needs no exchange
    for r in range(world):
        ms, row0 = np.load(tmp_path / f"ms{r}.npy")
        assert ms == 15.0 and row0 == r * ROWS_PER_RANK                  # every rank reports the maximum
    assert bench.max_over_ranks(7.5, None, "cpu") == 7.5
    assert abs(bench.whole_job_value(2, 1e12, 1000.0) - 2.0) < 1e-12     # 2 ranks x 1 Tera-op in 1 s = 2 TOPS
