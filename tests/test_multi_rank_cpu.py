"""The N > 1 path on CPU: two gloo ranks, work assignment and the max-over-ranks timing reduction.

Nothing on the data path is exchanged between ranks (replicas of the net, inputs sharded), so what there
is to test without GPUs is the host logic: the shards are disjoint and cover the job, and every rank
reports the same whole-job throughput, computed from the slowest rank's time."""
import os
import socket

import numpy as np
import pytest

from paper_2104_11805_b200 import shard


def test_split_inputs_is_a_balanced_partition():
    for n in (0, 1, 7, 60000, 60001):
        for world in (1, 2, 3, 8):
            parts = [shard.split_inputs(n, r, world) for r in range(world)]
            assert parts[0][0] == 0 and sum(c for _, c in parts) == n
            for (s0, c0), (s1, _) in zip(parts, parts[1:]):
                assert s0 + c0 == s1
            sizes = [c for _, c in parts]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    assert [shard.rank_inputs(r, 4, 100) for r in range(4)] == [(0, 100), (100, 100), (200, 100), (300, 100)]
    with pytest.raises(ValueError):
        shard.split_inputs(10, 2, 2)


def _worker(rank, world, port, out_dir):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import gen
        spec = gen.CFG1_INF
        start, count = shard.rank_inputs(rank, world, 5)
        x = gen.inputs(spec, count, start=start)                   # this rank's inputs of the job's input stream
        local_ms = 10.0 * (rank + 1)                               # rank 1 is the slow one
        value, ms = shard.job_throughput(1000.0, local_ms, world)
        np.save(os.path.join(out_dir, f"x{rank}.npy"), x)
        np.save(os.path.join(out_dir, f"v{rank}.npy"), np.array([value, ms, start, count]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_inputs_and_agree_on_the_job_throughput(tmp_path):
    mp = pytest.importorskip("torch.multiprocessing")
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    import gen
    v = [np.load(tmp_path / f"v{r}.npy") for r in range(2)]
    x = [np.load(tmp_path / f"x{r}.npy") for r in range(2)]
    assert v[0][0] == v[1][0] == pytest.approx(2 * 1000.0 / 20e-3) and v[0][1] == v[1][1] == 20.0
    assert (v[0][2], v[0][3], v[1][2], v[1][3]) == (0, 5, 5, 5)
    whole = gen.inputs(gen.CFG1_INF, 10)
    assert np.array_equal(np.concatenate(x), whole)                # disjoint shards that cover the job's inputs
