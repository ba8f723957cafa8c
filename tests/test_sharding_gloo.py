"""The N>1 path on CPU: two gloo ranks shard the rows of one batch, each evaluates its shard with the
CPU oracle (standing in for its GPU), and the reassembled result equals the unsharded one; the
timing reduction returns the slowest rank."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

from paper_2311_06281_b200 import sharding, workloads


def test_shard_rows_partitions_exactly():
    for rows in (0, 1, 7, 16384, 16385):
        for world in (1, 2, 3, 8):
            got = [sharding.shard_rows(rows, world, r) for r in range(world)]
            assert got[0][0] == 0 and sum(c for _, c in got) == rows
            for (f0, c0), (f1, _) in zip(got, got[1:]):
                assert f0 + c0 == f1
            assert max(c for _, c in got) - min(c for _, c in got) <= 1
    with pytest.raises(ValueError):
        sharding.shard_rows(4, 2, 2)


def _worker(rank, world, port, outdir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    from oracle import heinsen_oracle
    r, w, _ = sharding.init_from_env("gloo")
    assert (r, w) == (rank, world)
    t = workloads.make(2, rows=10, n=257).tensors
    first, count = sharding.shard_rows(10, world, rank)
    sl = slice(first, first + count)
    lx, _ = heinsen_oracle.scan_log(t["log_a"][sl], t["log_b"][sl], t["log_x0"][sl], nthreads=1)
    np.save(os.path.join(outdir, f"part{rank}.npy"), lx)
    sharding.barrier()
    slowest = sharding.max_over_ranks(1.0 + rank)
    total = sharding.sum_over_ranks(float(count))
    assert slowest == float(world) and total == 10.0
    torch.distributed.destroy_process_group()


def test_two_gloo_ranks_shard_rows_without_a_collective_in_the_data_path(tmp_path, oracle):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    t = workloads.make(2, rows=10, n=257).tensors
    whole, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    parts = np.concatenate([np.load(tmp_path / f"part{r}.npy") for r in range(2)], axis=0)
    np.testing.assert_array_equal(parts, whole)
