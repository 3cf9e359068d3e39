"""The multi-GPU path has no data exchange; what it has -- batch sharding and the max-time /
sum-bytes bookkeeping of the benchmark -- is tested here with two gloo ranks on the CPU."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1905_10830_b200 import sharding


def test_shard_range_covers_the_batch_without_overlap():
    for total in (0, 1, 7, 64, 4096, 4099):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                first, count = sharding.shard_range(total, r, world)
                seen.extend(range(first, first + count))
                assert count in (total // world, total // world + 1)
            assert seen == list(range(total))
    with pytest.raises(ValueError):
        sharding.shard_range(8, 2, 2)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r codes (r + 1) GB in (10 + 5 r) ms
        total_bytes, ms = sharding.aggregate((rank + 1) * 1e9, 10.0 + 5.0 * rank)
        out[rank] = (total_bytes, ms)
    finally:
        dist.destroy_process_group()


def test_aggregate_takes_max_time_and_sum_of_bytes_over_two_gloo_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    assert dict(out) == {0: (3e9, 15.0), 1: (3e9, 15.0)}


def test_aggregate_without_a_process_group_is_the_identity():
    assert sharding.aggregate(5.0, 2.0) == (5.0, 2.0)


def _state_of(rank: int):
    import numpy as np
    rng = np.random.default_rng(100 + rank)
    x = rng.standard_normal((50 + 10 * rank, 6))            # (samples, channels) held by this rank
    return x.shape[0], x.sum(axis=0), x.T @ x, x


def _fit_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        count, s1, s2, _ = _state_of(rank)
        out[rank] = sharding.merge_fit_state(count, s1, s2)
    finally:
        dist.destroy_process_group()


def test_fit_state_merges_by_one_sum_over_two_gloo_ranks():
    import numpy as np
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    procs = [ctx.Process(target=_fit_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    allx = np.concatenate([_state_of(r)[3] for r in range(2)])
    for r in range(2):
        count, s1, s2 = out[r]
        assert count == allx.shape[0]
        assert np.allclose(s1, allx.sum(axis=0), rtol=1e-13, atol=1e-13)
        assert np.allclose(s2, allx.T @ allx, rtol=1e-13, atol=1e-13)
        # the merged state gives the covariance of all samples
        m = float(count)
        cov = (s2 - np.outer(s1, s1) / m) / (m - 1.0)
        assert np.allclose(cov, np.cov(allx.T), rtol=1e-10, atol=1e-12)
    # no process group: the local state comes back unchanged
    count, s1, s2, _ = _state_of(0)
    c2, a, b = sharding.merge_fit_state(count, s1, s2)
    assert c2 == count and np.array_equal(a, s1) and np.array_equal(b, s2)
