"""world_size-2 gloo test of the data-parallel bookkeeping (CPU only)."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp

from paper_2512_14090_b200.sharding import shard_bounds, reduce_counts


def test_shard_bounds_partition():
    for n in (0, 1, 7, 10000, 10001):
        for w in (1, 2, 3, 8):
            spans = [shard_bounds(n, r, w) for r in range(w)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, ret):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    preds = np.random.default_rng(0).integers(0, 10, (5, 1001))      # same on every rank
    labels = np.random.default_rng(1).integers(0, 10, 1001)
    lo, hi = shard_bounds(1001, rank, world)
    local = (preds[:, lo:hi] == labels[None, lo:hi]).sum(axis=1)
    counts, total, acc = reduce_counts(local, hi - lo)
    ret[rank] = (counts.tolist(), total, acc.tolist())
    dist.destroy_process_group()


def test_two_rank_count_reduction_matches_single_process():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(2, port, ret), nprocs=2, join=True)
    preds = np.random.default_rng(0).integers(0, 10, (5, 1001))
    labels = np.random.default_rng(1).integers(0, 10, 1001)
    want = (preds == labels[None, :]).sum(axis=1)
    for r in (0, 1):
        counts, total, acc = ret[r]
        assert counts == want.tolist() and total == 1001
        assert np.allclose(acc, want / 1001.0)


def test_reduce_counts_without_process_group():
    counts, total, acc = reduce_counts(np.asarray([3, 4]), 8)
    assert counts.tolist() == [3, 4] and total == 8 and acc.tolist() == [0.375, 0.5]
