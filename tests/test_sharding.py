"""The host-side plumbing of the N > 1 path on CPU: the partition helper (shard_range), the
throughput bookkeeping and the MAX reduction of the timing over two gloo ranks.

What this file does NOT show: anything about the CUDA path.  In the two-rank test both the
sharded and the unsharded results come from the CPU oracle; it checks only that the partition
covers every segment exactly once and that no payload has to be exchanged.  The device path on
several GPUs is `bench.py --gpus N`."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_28115_b200 import sharding
from paper_2605_28115_b200 import workloads as W


def test_shard_range_partitions():
    for n in range(0, 40):
        for world in range(1, 9):
            spans = [sharding.shard_range(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        sharding.shard_range(4, 2, 2)


def test_job_throughput():
    assert sharding.job_throughput_gbs(2_000_000_000, 4, 1.0) == pytest.approx(8000.0)
    assert sharding.max_over_ranks(3.5) == 3.5  # no process group: identity


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    import oracle

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = W.C3.replace(n_seg=5, n_layers=2)
    b, e = sharding.shard_range(wl.n_seg, world, rank)
    s = W.scores(wl)[b:e]
    o = oracle.default
    keep = o.select(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
    idx = o.seq_indices(keep, wl.seq_len, wl.text_before, wl.n)
    np.save(os.path.join(out_dir, f"idx_{rank}.npy"), idx)
    slowest = sharding.max_over_ranks(10.0 + rank)  # pretend rank r needed 10 + r ms
    assert slowest == 10.0 + world - 1
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_unsharded_result(tmp_path):
    import oracle

    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    wl = W.C3.replace(n_seg=5, n_layers=2)
    o = oracle.default
    keep = o.select(W.scores(wl), wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
    want = o.seq_indices(keep, wl.seq_len, wl.text_before, wl.n)
    got = np.concatenate([np.load(tmp_path / f"idx_{r}.npy") for r in range(world)])
    assert np.array_equal(got, want)
