"""The multi-GPU path is batch replication/splitting with no data-path collective; its host
logic (slab ownership, max-over-ranks timing, aggregate rate) runs here as two gloo ranks on CPU."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2608_20725_b200 import replicas, workloads

DIMS = dict(N=5, C=3, H=8, W=7, Co=4, Kh=3, Kw=3, stride=1, pad=1)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        layer = workloads.Layer("t", **DIMS, seed=5, x_dist="normal01", f_dist="he_normal")
        x, f = workloads.make_inputs(layer)           # every rank draws the same tensors from the seed
        b, e = replicas.batch_slice(DIMS["N"], rank, world)
        y, _ = oracle.conv_im2win_range(x.numpy(), f.numpy(), DIMS, b, e)   # this rank's slab only
        np.save(os.path.join(out_dir, f"y{rank}.npy"), y)
        # timing: each rank reports a different time; all must see the maximum
        t = replicas.max_over_ranks([10.0 + rank, 5.0 - rank])
        np.save(os.path.join(out_dir, f"t{rank}.npy"), np.array(t))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_split_the_batch_without_exchange(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    layer = workloads.Layer("t", **DIMS, seed=5, x_dist="normal01", f_dist="he_normal")
    x, f = workloads.make_inputs(layer)
    want, _ = oracle.conv_im2win(x.numpy(), f.numpy(), DIMS)
    got = np.concatenate([np.load(tmp_path / f"y{r}.npy") for r in range(world)], axis=0)
    assert np.array_equal(got, want)
    for r in range(world):
        assert np.load(tmp_path / f"t{r}.npy").tolist() == [11.0, 5.0]


@pytest.mark.parametrize("n,world", [(128, 8), (5, 2), (3, 4), (0, 3), (7, 7)])
def test_batch_slices_partition_the_batch(n, world):
    cover = []
    for r in range(world):
        b, e = replicas.batch_slice(n, r, world)
        assert 0 <= b <= e <= n and e - b in (n // world, n // world + 1)
        cover.extend(range(b, e))
    assert cover == list(range(n))


def test_whole_job_rate_and_identity_without_group():
    assert replicas.whole_job_rate(100.0, 8, 50.0) == pytest.approx(16000.0)
    assert replicas.max_over_ranks([1.0, 2.0]) == [1.0, 2.0]
