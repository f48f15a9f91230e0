"""Token-sharded forward (Sec. 4.3) over a 2-rank gloo group on CPU.

The CUDA kernels cannot run here, so each rank uses the fp64 oracle as the stand-in for the two
halves of the library (state of the local K/V tokens; apply to the local Q tokens); the sharding
arithmetic, the driver and the collective are the real ones."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2409_02097_b200 import sharding

EPS = 1e-6


def test_token_shard_covers_the_range_without_overlap():
    for n in (0, 1, 7, 64, 1000, 524288):
        for world in (1, 2, 3, 8):
            runs = [sharding.token_shard(n, r, world) for r in range(world)]
            assert runs[0][0] == 0 and runs[-1][1] == n
            for (a0, a1), (b0, b1) in zip(runs[:-1], runs[1:]):
                assert a1 == b0 and a0 <= a1
            lengths = [b - a for a, b in runs]
            assert max(lengths) - min(lengths) <= 1
    with pytest.raises(ValueError):
        sharding.token_shard(10, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, n, d, slabs, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rng = np.random.default_rng(123)                       # same full tensors on every rank
        q, k, v = (rng.standard_normal((slabs, n, d)) for _ in range(3))
        b, e = sharding.token_shard(n, rank, world)
        box = {}

        def state_fn(k_, v_):
            S, z = oracle.state(k_, v_)
            box["buf"] = torch.from_numpy(np.concatenate([S.reshape(slabs, -1), z], axis=1))
            return box["buf"]

        def allreduce_sum(buf):
            dist.all_reduce(buf, op=dist.ReduceOp.SUM)

        def apply_fn(q_):
            buf = box["buf"].numpy()
            S = buf[:, :d * d].reshape(slabs, d, d)
            z = buf[:, d * d:]
            return oracle.apply(q_, S, z, EPS)

        y_local = sharding.sharded_forward(state_fn, apply_fn, allreduce_sum,
                                           q[:, b:e], k[:, b:e], v[:, b:e])
        np.save(os.path.join(out_dir, f"y_{rank}.npy"), y_local)
        if rank == 0:
            np.save(os.path.join(out_dir, "y_full.npy"), oracle.linear(q, k, v, EPS))
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("n", [257, 64])
def test_two_rank_sharded_forward_equals_the_unsharded_one(tmp_path, n):
    world, d, slabs = 2, 16, 3
    mp.spawn(_rank_main, args=(world, _free_port(), n, d, slabs, str(tmp_path)), nprocs=world, join=True)
    parts = [np.load(tmp_path / f"y_{r}.npy") for r in range(world)]
    y = np.concatenate(parts, axis=1)
    ref = np.load(tmp_path / "y_full.npy")
    assert y.shape == ref.shape
    np.testing.assert_allclose(y, ref, rtol=1e-12, atol=1e-14)
