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


class _StubOp:
    """CPU stand-in for the binding's handle object, with the same members the sharded driver
    uses: the fp64 oracle does both halves, the state lives (as fp32, like the library's) at a
    fixed offset inside the workspace tensor that the driver lends."""
    STATE_OFFSET = 1024
    device = "cpu"

    def __init__(self, slabs, d, log):
        self.slabs, self.d, self.log = slabs, d, log
        self.floats = slabs * d * (d + 1)
        self.ws = None

    def workspace_bytes(self):
        return self.STATE_OFFSET + 4 * self.floats + 64

    def set_workspace(self, tensor):
        assert tensor.data_ptr() % 256 == 0 and tensor.numel() >= self.workspace_bytes()
        self.ws = tensor
        self.log.append("set_workspace")

    def _state_view(self):
        return self.ws[self.STATE_OFFSET:self.STATE_OFFSET + 4 * self.floats].view(torch.float32)

    def state_buffer(self):
        return self.ws.data_ptr() + self.STATE_OFFSET, self.floats

    def state(self, k, v):
        S, z = oracle.state(k, v)
        buf = np.concatenate([S.reshape(self.slabs, -1), z], axis=1).astype(np.float32)
        self._state_view().copy_(torch.from_numpy(buf.reshape(-1)))
        self.log.append("state")

    def _apply_from(self, q, flat):
        buf = np.asarray(flat, dtype=np.float64).reshape(self.slabs, -1)
        d = self.d
        return oracle.apply(q, buf[:, :d * d].reshape(self.slabs, d, d), buf[:, d * d:], EPS)

    def apply(self, q, y=None):
        self.log.append("apply")
        return self._apply_from(q, self._state_view().numpy())

    def apply_peers(self, q, ptrs, y=None):
        import ctypes
        self.log.append("apply_peers")
        total = np.zeros(self.floats, dtype=np.float32)
        for p in ptrs:                                   # in list order, in fp32, like the kernel
            total = total + np.ctypeslib.as_array((ctypes.c_float * self.floats).from_address(p))
        return self._apply_from(q, total)

    def close(self):
        self.log.append("close")


def _driver_rank_main(rank, world, port, n, d, slabs, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rng = np.random.default_rng(321)
        q, k, v = (rng.standard_normal((slabs, n, d)) for _ in range(3))
        b, e = sharding.token_shard(n, rank, world)
        log = []
        op = _StubOp(slabs, d, log)
        sh = sharding.TokenShardedAttention(1, slabs, e - b, d, op=op, workspace_bytes=op.workspace_bytes())
        assert log == ["set_workspace"]
        assert sh.state.dtype == torch.float32 and sh.state.numel() == op.floats
        assert sh.state.data_ptr() == op.state_buffer()[0]          # the view IS the library's buffer
        y_local = sh.forward(q[:, b:e], k[:, b:e], v[:, b:e])
        assert log == ["set_workspace", "state", "apply"]
        # after the exchange every rank holds the same, summed state
        gathered = [torch.empty_like(sh.state) for _ in range(world)]
        dist.all_gather(gathered, sh.state)
        assert all(torch.equal(g, gathered[0]) for g in gathered)
        np.save(os.path.join(out_dir, f"y_{rank}.npy"), y_local)
        if rank == 0:
            np.save(os.path.join(out_dir, "y_full.npy"), oracle.linear(q, k, v, EPS))
        sh.close()
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_rank_token_sharded_attention_control_flow(tmp_path):
    """TokenShardedAttention itself over gloo: workspace lending, the state view handed to the
    all-reduce, state -> all-reduce -> apply ordering."""
    world, n, d, slabs = 2, 301, 16, 3
    mp.spawn(_driver_rank_main, args=(world, _free_port(), n, d, slabs, str(tmp_path)), nprocs=world, join=True)
    y = np.concatenate([np.load(tmp_path / f"y_{r}.npy") for r in range(world)], axis=1)
    ref = np.load(tmp_path / "y_full.npy")
    np.testing.assert_allclose(y, ref, rtol=2e-5, atol=2e-6)      # the exchanged state is fp32


def test_forward_peers_keeps_its_two_barriers_around_the_peer_reads():
    """forward_peers with two ranks as two threads of one process (so that each can read the
    other's state buffer by address): state, barrier, apply_peers, barrier — the first barrier
    keeps a rank from reading a peer's state before it is complete, the second from overwriting
    its own while a peer still reads it."""
    import threading
    world, n, d, slabs = 2, 200, 8, 2
    rng = np.random.default_rng(7)
    q, k, v = (rng.standard_normal((slabs, n, d)) for _ in range(3))
    sync = threading.Barrier(world)
    ranks, outs, logs = [], [None] * world, [[] for _ in range(world)]
    for r in range(world):
        op = _StubOp(slabs, d, logs[r])
        b, e = sharding.token_shard(n, r, world)
        ranks.append((sharding.TokenShardedAttention(1, slabs, e - b, d, op=op, workspace_bytes=op.workspace_bytes()), b, e))
    ptrs = [sh.op.state_buffer()[0] for sh, _, _ in ranks]

    def run(r):
        sh, b, e = ranks[r]

        def barrier():
            logs[r].append("barrier")
            sync.wait(timeout=60)

        for _ in range(2):                               # two layers in a row reuse the buffers
            outs[r] = sh.forward_peers(q[:, b:e], k[:, b:e], v[:, b:e], ptrs, barrier)

    threads = [threading.Thread(target=run, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=120)
    for r in range(world):
        assert logs[r] == ["set_workspace"] + ["state", "barrier", "apply_peers", "barrier"] * 2
    y = np.concatenate(outs, axis=1)
    np.testing.assert_allclose(y, oracle.linear(q, k, v, EPS), rtol=2e-5, atol=2e-6)
    with pytest.raises(RuntimeError):
        ranks[0][0].peer_state_ptrs()                    # needs the symmetric allocation
