"""Token-sharded (sequence-parallel) forward across devices — the distributed inference of Sec. 4.3.

Every rank owns a contiguous run of the N tokens of Q, K, V and Y.  Each rank builds the state
S | z of its own K/V tokens, the ranks sum their states (one all-reduce of B*H*d*(d+1) floats,
whatever N is — the "constant communication" the paper points out), and each rank applies the
summed state to its own Q tokens.  The arithmetic is in the CUDA library (``attn``); this module
only cuts the token range and calls the collective.
"""
from __future__ import annotations

from typing import Callable, Tuple


def token_shard(n_tokens: int, rank: int, world_size: int) -> Tuple[int, int]:
    """[begin, end) of the tokens owned by ``rank``: contiguous runs whose lengths differ by at
    most one, the first ``n_tokens % world_size`` ranks holding the longer ones."""
    if world_size <= 0 or not 0 <= rank < world_size or n_tokens < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_tokens, world_size)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def sharded_forward(state_fn: Callable, apply_fn: Callable, allreduce_sum: Callable, q, k, v):
    """One layer on one rank: ``state_fn(k, v)`` returns this rank's state buffer (any object the
    collective accepts), ``allreduce_sum(buf)`` sums it over ranks in place, ``apply_fn(q)``
    returns Y for the local tokens.  The split into three callables keeps this module free of
    arithmetic, so the same driver serves the CUDA library and the tests' CPU stand-in."""
    buf = state_fn(k, v)
    allreduce_sum(buf)
    return apply_fn(q)


class TokenShardedAttention:
    """The CUDA library on one rank of a ``torch.distributed`` process group (NCCL).

    ``n_local`` is this rank's token count (``token_shard``).  The handle's workspace is a torch
    tensor lent to the library, so that the state buffer can be handed to ``all_reduce`` as a
    tensor view without wrapping raw pointers.  With ``symmetric=True`` that tensor comes from
    ``torch.distributed._symmetric_memory`` and is mapped into every rank of the group, which lets
    ``forward_symmetric`` hand the peers' state buffers to the apply step (plain loads over
    NVLink; no multicast of any kind is used here).

    ``op`` may be supplied by the caller (anything with the binding's ``state`` / ``apply`` /
    ``apply_peers`` / ``set_workspace`` / ``state_buffer`` / ``desc`` members); the tests drive the
    control flow below with a stand-in on CPU.
    """

    def __init__(self, B, H, n_local, d, group=None, phi=0, eps=1e-6, device=0, variant="auto",
                 dtype="bf16", symmetric=False, op=None, workspace_bytes=None, sm_count=None):
        import torch
        if variant == "auto":
            variant = "stream" if d == 64 else "split"
        self.group = group
        self.symmetric = bool(symmetric)
        self._symm = None
        if op is None:
            from . import attn
            op = attn.LinFusionAttention(B, H, n_local, d, phi=phi, eps=eps, device=device,
                                         variant=variant, dtype=dtype)
            if sm_count is None:
                sm_count = torch.cuda.get_device_properties(device).multi_processor_count
            workspace_bytes = attn.linfusion_attn_workspace_bytes(op.desc, sm_count)
            dev = f"cuda:{device}"
        else:
            dev = getattr(op, "device", "cpu")
        self.op = op
        nbytes = int(workspace_bytes)
        if self.symmetric:
            import torch.distributed as dist
            import torch.distributed._symmetric_memory as symm_mem
            self._ws = symm_mem.empty(nbytes + 256, dtype=torch.uint8, device=dev)
            pg = group if group is not None else dist.distributed_c10d._get_default_group()
            self._symm = symm_mem.rendezvous(self._ws, pg.group_name)
        else:
            self._ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=dev)
        off = (-self._ws.data_ptr()) % 256
        ws = self._ws[off:off + nbytes]
        self.op.set_workspace(ws)
        ptr, n = self.op.state_buffer()
        start = ptr - ws.data_ptr()
        assert 0 <= start and start + 4 * n <= nbytes
        self.state = ws[start:start + 4 * n].view(torch.float32)
        self._state_offset = off + start          # of the state buffer inside the (symmetric) allocation

    def peer_state_ptrs(self):
        """Device addresses of every rank's state buffer, in rank order (``symmetric=True`` only):
        the same offset inside each rank's mapping of the symmetric allocation.  Valid because
        every rank builds the same handle (same shape, same workspace layout, same alignment of a
        fresh symmetric allocation)."""
        if self._symm is None:
            raise RuntimeError("peer_state_ptrs() needs symmetric=True")
        return [int(p) + self._state_offset for p in self._symm.buffer_ptrs]

    def forward(self, q, k, v, y=None, events=None):
        """state -> all-reduce of S | z -> apply.  ``events`` (optional, four CUDA events) are
        recorded before the state half, before and after the exchange, and after the apply half."""
        import torch.distributed as dist

        def rec(i):
            if events is not None:
                events[i].record()

        def state_fn(k_, v_):
            rec(0)
            self.op.state(k_, v_)
            rec(1)
            return self.state

        def allreduce_sum(buf):
            if dist.is_available() and dist.is_initialized() and dist.get_world_size(self.group) > 1:
                dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=self.group)
            rec(2)

        def apply_fn(q_):
            out = self.op.apply(q_, y)
            rec(3)
            return out

        return sharded_forward(state_fn, apply_fn, allreduce_sum, q, k, v)

    def forward_peers(self, q, k, v, peer_state_ptrs, barrier: Callable[[], None], y=None, events=None):
        """The same layer with the cross-device sum done by the apply step itself instead of an
        all-reduce: ``peer_state_ptrs`` lists, in rank order, device addresses of every rank's
        state buffer that this device can load from (this rank's own is
        ``self.op.state_buffer()[0]``; peers' come from whatever maps their memory here — peer
        access within a process, CUDA IPC or symmetric memory across processes).  ``barrier()``
        must return only when every rank's state kernel has completed (it is called between the
        two halves, and once more after the apply so that no rank overwrites a state that a peer
        is still reading)."""
        def rec(i):
            if events is not None:
                events[i].record()
        rec(0)
        self.op.state(k, v)
        rec(1)
        barrier()
        rec(2)
        out = self.op.apply_peers(q, peer_state_ptrs, y)
        barrier()
        rec(3)
        return out

    def forward_symmetric(self, q, k, v, y=None, events=None):
        """``forward_peers`` over the symmetric allocation: the peers' addresses come from the
        rendezvous, the two barriers are the symmetric-memory barrier, enqueued on the current
        stream (every rank runs one process and one GPU, so the barrier's kernels of all ranks
        are resident at the same time)."""
        if self._symm is None:
            raise RuntimeError("forward_symmetric() needs symmetric=True")
        calls = [0]

        def barrier():
            self._symm.barrier(channel=calls[0] % 2)
            calls[0] += 1

        return self.forward_peers(q, k, v, self.peer_state_ptrs(), barrier, y, events)

    def close(self):
        self.op.close()
