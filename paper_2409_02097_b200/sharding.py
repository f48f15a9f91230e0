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
    tensor view without wrapping raw pointers.
    """

    def __init__(self, B, H, n_local, d, group=None, phi=0, eps=1e-6, device=0, variant="auto"):
        import torch
        from . import attn
        if variant == "auto":
            variant = "stream" if d == 64 else "split"
        self.group = group
        self.op = attn.LinFusionAttention(B, H, n_local, d, phi=phi, eps=eps, device=device,
                                          variant=variant)
        sm = torch.cuda.get_device_properties(device).multi_processor_count
        nbytes = attn.linfusion_attn_workspace_bytes(self.op.desc, sm)
        self._ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=f"cuda:{device}")
        off = (-self._ws.data_ptr()) % 256
        ws = self._ws[off:off + nbytes]
        self.op.set_workspace(ws)
        ptr, n = self.op.state_buffer()
        start = ptr - ws.data_ptr()
        assert 0 <= start and start + 4 * n <= nbytes
        self.state = ws[start:start + 4 * n].view(torch.float32)

    def forward(self, q, k, v, y=None):
        import torch.distributed as dist

        def state_fn(k_, v_):
            self.op.state(k_, v_)
            return self.state

        def allreduce_sum(buf):
            if dist.is_available() and dist.is_initialized() and dist.get_world_size(self.group) > 1:
                dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=self.group)

        return sharded_forward(state_fn, lambda q_: self.op.apply(q_, y), allreduce_sum, q, k, v)

    def forward_peers(self, q, k, v, peer_state_ptrs, barrier: Callable[[], None], y=None):
        """The same layer with the cross-device sum done by the apply step itself instead of an
        all-reduce: ``peer_state_ptrs`` lists, in rank order, device addresses of every rank's
        state buffer that this device can load from (this rank's own is
        ``self.op.state_buffer()[0]``; peers' come from whatever maps their memory here — peer
        access within a process, CUDA IPC or symmetric memory across processes).  ``barrier()``
        must return only when every rank's state kernel has completed (it is called between the
        two halves, and once more after the apply so that no rank overwrites a state that a peer
        is still reading)."""
        self.op.state(k, v)
        barrier()
        out = self.op.apply_peers(q, peer_state_ptrs, y)
        barrier()
        return out

    def close(self):
        self.op.close()
