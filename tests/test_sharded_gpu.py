"""Token-sharded forward on one GPU: two shards of the tokens are processed one after the other
through linfusion_attn_state / _state_buffer / _apply, their states summed by hand in between
(the stand-in for the all-reduce between devices), and compared with the oracle on the whole N."""
import numpy as np
import pytest
import torch

from paper_2409_02097_b200 import attn, sharding, workloads as wl

from _util import EPS, assert_parity, oracle_y

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dims,variant", [((2, 5, 9000, 64), "stream"), ((1, 4, 3001, 64), "split"),
                                          ((2, 3, 1500, 40), "split"), ((1, 2, 700, 160), "split")],
                         ids=lambda x: str(x))
def test_two_token_shards_summed_state(dims, variant):
    B, H, N, d = dims
    q, k, v = wl.make_small(B, H, N, d, seed=77, device="cuda")
    ref = oracle_y(q, k, v)
    world = 2
    shards = []
    for r in range(world):
        b, e = sharding.token_shard(N, r, world)
        sh = sharding.TokenShardedAttention(B, H, e - b, d, eps=EPS, variant=variant)
        qs, ks, vs = (t[:, :, b:e].contiguous() for t in (q, k, v))
        sh.op.state(ks, vs)
        shards.append((sh, qs, b, e))
    torch.cuda.synchronize()
    total = sum(sh.state.clone() for sh, *_ in shards)          # what the all-reduce would leave
    y = torch.empty_like(q)
    for sh, qs, b, e in shards:
        sh.state.copy_(total)
        y[:, :, b:e] = sh.op.apply(qs)
    torch.cuda.synchronize()
    for sh, *_ in shards:
        assert sh.op.status() == attn.OK
        sh.close()
    assert_parity(y, ref, f"sharded {dims} {variant}")


@pytest.mark.parametrize("dims,variant,world", [((2, 5, 9000, 64), "stream", 2), ((1, 4, 3001, 64), "split", 3),
                                                ((1, 2, 700, 160), "split", 2), ((1, 3, 20000, 64), "stream", 8)],
                         ids=lambda x: str(x))
def test_apply_sums_the_shards_states_itself(dims, variant, world):
    """apply_peers on one GPU: the shards' handles stand in for the ranks, their state buffers for
    the peers' memory.  Every shard is given the same list, so every shard sums in the same order."""
    B, H, N, d = dims
    q, k, v = wl.make_small(B, H, N, d, seed=79, device="cuda")
    ref = oracle_y(q, k, v)
    ops, cuts = [], []
    for r in range(world):
        b, e = sharding.token_shard(N, r, world)
        op = attn.LinFusionAttention(B, H, e - b, d, eps=EPS, variant=variant)
        op.state(k[:, :, b:e].contiguous(), v[:, :, b:e].contiguous())
        ops.append(op)
        cuts.append((b, e))
    torch.cuda.synchronize()                                    # the stand-in for the cross-rank barrier
    ptrs = [op.state_buffer()[0] for op in ops]
    y = torch.empty_like(q)
    for op, (b, e) in zip(ops, cuts):
        y[:, :, b:e] = op.apply_peers(q[:, :, b:e].contiguous(), ptrs)
    torch.cuda.synchronize()
    assert_parity(y, ref, f"apply_peers {dims} {variant} x{world}")
    # the local states were left alone, and their sum is the whole sequence's state
    S_sum = sum(op.read_state()[0] for op in ops)
    full = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant=variant)
    full.forward(q, k, v)
    S_full, _ = full.read_state()
    assert np.linalg.norm(S_sum - S_full) <= 1e-5 * np.linalg.norm(S_full)
    with pytest.raises(attn.LinFusionError):
        ops[0].apply_peers(q[:, :, cuts[0][0]:cuts[0][1]].contiguous(), [])
    with pytest.raises(attn.LinFusionError):
        ops[0].apply_peers(q[:, :, cuts[0][0]:cuts[0][1]].contiguous(), ptrs * 9)
    for op in ops + [full]:
        assert op.status() == attn.OK
        op.close()


def test_single_rank_sharded_forward_equals_forward_bits():
    """World size 1: state + apply is the same computation as forward."""
    B, H, N, d = 2, 4, 5000, 64
    q, k, v = wl.make_small(B, H, N, d, seed=78, device="cuda")
    sh = sharding.TokenShardedAttention(B, H, N, d, eps=EPS)
    y1 = sh.forward(q, k, v)
    op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant="stream")
    y2 = op.forward(q, k, v)
    torch.cuda.synchronize()
    assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))
    sh.close()
    op.close()


def test_cluster_handles_refuse_to_be_split():
    op = attn.LinFusionAttention(1, 2, 128, 64, variant="cluster")
    q, k, v = wl.make_small(1, 2, 128, 64, seed=1, device="cuda")
    with pytest.raises(attn.LinFusionError) as e:
        op.state(k, v)
    assert e.value.code == attn.ERR_UNSUPPORTED
    op.close()
