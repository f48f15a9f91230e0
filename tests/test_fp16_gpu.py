"""GPU parity with fp16 storage (the precision the paper's implementation runs in) against the fp64
oracle on the same fp16-rounded inputs.  fp16 carries three more mantissa bits than bf16, so the
gates of the bf16 tests hold with room to spare; what is specific to fp16 is range: z ~ N would
overflow the format as a tensor-core operand, so the library scales S | z by a power of two."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_02097_b200 import attn, workloads as wl

from _util import EPS, MAX_ABS_TOL, MEAN_ABS_TOL, REL_FRO_TOL, assert_parity, error_metrics, to_f64

pytestmark = pytest.mark.gpu


def make_fp16(B, H, N, d, seed):
    q, k, v = wl.make_small(B, H, N, d, seed=seed, device="cuda")
    return q.half(), k.half(), v.half()


def run_fp16(q, k, v, variant, **kw):
    B, H, N, d = q.shape
    op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant=variant, dtype="fp16", **kw)
    y = op.forward(q, k, v)
    torch.cuda.synchronize()
    assert op.status() == attn.OK
    assert y.dtype == torch.float16
    return y, op


CASES = [
    (2, 3, 1000, 64, ("split", "stream", "cluster")),
    (1, 2, 333, 40, ("split", "cluster")),
    (1, 4, 2500, 160, ("split",)),
    (1, 2, 129, 80, ("split", "cluster")),
    (1, 10, 70000, 64, ("auto", "stream", "split")),     # z ~ 8e4 > 65504: needs the operand scale
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(map(str, c[:4])))
def test_fp16_matches_oracle(case):
    B, H, N, d, variants = case
    q, k, v = make_fp16(B, H, N, d, seed=51)
    ref = oracle.linear(to_f64(q), to_f64(k), to_f64(v), EPS)
    for variant in variants:
        y, op = run_fp16(q, k, v, variant)
        max_abs, mean_abs, rel_fro = assert_parity(y, ref, f"fp16 {case[:4]}/{variant}->{op.variant}")
        # three more mantissa bits than bf16: the error must be clearly below the bf16 level (1.8e-3)
        assert rel_fro <= 1.0e-3, (variant, rel_fro)
        S, z = oracle.state(to_f64(k), to_f64(v))
        S_gpu, z_gpu = op.read_state()
        assert np.abs(z_gpu - z).max() <= 2e-3 * np.abs(z).max()
        assert np.linalg.norm(S_gpu - S) <= 5e-3 * np.linalg.norm(S)
        op.close()


def test_fp16_full_size_level_sampled_slabs():
    """N = 524 288: z ~ 6e5, ten times fp16's largest number."""
    shape = wl.find_shape("sdxl_16k_L1")
    q, k, v = (t.half() for t in wl.make_qkv(shape, seed=wl.BASE_SEED, device="cuda"))
    y, op = run_fp16(q, k, v, "auto")
    assert op.variant == "stream"
    assert torch.isfinite(y.view(-1)[::4097].float()).all()
    for b, h in [(0, 0), (shape.B - 1, shape.H - 1)]:
        ref = oracle.linear(to_f64(q[b, h]), to_f64(k[b, h]), to_f64(v[b, h]), EPS)
        assert_parity(y[b, h], ref, f"fp16 {shape.name}[{b},{h}]")
    op.close()


def test_fp16_unnormalized_and_token_major():
    B, H, N, d = 1, 4, 3000, 64
    q, k, v = make_fp16(B, H, N, d, seed=52)
    ref_un = oracle.linear_unnormalized(to_f64(q), to_f64(k), to_f64(v))
    for variant in ("split", "stream"):
        y, op = run_fp16(q, k, v, variant, normalize=False)
        scale = float(np.abs(ref_un).max())
        max_abs, mean_abs, rel_fro = error_metrics(y, ref_un)
        assert max_abs <= MAX_ABS_TOL * scale and mean_abs <= MEAN_ABS_TOL * scale and rel_fro <= REL_FRO_TOL, variant
        op.close()
    ref = oracle.linear(to_f64(q), to_f64(k), to_f64(v), EPS)
    tm = lambda t: t.permute(0, 2, 1, 3).contiguous()
    op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant="stream", layout="token_major", dtype="fp16")
    y_tm = op.forward(tm(q), tm(k), tm(v))
    torch.cuda.synchronize()
    assert_parity(y_tm.permute(0, 2, 1, 3), ref, "fp16 token-major")
    op.close()


def test_fp16_rejects_bf16_tensors():
    op = attn.LinFusionAttention(1, 1, 256, 64, dtype="fp16")
    x = torch.zeros((1, 1, 256, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ValueError):
        op.forward(x, x, x)
    op.close()


def test_fp16_host_buffers_no_alloc_and_peer_sum():
    B, H, N, d = 1, 4, 9000, 64
    q, k, v = make_fp16(B, H, N, d, seed=53)
    ref = oracle.linear(to_f64(q), to_f64(k), to_f64(v), EPS)
    # host-buffer forward
    op = attn.LinFusionAttention(B, H, N, d, eps=EPS, dtype="fp16")
    qh, kh, vh = q.cpu(), k.cpu(), v.cpu()
    yh = torch.empty_like(qh)
    op.forward_host(qh, kh, vh, yh)
    torch.cuda.synchronize()
    assert_parity(yh, ref, "fp16 forward_host")
    op.close()
    # allocation-free entry point
    y = torch.empty_like(q)
    desc = attn.make_desc(B, H, N, d, eps=EPS, dtype="fp16")
    attn.linfusion_attn_forward_noalloc(desc, q.data_ptr(), k.data_ptr(), v.data_ptr(), y.data_ptr(),
                                        torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert_parity(y, ref, "fp16 forward_noalloc")
    # token shards whose states the apply step sums itself (the operand scale follows the shard's N)
    from paper_2409_02097_b200 import sharding
    ops, cuts = [], []
    for r in range(3):
        b, e = sharding.token_shard(N, r, 3)
        o = attn.LinFusionAttention(B, H, e - b, d, eps=EPS, variant="stream", dtype="fp16")
        o.state(k[:, :, b:e].contiguous(), v[:, :, b:e].contiguous())
        ops.append(o)
        cuts.append((b, e))
    torch.cuda.synchronize()
    ptrs = [o.state_buffer()[0] for o in ops]
    y2 = torch.empty_like(q)
    for o, (b, e) in zip(ops, cuts):
        y2[:, :, b:e] = o.apply_peers(q[:, :, b:e].contiguous(), ptrs)
    torch.cuda.synchronize()
    assert_parity(y2, ref, "fp16 apply_peers")
    for o in ops:
        o.close()
