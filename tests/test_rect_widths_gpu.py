"""Two widths (Prop. 3): Q and K carry d' features, V and Y carry d channels, the state is d' x d.
The CUDA library (split path, cluster kernel, allocation-free entry point, token-sharded halves)
against the fp64 oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_02097_b200 import attn, workloads as wl

from _util import EPS, assert_parity, to_f64

pytestmark = pytest.mark.gpu

PAIRS = [(128, 64), (80, 40), (32, 64)]          # (d', d)
# (B, H, N): several K/V tiles and Q tiles with ragged tails, one tiny, one mid-size
SIZES = [(2, 3, 1000), (1, 2, 1), (1, 1, 65), (2, 8, 4096)]


def _inputs(B, H, N, dk, dv, seed, v_mean=0.0, device="cuda"):
    """Q, K ~ N(0,1) with dk channels, V ~ N(v_mean,1) with dv channels, from the workload generator."""
    q, k, _ = wl.make_small(B, H, N, dk, seed=seed, device=device)
    _, _, v = wl.make_small(B, H, N, dv, seed=seed + 1, device=device, v_mean=v_mean)
    return q, k, v


@pytest.mark.parametrize("pair", PAIRS, ids=lambda p: f"dk{p[0]}_dv{p[1]}")
@pytest.mark.parametrize("size", SIZES, ids=lambda s: "x".join(map(str, s)))
def test_rectangular_state_split_and_cluster_match_the_oracle(pair, size):
    dk, dv = pair
    B, H, N = size
    for v_mean in (0.0, 1.0):
        q, k, v = _inputs(B, H, N, dk, dv, seed=71, v_mean=v_mean)
        ref = oracle.linear(to_f64(q), to_f64(k), to_f64(v), EPS)
        assert ref.shape == (B, H, N, dv)
        S_ref, z_ref = oracle.state(to_f64(k), to_f64(v))
        for variant in ("auto", "split", "cluster"):
            op = attn.LinFusionAttention(B, H, N, dv, eps=EPS, variant=variant, d_qk=dk)
            assert op.variant in ("split", "cluster")
            y = op.forward(q, k, v)
            torch.cuda.synchronize()
            assert op.status() == attn.OK
            assert tuple(y.shape) == (B, H, N, dv)
            assert_parity(y, ref, f"dk={dk} dv={dv} {size} {variant} v_mean={v_mean}")
            S, z = op.read_state()
            assert S.shape == (B, H, dk, dv) and z.shape == (B, H, dk)
            # every phi(K_jc) is a 16-bit operand (unit roundoff 2^-8): that bounds the error of their
            # sum z for any N; over many tokens the roundings average out and the tighter gate holds
            z_tol = 2e-3 if N >= 256 else 2.0 ** -8
            assert np.abs(z - z_ref).max() <= z_tol * np.abs(z_ref).max()
            assert np.linalg.norm(S - S_ref) <= 5e-3 * np.linalg.norm(S_ref) + 1e-6
            y2 = op.forward(q, k, v)
            torch.cuda.synchronize()
            assert torch.equal(y, y2), "not bit-reproducible"
            op.close()


@pytest.mark.parametrize("pair", PAIRS, ids=lambda p: f"dk{p[0]}_dv{p[1]}")
def test_rectangular_token_major_fp16_unnormalized_and_noalloc(pair):
    dk, dv = pair
    B, H, N = 2, 3, 777
    q, k, v = _inputs(B, H, N, dk, dv, seed=73, v_mean=1.0)
    ref = oracle.linear(to_f64(q), to_f64(k), to_f64(v), EPS)
    base = attn.LinFusionAttention(B, H, N, dv, eps=EPS, variant="split", d_qk=dk)
    y_hm = base.forward(q, k, v)
    # token-major [B, N, H, .]: same arithmetic in the same order, so the same bits
    tm = lambda t: t.permute(0, 2, 1, 3).contiguous()
    op = attn.LinFusionAttention(B, H, N, dv, eps=EPS, variant="split", layout="token_major", d_qk=dk)
    y_tm = op.forward(tm(q), tm(k), tm(v))
    torch.cuda.synchronize()
    assert torch.equal(y_tm.permute(0, 2, 1, 3), y_hm)
    op.close()
    # fp16 storage
    qh, kh, vh = q.half(), k.half(), v.half()
    ref_h = oracle.linear(to_f64(qh), to_f64(kh), to_f64(vh), EPS)
    op = attn.LinFusionAttention(B, H, N, dv, eps=EPS, variant="split", dtype="fp16", d_qk=dk)
    y = op.forward(qh, kh, vh)
    torch.cuda.synchronize()
    assert_parity(y, ref_h, f"fp16 dk={dk} dv={dv}", rel_fro_tol=1e-3)
    op.close()
    # without the normalizer: Y_i = phi(Q_i) S (|Y| grows with N: gates scale with max|Y|)
    S_ref, _ = oracle.state(to_f64(k), to_f64(v))
    ref_un = oracle.apply_unnormalized(to_f64(q), S_ref)
    op = attn.LinFusionAttention(B, H, N, dv, eps=EPS, variant="split", normalize=False, d_qk=dk)
    y = op.forward(q, k, v)
    torch.cuda.synchronize()
    diff = np.abs(to_f64(y) - ref_un)
    assert diff.max() <= 2e-2 * np.abs(ref_un).max()
    assert np.linalg.norm(diff) <= 1e-2 * np.linalg.norm(ref_un)
    op.close()
    # the allocation-free entry point runs the same split path
    y_na = torch.empty_like(y_hm)
    desc = attn.make_desc(B, H, N, dv, eps=EPS, variant="split", d_qk=dk)
    for _ in range(2):
        y_na.fill_(float("nan"))
        attn.linfusion_attn_forward_noalloc(desc, q.data_ptr(), k.data_ptr(), v.data_ptr(), y_na.data_ptr(),
                                            torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert_parity(y_na, ref, f"noalloc dk={dk} dv={dv}")
    # host buffers
    qc, kc, vc = (t.cpu().pin_memory() for t in (q, k, v))
    yc = torch.empty(B, H, N, dv, dtype=torch.bfloat16).pin_memory()
    base.forward_host(qc, kc, vc, yc)
    torch.cuda.synchronize()
    assert torch.equal(yc, y_hm.cpu())
    base.close()


def test_rectangular_token_sharded_halves_add_up():
    """Sec. 4.3 with Prop. 3's widths: the d' x d states of two token shards, summed, applied to each
    shard's Q, give the unsharded result."""
    dk, dv, B, H, N = 128, 64, 1, 2, 1500
    q, k, v = _inputs(B, H, N, dk, dv, seed=79, v_mean=1.0)
    ref = oracle.linear(to_f64(q), to_f64(k), to_f64(v), EPS)
    cut = 700
    ops, bufs = [], []
    for lo, hi in ((0, cut), (cut, N)):
        op = attn.LinFusionAttention(B, H, hi - lo, dv, eps=EPS, variant="split", d_qk=dk)
        op.state(k[:, :, lo:hi].contiguous(), v[:, :, lo:hi].contiguous())
        ops.append(op)
        bufs.append(op.state_buffer())
    torch.cuda.synchronize()
    assert bufs[0][1] == B * H * dk * (dv + 1)
    ptrs = [b[0] for b in bufs]
    outs = []
    for op, (lo, hi) in zip(ops, ((0, cut), (cut, N))):
        outs.append(op.apply_peers(q[:, :, lo:hi].contiguous(), ptrs))
    torch.cuda.synchronize()
    y = torch.cat(outs, dim=2)
    assert_parity(y, ref, "two shards, d'=128 d=64")
    for op in ops:
        op.close()


def test_unsupported_width_requests_are_refused():
    for kw in (dict(d=64, d_qk=48), dict(d=40, d_qk=128), dict(d=64, d_qk=128, variant="stream"),
               dict(d=64, d_qk=128, variant="fused")):
        with pytest.raises(attn.LinFusionError) as e:
            attn.LinFusionAttention(1, 1, 256, kw["d"], d_qk=kw["d_qk"], variant=kw.get("variant", "auto"))
        assert e.value.code == attn.ERR_UNSUPPORTED
