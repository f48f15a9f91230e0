"""The single-launch TMA + tcgen05 kernel for head widths 40, 80 and 160 (variant "fused" at those
widths; Prop. 2, Eq. 5) against the fp64 oracle on the same seeded inputs: ragged tails, one to many
CTAs per slab, both layouts, both storage types, the operator without its normalizer."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_02097_b200 import attn, workloads as wl

from _util import EPS, assert_parity, to_f64

pytestmark = pytest.mark.gpu

WIDTHS = [40, 80, 160]
# (B, H, N): one CTA per slab with a ragged tile; one tile each for many CTAs; several tiles per CTA;
# more CTAs per slab than the reduction's batch of four; a single slab cut into many runs; as many
# slabs as a B200 has SMs (one CTA per slab, several tiles each)
SIZES = [(1, 2, 1), (1, 3, 63), (2, 2, 129), (2, 8, 256), (2, 8, 1000), (1, 12, 1500), (1, 1, 5000), (4, 37, 300),
         (4, 50, 300), (1, 149, 129), (3, 111, 64),   # more slabs than SMs: a CTA takes two or three whole slabs in turn
         (1, 150, 8200),                              # ... of 65 tiles each: one long accumulation chain per slab
         (2, 8, 1500), (1, 1, 30000)]                 # long runs on few slabs: the CTAs of a slab share the summing (two rounds)


@pytest.mark.parametrize("d", WIDTHS)
@pytest.mark.parametrize("size", SIZES, ids=lambda s: "x".join(map(str, s)))
def test_fused_at_padded_widths_matches_the_oracle(d, size):
    B, H, N = size
    for v_mean in (0.0, 1.0):
        q, k, v = wl.make_small(B, H, N, d, seed=61, device="cuda", v_mean=v_mean)
        ref = oracle.linear(to_f64(q), to_f64(k), to_f64(v), EPS)
        S_ref, z_ref = oracle.state(to_f64(k), to_f64(v))
        op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant="fused")
        assert op.variant == "fused" and op.launches_per_forward == 1
        y = op.forward(q, k, v)
        torch.cuda.synchronize()
        assert op.status() == attn.OK
        assert_parity(y, ref, f"d={d} {size} v_mean={v_mean}")
        S, z = op.read_state()
        # 16-bit operands phi(K), V (unit roundoff 2^-8 each) bound the error for any N; the tight
        # gates hold once many tokens average the roundings out
        z_tol, s_tol = (2e-3, 5e-3) if N >= 256 else (2.0 ** -8, 2.0 ** -7)
        assert np.abs(z - z_ref).max() <= z_tol * np.abs(z_ref).max()
        assert np.linalg.norm(S - S_ref) <= s_tol * np.linalg.norm(S_ref) + 1e-6
        y2 = op.forward(q, k, v)
        torch.cuda.synchronize()
        assert torch.equal(y, y2), "not bit-reproducible"
        op.close()


@pytest.mark.parametrize("d", WIDTHS)
def test_fused_at_padded_widths_layouts_types_and_normalizer(d):
    B, H, N = 2, 3, 777
    q, k, v = wl.make_small(B, H, N, d, seed=63, device="cuda", v_mean=1.0)
    ref = oracle.linear(to_f64(q), to_f64(k), to_f64(v), EPS)
    base = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant="fused")
    y_hm = base.forward(q, k, v)
    torch.cuda.synchronize()
    assert_parity(y_hm, ref, f"d={d} head-major")
    # token-major [B, N, H, d]: same arithmetic in the same order, so the same bits
    tm = lambda t: t.permute(0, 2, 1, 3).contiguous()
    op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant="fused", layout="token_major")
    y_tm = op.forward(tm(q), tm(k), tm(v))
    torch.cuda.synchronize()
    assert op.status() == attn.OK
    assert torch.equal(y_tm.permute(0, 2, 1, 3), y_hm)
    op.close()
    # the split path computes the same operator: results agree to output rounding
    op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant="split")
    y_split = op.forward(q, k, v)
    torch.cuda.synchronize()
    assert_parity(y_split, ref, f"d={d} split")
    op.close()
    # fp16 storage
    qh, kh, vh = q.half(), k.half(), v.half()
    ref_h = oracle.linear(to_f64(qh), to_f64(kh), to_f64(vh), EPS)
    op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant="fused", dtype="fp16")
    y = op.forward(qh, kh, vh)
    torch.cuda.synchronize()
    assert op.status() == attn.OK
    assert_parity(y, ref_h, f"d={d} fp16", rel_fro_tol=1e-3)
    op.close()
    # without the normalizer: Y_i = phi(Q_i) S (|Y| grows with N: gates scale with max|Y|)
    S_ref, _ = oracle.state(to_f64(k), to_f64(v))
    ref_un = oracle.apply_unnormalized(to_f64(q), S_ref)
    op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant="fused", normalize=False)
    y = op.forward(q, k, v)
    torch.cuda.synchronize()
    diff = np.abs(to_f64(y) - ref_un)
    assert diff.max() <= 2e-2 * np.abs(ref_un).max()
    assert np.linalg.norm(diff) <= 1e-2 * np.linalg.norm(ref_un)
    op.close()
    # identity feature map
    qp, kp = q.abs() + 0.5, k.abs() + 0.5
    ref_id = oracle.linear(to_f64(qp), to_f64(kp), to_f64(v), EPS, oracle.PHI_IDENTITY)
    op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant="fused", phi=attn.PHI_IDENTITY)
    y = op.forward(qp, kp, v)
    torch.cuda.synchronize()
    assert_parity(y, ref_id, f"d={d} identity phi")
    op.close()
    base.close()


def test_fused_at_padded_widths_limits():
    """More than 512 tiles per CTA are refused when asked for by name and fall to another variant
    under AUTO; d' != d has no such kernel."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    with pytest.raises(attn.LinFusionError) as e:
        attn.LinFusionAttention(1, sms + 1, 128 * 513, 40, variant="fused")
    assert e.value.code == attn.ERR_UNSUPPORTED
    with pytest.raises(attn.LinFusionError) as e:
        attn.LinFusionAttention(1, sms, 128 * 513, 80, variant="fused")
    assert e.value.code == attn.ERR_UNSUPPORTED
    with pytest.raises(attn.LinFusionError) as e:
        attn.LinFusionAttention(1, 2, 256, 40, variant="fused", d_qk=80)
    assert e.value.code == attn.ERR_UNSUPPORTED
    op = attn.LinFusionAttention(1, sms + 1, 128 * 513, 40)
    assert op.variant != "fused"
    op.close()
    op = attn.LinFusionAttention(1, sms + 1, 256, 40)     # whole slabs, several per CTA
    assert op.variant == "fused"
    op.close()


def test_fused_at_padded_widths_back_to_back_and_graph():
    """Forwards chained on one stream (each starts while the one before drains; the per-slab counters
    are put back to zero by the last CTA) and replayed from a CUDA graph give the same bits."""
    B, H, N, d = 2, 8, 1024, 80
    q, k, v = wl.make_small(B, H, N, d, seed=65, device="cuda", v_mean=1.0)
    op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant="fused")
    y0 = op.forward(q, k, v).clone()
    ys = [torch.empty_like(y0) for _ in range(6)]
    for y in ys:
        op.forward(q, k, v, y=y)
    torch.cuda.synchronize()
    assert op.status() == attn.OK
    for y in ys:
        assert torch.equal(y, y0)
    g = torch.cuda.CUDAGraph()
    yg = torch.empty_like(y0)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        op.forward(q, k, v, y=yg)
        with torch.cuda.graph(g, stream=s):
            op.forward(q, k, v, y=yg)
            op.forward(q, k, v, y=yg)
    torch.cuda.current_stream().wait_stream(s)
    yg.zero_()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    assert op.status() == attn.OK
    assert torch.equal(yg, y0)
    op.close()
