"""GPU parity: the CUDA library (through its C ABI) against the fp64 CPU oracle on the same
seeded inputs, element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_02097_b200 import attn, workloads as wl

from _util import EPS, assert_parity, error_metrics, oracle_y, scaled_max_units, to_f64

pytestmark = pytest.mark.gpu

SMALL_SHAPES = [s for cfg in wl.CONFIGS[:4] for s in cfg]
SMALL_SHAPES = list({s.name: s for s in SMALL_SHAPES}.values())
BIG_SHAPES = wl.CONFIGS[4]


def run_gpu(q, k, v, variant="auto", eps=EPS, phi=attn.PHI_ELU_PLUS_ONE):
    B, H, N, d = q.shape
    op = attn.LinFusionAttention(B, H, N, d, phi=phi, eps=eps, device=q.device.index or 0,
                                 variant=variant)
    y = op.forward(q, k, v)
    torch.cuda.synchronize()
    assert op.status() == attn.OK
    return y, op


def variants_for(shape):
    out = ["auto", "split"]
    if shape.d == 64:
        out.append("stream")
    if shape.d in (40, 64, 80, 160):
        out.append("fused")
    if shape.N <= 16384:
        out.append("cluster")
    return out


@pytest.mark.parametrize("shape", SMALL_SHAPES, ids=lambda s: s.name)
def test_workload_shapes_all_variants(shape):
    q, k, v = wl.make_qkv(shape, seed=wl.BASE_SEED, device="cuda")
    ref = oracle_y(q, k, v)
    for variant in variants_for(shape):
        y, op = run_gpu(q, k, v, variant)
        assert_parity(y, ref, f"{shape.name}/{variant}->{op.variant}")
        op.close()


@pytest.mark.parametrize("shape", SMALL_SHAPES, ids=lambda s: s.name)
def test_workload_shapes_shifted_v(shape):
    """V ~ N(1, 1): |Y| ~ 1, where the absolute gate bites (at |Y| in [1, 2) bf16 output rounding
    alone has a mean error of about 1.95e-3, in [0.5, 1) half of that)."""
    q, k, v = wl.make_qkv(shape, seed=wl.BASE_SEED + 1, device="cuda", v_mean=1.0)
    ref = oracle_y(q, k, v)
    y, op = run_gpu(q, k, v)
    assert_parity(y, ref, f"{shape.name}/v_mean=1")
    op.close()


SAMPLED_ROWS = 4096


def _sampled_rows(N, tile, rng):
    """Rows of a slab that the oracle computes one by one: a seeded random set plus the places
    where an indexing mistake would show first (both ends of the slab, the rows on either side of
    the first tile boundaries and of the last one, the ragged tail)."""
    fixed = [0, 1, tile - 1, tile, tile + 1, 2 * tile - 1, 2 * tile, N // 2, N - 1, N - 2,
             (N - 1) // tile * tile - 1, (N - 1) // tile * tile]
    fixed = [r for r in fixed if 0 <= r < N]
    rows = np.unique(np.concatenate([np.asarray(fixed, dtype=np.int64),
                                     rng.integers(0, N, size=SAMPLED_ROWS, dtype=np.int64)]))
    return rows


@pytest.mark.parametrize("v_mean", [0.0, 1.0], ids=["v_zero_mean", "v_mean_1"])
@pytest.mark.parametrize("shape", BIG_SHAPES, ids=lambda s: s.name)
def test_full_size_16k_shapes_every_slab(shape, v_mean):
    """Full size, in the configuration the benchmark times.  Every (batch, head) slab: its reduced
    state S | z against the oracle's, and its Y against the oracle's — whole slabs for the first, a
    middle and the last one, 4096 seeded rows plus the tile-boundary rows for every other slab.
    With V ~ N(1, 1) |Y| is about 1 (Eq. 5's row sums of one pass V's mean through), so the
    absolute gates bite; with V ~ N(0, 1) |Y| ~ 1/sqrt(N) and the scale-aware gates carry the check."""
    q, k, v = wl.make_qkv(shape, seed=wl.BASE_SEED + (1 if v_mean else 0), device="cuda", v_mean=v_mean)
    y, op = run_gpu(q, k, v)
    assert op.variant == "stream"
    assert torch.isfinite(y.view(-1)[:: 4097].float()).all()
    S_gpu, z_gpu = op.read_state()
    rng = np.random.default_rng(20240902)
    whole = {(0, 0), (1, shape.H // 2), (shape.B - 1, shape.H - 1)}
    worst = 0.0
    for b in range(shape.B):
        for h in range(shape.H):
            S, z = oracle.state(to_f64(k[b, h]), to_f64(v[b, h]))
            # state: relative to its own scale (entries are sums of N terms)
            assert np.abs(z_gpu[b, h] - z).max() <= 2e-3 * np.abs(z).max(), (b, h)
            assert np.linalg.norm(S_gpu[b, h] - S) <= 5e-3 * np.linalg.norm(S), (b, h)
            if (b, h) in whole:
                ref = oracle.apply(to_f64(q[b, h]), S, z, EPS)
                assert_parity(y[b, h], ref, f"{shape.name}[{b},{h}] whole slab")
                worst = max(worst, scaled_max_units(y[b, h], ref))
            else:
                rows = torch.from_numpy(_sampled_rows(shape.N, 128, rng)).to(q.device)
                ref = oracle.apply(to_f64(q[b, h][rows]), S, z, EPS)
                got = y[b, h][rows]
                # (the sample's own max|Y| is a little below the slab's: that only tightens the gate)
                assert_parity(got, ref, f"{shape.name}[{b},{h}] sampled rows")
                worst = max(worst, scaled_max_units(got, ref))
    print(f"{shape.name} v_mean={v_mean}: worst scaled max error {worst:.2f} units")
    op.close()


EDGE_CASES = [
    # (B, H, N, d): ragged tails, tiny N, N around tile sizes, odd slab counts
    (1, 1, 1, 64), (1, 1, 1, 40), (1, 3, 7, 160), (2, 1, 63, 64), (1, 2, 65, 64),
    (1, 1, 127, 64), (1, 1, 129, 64), (1, 5, 191, 64), (1, 1, 193, 64), (3, 1, 1000, 80),
    (1, 7, 333, 40), (1, 1, 4097, 128), (2, 3, 257, 32), (1, 2, 12289, 64), (1, 148, 64, 64),
    (8, 25, 300, 64),   # more slabs than SMs
    (3, 100, 100, 64),  # 300 one-tile slabs: the single-launch variant deals whole slabs, two or three per CTA

]


@pytest.mark.parametrize("dims", EDGE_CASES, ids=lambda d: "x".join(map(str, d)))
def test_edge_shapes_all_variants(dims):
    B, H, N, d = dims
    q, k, v = wl.make_small(B, H, N, d, seed=11, device="cuda")
    ref = oracle_y(q, k, v)
    for variant in variants_for(wl.AttnShape("e", B, H, N, d)):
        y, op = run_gpu(q, k, v, variant)
        assert_parity(y, ref, f"{dims}/{variant}->{op.variant}")
        op.close()


def test_stream_variant_tail_and_slab_crossing():
    """Many slabs, ragged N: every CTA's run crosses slab boundaries and tail tiles are masked."""
    # the last case gives every CTA a run of 60 tiles: more than one tensor-memory segment per slab
    # and, for the CTAs at the seams, a change of slab in mid-run
    # (1, 7, 200000): long enough for the apply kernel to hand its tiles out through the per-slab counters
    # (the shorter cases get fixed runs), with CTAs moving on to other slabs at the end
    for (B, H, N) in [(2, 37, 1000), (1, 100, 130), (2, 20, 2500), (1, 3, 378917), (1, 7, 200000)]:
        q, k, v = wl.make_small(B, H, N, 64, seed=5, device="cuda")
        ref = oracle_y(q, k, v)
        for variant in ("stream", "fused"):
            y, op = run_gpu(q, k, v, variant)
            assert op.variant == variant
            assert_parity(y, ref, f"{variant} {(B, H, N)}")
            op.close()


def test_auto_policy_follows_the_measured_crossovers():
    for dims, want in [((2, 10, 16384, 64), "stream"), ((2, 20, 4096, 64), "stream"),
                       ((2, 20, 2304, 64), "stream"), ((2, 10, 9216, 64), "stream"), ((1, 10, 2304, 64), "split"), ((2, 20, 144, 64), "cluster"), ((2, 20, 576, 64), "fused"),
                       ((2, 2, 144, 64), "cluster"), ((2, 8, 4096, 40), "fused"), ((2, 8, 1024, 80), "fused"),
                       ((2, 8, 64, 160), "fused"), ((2, 8, 256, 160), "fused"), ((2, 100, 256, 160), "fused"),
                       ((2, 100, 64, 160), "fused"), ((2, 100, 8192, 160), "fused"), ((2, 100, 131072, 160), "split"),
                       ((2, 8, 1000, 160), "fused"), ((1, 1, 100000, 160), "fused"), ((2, 8, 16384, 160), "fused"), ((2, 8, 4096, 128), "split")]:
        op = attn.LinFusionAttention(*dims)
        assert op.variant == want, (dims, op.variant)
        op.close()


def test_bit_reproducible_run_to_run():
    for shape, variant in [(wl.find_shape("sdxl_2048_L2"), "stream"),
                           (wl.find_shape("sdxl_2048_L2"), "fused"),
                           (wl.find_shape("sd21_768_L4"), "fused"),
                           (wl.find_shape("sd15_512_L1"), "split"),
                           (wl.find_shape("sd15_512_L1"), "fused"),
                           (wl.find_shape("sd15_512_L3"), "fused"),
                           (wl.find_shape("sd15_512_L2"), "cluster")]:
        q, k, v = wl.make_qkv(shape, seed=3, device="cuda")
        y1, op = run_gpu(q, k, v, variant)
        y2 = op.forward(q, k, v)
        torch.cuda.synchronize()
        op.close()
        y3, op3 = run_gpu(q, k, v, variant)
        op3.close()
        assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))
        assert torch.equal(y1.view(torch.int16), y3.view(torch.int16))


def test_state_matches_oracle_state():
    shape = wl.find_shape("sd21_768_L2")
    q, k, v = wl.make_qkv(shape, seed=9, device="cuda")
    S, z = oracle.state(to_f64(k), to_f64(v))
    for variant in ("split", "stream", "cluster", "fused"):
        _, op = run_gpu(q, k, v, variant)
        S_gpu, z_gpu = op.read_state()
        op.close()
        assert np.abs(z_gpu - z).max() <= 2e-3 * np.abs(z).max(), variant
        assert np.linalg.norm(S_gpu - S) <= 5e-3 * np.linalg.norm(S), variant


def test_constant_v_and_zero_qk_properties():
    B, H, N, d = 1, 2, 3000, 64
    q, k, _ = wl.make_small(B, H, N, d, seed=21, device="cuda")
    row = torch.linspace(-2, 2, d, device="cuda").bfloat16()
    v = row.expand(B, H, N, d).contiguous()
    for variant in ("split", "stream", "cluster"):
        y, op = run_gpu(q, k, v, variant)
        op.close()
        # row sums of the attention weights are one: constant V comes back (to bf16 rounding)
        assert (y.float() - row.float()).abs().max().item() <= 2.0 * 2 ** -8
    z = torch.zeros_like(q)
    _, _, v2 = wl.make_small(B, H, N, d, seed=22, device="cuda")
    y, op = run_gpu(z, z, v2, "stream")
    op.close()
    mean = v2.float().mean(dim=2, keepdim=True)
    assert (y.float() - mean).abs().max().item() <= 2e-3


def test_outlier_scale_inputs_and_identity_phi():
    q, k, v = wl.make_small(1, 4, 2048, 64, seed=31, device="cuda", scale=8.0)
    ref = oracle_y(q, k, v)
    for variant in ("split", "stream", "cluster"):
        y, op = run_gpu(q, k, v, variant)
        op.close()
        assert_parity(y, ref, f"x8/{variant}")
    qa, ka = q.abs(), k.abs()
    ref = oracle_y(qa, ka, v, phi_kind=oracle.PHI_IDENTITY)
    for variant in ("split", "stream", "cluster"):
        y, op = run_gpu(qa, ka, v, variant, phi=attn.PHI_IDENTITY)
        op.close()
        assert_parity(y, ref, f"identity/{variant}")


def test_forward_host_matches_device_forward():
    shape = wl.find_shape("sd21_768_L3")
    q, k, v = wl.make_qkv(shape, seed=13, device="cpu")
    qp, kp, vp = (t.pin_memory() for t in (q, k, v))
    yp = torch.empty_like(qp).pin_memory()
    op = attn.LinFusionAttention(shape.B, shape.H, shape.N, shape.d)
    op.forward_host(qp, kp, vp, yp)
    torch.cuda.synchronize()
    y_dev = op.forward(q.cuda(), k.cuda(), v.cuda())
    torch.cuda.synchronize()
    assert torch.equal(yp.view(torch.int16), y_dev.cpu().view(torch.int16))
    assert_parity(yp, oracle_y(q, k, v), "forward_host")
    op.close()


def test_lent_workspace_gives_same_bits():
    shape = wl.find_shape("sdxl_2048_L2")
    q, k, v = wl.make_qkv(shape, seed=17, device="cuda")
    y1, op = run_gpu(q, k, v, "stream")
    nbytes = attn.linfusion_attn_workspace_bytes(op.desc, torch.cuda.get_device_properties(0).multi_processor_count)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    off = (-ws.data_ptr()) % 256
    op.set_workspace(ws[off:off + nbytes])
    y2 = op.forward(q, k, v)
    torch.cuda.synchronize()
    assert op.status() == attn.OK
    assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))
    with pytest.raises(attn.LinFusionError) as e:
        op.set_workspace(ws[off:off + 256])
    assert e.value.code == attn.ERR_ALLOC
    op.close()


def test_forward_argument_errors_touch_no_memory():
    op = attn.LinFusionAttention(1, 1, 256, 64)
    q, k, v = wl.make_small(1, 1, 256, 64, seed=1, device="cuda")
    y = torch.empty_like(q)
    lib = attn.load_library()
    args = [q.data_ptr(), k.data_ptr(), v.data_ptr(), y.data_ptr()]
    for i in range(4):
        bad = list(args)
        bad[i] = 0
        assert lib.linfusion_attn_forward(op._h, *bad, None) == attn.ERR_INVALID_ARG
        bad[i] = args[i] + 2
        assert lib.linfusion_attn_forward(op._h, *bad, None) == attn.ERR_INVALID_ARG
    assert lib.linfusion_attn_forward(op._h, args[0], args[1], args[2], args[0], None) == attn.ERR_INVALID_ARG
    assert lib.linfusion_attn_forward(op._h, args[0], args[1], args[2], args[2] + 64, None) == attn.ERR_INVALID_ARG
    with pytest.raises(attn.LinFusionError) as e:
        attn.LinFusionAttention(1, 1, 256, 64, device=torch.cuda.device_count())
    assert e.value.code == attn.ERR_INVALID_ARG
    op.close()


def test_forward_host_pipelined_groups():
    """Large enough for the grouped copy/compute pipeline of forward_host (5 groups of 4 slabs)."""
    B, H, N, d = 2, 10, 65536, 64
    q, k, v = wl.make_small(B, H, N, d, seed=19, device="cpu")
    qp, kp, vp = (t.pin_memory() for t in (q, k, v))
    yp = torch.full_like(qp, float("nan")).pin_memory()
    op = attn.LinFusionAttention(B, H, N, d)
    op.forward_host(qp, kp, vp, yp)
    torch.cuda.synchronize()
    first = yp.clone()
    op.forward_host(qp, kp, vp, yp)          # second call: same bits, buffers reused
    torch.cuda.synchronize()
    assert op.status() == attn.OK
    assert torch.equal(first.view(torch.int16), yp.view(torch.int16))
    y_dev = op.forward(q.cuda(), k.cuda(), v.cuda())
    torch.cuda.synchronize()
    diff = (yp.float() - y_dev.cpu().float()).abs()
    assert diff.max().item() <= 2e-3                      # same math, different split of N
    for b, h in [(0, 0), (1, 9), (1, 4)]:
        assert_parity(yp[b, h], oracle_y(q[b, h], k[b, h], v[b, h]), f"forward_host[{b},{h}]")
    op.close()


@pytest.mark.parametrize("dims,variant", [((2, 10, 4100, 64), "stream"), ((2, 8, 1000, 40), "split"),
                                          ((1, 4, 130, 160), "cluster"), ((2, 5, 100, 64), "cluster"),
                                          ((1, 3, 2049, 80), "auto")], ids=lambda x: str(x))
def test_token_major_layout_gives_the_same_bits(dims, variant):
    """[B, N, H, d] tensors (a UNet's [B, N, C] with heads split in place).  The split and cluster
    variants do the same arithmetic in the same order as in the head-major layout, so their outputs
    must agree bit for bit; the stream variant deals its CTAs to the slabs differently in this
    layout (another fixed split of N), so there only the last bits may differ."""
    B, H, N, d = dims
    q, k, v = wl.make_small(B, H, N, d, seed=23, device="cuda")
    y_hm, op = run_gpu(q, k, v, variant)
    resolved = op.variant
    op.close()
    tm = lambda t: t.permute(0, 2, 1, 3).contiguous()
    op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant=resolved, layout="token_major")
    qt, kt, vt = tm(q), tm(k), tm(v)
    y_tm = op.forward(qt, kt, vt)
    torch.cuda.synchronize()
    assert op.status() == attn.OK
    assert y_tm.shape == (B, N, H, d)
    y_back = y_tm.permute(0, 2, 1, 3).contiguous()
    if resolved == "stream":
        diff = (y_back.float() - y_hm.float()).abs()
        assert diff.max().item() <= 4e-3 * y_hm.float().abs().max().item()     # bf16 rounding flips only
        y_again = op.forward(qt, kt, vt)                                       # and reproducible
        torch.cuda.synchronize()
        assert torch.equal(y_again.view(torch.int16), y_tm.view(torch.int16))
    else:
        assert torch.equal(y_back.view(torch.int16), y_hm.view(torch.int16))
    assert_parity(y_tm.permute(0, 2, 1, 3), oracle_y(q, k, v), f"token-major {dims} {variant}")
    # the allocation-free entry point follows the layout flag too
    if d != 160 or B * H <= 81:
        y2 = torch.empty_like(y_tm)
        desc = attn.make_desc(B, H, N, d, eps=EPS, layout="token_major")
        attn.linfusion_attn_forward_noalloc(desc, qt.data_ptr(), kt.data_ptr(), vt.data_ptr(),
                                            y2.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert_parity(y2.permute(0, 2, 1, 3), oracle_y(q, k, v), f"token-major noalloc {dims}")
    op.close()


def test_kernel_timing_stride_samples_every_nth_forward():
    shape = wl.find_shape("sdxl_2048_L1")
    q, k, v = wl.make_qkv(shape, seed=3, device="cuda")
    y, op = run_gpu(q, k, v, "stream")
    op.enable_kernel_timing(16)
    op.set_kernel_timing_stride(4)
    outs = [op.forward(q, k, v).clone() for _ in range(10)]
    sums, calls = op.kernel_times()
    assert calls == 3                      # forwards 0, 4 and 8
    assert all(t > 0 for t in sums[:op.launches_per_forward])
    op.enable_kernel_timing(0)
    for o in outs:                         # timed or not, chained or not: the same bits
        assert torch.equal(o.view(torch.int16), y.view(torch.int16))
    with pytest.raises(attn.LinFusionError):
        op.set_kernel_timing_stride(0)
    op.close()


def test_a_wait_that_cannot_complete_gives_up_and_is_reported():
    """Failure reporting without a fault: a bounded wait on a barrier nothing arrives on runs out,
    the kernel returns normally, the status word says so, and the handle keeps working."""
    shape = wl.find_shape("sdxl_2048_L2")
    q, k, v = wl.make_qkv(shape, seed=4, device="cuda")
    y0, op = run_gpu(q, k, v, "stream")
    rc, ms = op.selftest_wait()
    assert rc == attn.ERR_TIMEOUT
    assert 200.0 <= ms <= 2000.0, ms          # the bound is a quarter of a second
    assert op.status() == attn.OK              # cleared again
    y1 = op.forward(q, k, v)
    torch.cuda.synchronize()
    assert op.status() == attn.OK
    assert torch.equal(y0.view(torch.int16), y1.view(torch.int16))
    op.close()


def test_forwards_of_several_handles_replay_from_a_cuda_graph():
    """A UNet level's handles captured once and replayed: forward() only enqueues kernels on the
    given stream (no allocation, no synchronization), chained launches included."""
    shapes = [(wl.find_shape("sdxl_2048_L1"), "auto"), (wl.find_shape("sd15_512_L2"), "auto"),
              (wl.find_shape("sd21_768_L2"), "fused"), (wl.find_shape("sd21_768_L4"), "fused")]
    layers = []
    for i, (s, variant) in enumerate(shapes):
        q, k, v = wl.make_qkv(s, seed=60 + i, device="cuda")
        op = attn.LinFusionAttention(s.B, s.H, s.N, s.d, eps=EPS, variant=variant)
        layers.append((op, q, k, v, op.forward(q, k, v).clone(), torch.empty_like(q)))
    torch.cuda.synchronize()
    st = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        for op, q, k, v, _, y in layers:                       # warm-up on the capture stream
            op.forward(q, k, v, y, stream=st.cuda_stream)
        st.synchronize()
        with torch.cuda.graph(graph, stream=st):
            for op, q, k, v, _, y in layers:
                op.forward(q, k, v, y, stream=st.cuda_stream)
    for *_, y in layers:
        y.zero_()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    for op, q, k, v, ref, y in layers:
        assert torch.equal(y.view(torch.int16), ref.view(torch.int16)), op.variant
        assert op.status() == attn.OK
        op.close()


def test_fused_variant_many_forwards_in_a_row_and_its_bounded_counter_wait():
    """The single-launch variant keeps per-slab arrival counters that are never reset (an epoch
    word says where they stood): many forwards in a row, alternating inputs, must keep giving the
    bits of the first ones; the bounded poll gives up on a counter nothing advances and reports."""
    shape = wl.find_shape("sd21_768_L3")
    qa, ka, va = wl.make_qkv(shape, seed=81, device="cuda")
    qb, kb, vb = wl.make_qkv(shape, seed=82, device="cuda")
    ya, op = run_gpu(qa, ka, va, "fused")
    yb = op.forward(qb, kb, vb).clone()
    assert_parity(ya, oracle_y(qa, ka, va), "fused a")
    assert_parity(yb, oracle_y(qb, kb, vb), "fused b")
    y = torch.empty_like(ya)
    for i in range(300):
        op.forward(*((qa, ka, va) if i % 2 == 0 else (qb, kb, vb)), y)
        if i % 50 in (0, 1):
            torch.cuda.synchronize()
            assert torch.equal(y.view(torch.int16), (ya if i % 2 == 0 else yb).view(torch.int16)), i
    assert op.status() == attn.OK
    S_gpu, z_gpu = op.read_state()
    S, z = oracle.state(to_f64(kb), to_f64(vb))
    assert np.abs(z_gpu - z).max() <= 2e-3 * np.abs(z).max()
    assert np.linalg.norm(S_gpu - S) <= 5e-3 * np.linalg.norm(S)
    rc, ms = op.selftest_counter_wait()
    assert rc == attn.ERR_TIMEOUT
    assert 200.0 <= ms <= 2000.0, ms
    assert op.status() == attn.OK
    y2 = op.forward(qa, ka, va)
    torch.cuda.synchronize()
    assert torch.equal(y2.view(torch.int16), ya.view(torch.int16))
    with pytest.raises(attn.LinFusionError) as e:
        op.state(ka, va)                       # one launch cannot be split in two halves
    assert e.value.code == attn.ERR_UNSUPPORTED
    op.close()


def test_many_back_to_back_forwards_give_the_same_bits():
    """A hundred chained forwards per shape (each starts while the one before drains) into rotating outputs:
    every one must equal the first bit for bit.  Covers the paths with cross-CTA hand-offs: counters and
    operand buffers of the stream kernels, fixed runs, the single launches with their slab counters, a CTA
    taking several slabs in turn."""
    cases = [(2, 8, 4096, 40, "fused"), (2, 8, 1024, 80, "fused"), (3, 111, 64, 160, "fused"), (4, 50, 300, 80, "fused"),
             (2, 20, 4096, 64, "stream"), (2, 5, 9216, 64, "stream"), (8, 25, 300, 64, "stream"),
             (3, 100, 100, 64, "stream"), (1, 7, 200000, 64, "stream"), (2, 20, 576, 64, "fused")]
    for (B, H, N, d, variant) in cases:
        q, k, v = wl.make_small(B, H, N, d, seed=17, device="cuda", v_mean=1.0)
        op = attn.LinFusionAttention(B, H, N, d, variant=variant)
        y0 = op.forward(q, k, v).clone()
        ys = [torch.empty_like(y0) for _ in range(4)]
        reps = 100 if N < 100000 else 24
        for r in range(reps):
            op.forward(q, k, v, y=ys[r % 4])
            if r % 4 == 3:
                torch.cuda.synchronize()
                for t in ys:
                    assert torch.equal(t, y0), (B, H, N, d, variant, r)
        assert op.status() == attn.OK
        op.close()
