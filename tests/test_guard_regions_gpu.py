"""Out-of-bounds writes, looked for from the host: Q, K, V, Y and a lent workspace sit inside larger
buffers with guard bands of a fixed byte pattern on both sides; after every variant, layout and
storage type has run on ragged shapes, every guard byte must still hold the pattern, the inputs must
be unchanged, and Y must have been written in full.  (The stand-in for a memory checker: TMA
stores clipped at N, streaming stores of ragged tails and the partial-state writes are what could
stray.)"""
import pytest
import torch

from paper_2409_02097_b200 import attn, workloads as wl

from _util import EPS, assert_parity, oracle_y

pytestmark = pytest.mark.gpu

GUARD = 64 * 1024
PATTERN = 0xA5

RAGGED = [(1, 1, 1, 64), (2, 1, 63, 64), (1, 2, 65, 64), (1, 1, 127, 64), (1, 3, 129, 64),
          (1, 2, 4097, 64), (1, 2, 12289, 64), (1, 3, 1, 40), (2, 2, 65, 40), (1, 2, 4097, 40),
          (1, 1, 63, 160), (1, 3, 129, 160), (1, 2, 4097, 160), (1, 2, 127, 80), (1, 1, 129, 128)]


class Guarded:
    """`count` regions of `nbytes` each inside one allocation, separated and surrounded by guards."""

    def __init__(self, nbytes, count):
        self.nbytes = (nbytes + 255) // 256 * 256
        self.count = count
        self.buf = torch.full((GUARD + count * (self.nbytes + GUARD),), PATTERN, dtype=torch.uint8, device="cuda")
        self.real = nbytes

    def region(self, i):
        start = GUARD + i * (self.nbytes + GUARD)
        return self.buf[start:start + self.real]

    def guards_intact(self):
        ok = True
        for i in range(self.count + 1):
            start = i * (self.nbytes + GUARD)
            lo = start - (self.nbytes - self.real) if i > 0 else start     # the round-up slack counts as guard
            ok = ok and bool((self.buf[lo:start + GUARD] == PATTERN).all().item())
        return ok


def _variants(N, d):
    out = ["split", "cluster"]
    if d == 64:
        out += ["stream"]
    if d in (40, 64, 80, 160):
        out += ["fused"]
    return out


@pytest.mark.parametrize("dims", RAGGED, ids=lambda d: "x".join(map(str, d)))
def test_no_write_lands_outside_y_or_the_workspace(dims):
    B, H, N, d = dims
    q0, k0, v0 = wl.make_small(B, H, N, d, seed=51, device="cuda")
    ref = oracle_y(q0, k0, v0)
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    for dtype in ("bf16", "fp16"):
        tdt = torch.bfloat16 if dtype == "bf16" else torch.float16
        ref_d = ref if dtype == "bf16" else oracle_y(q0.half(), k0.half(), v0.half())
        for layout in ("head_major", "token_major"):
            shape = (B, H, N, d) if layout == "head_major" else (B, N, H, d)
            g = Guarded(B * H * N * d * 2, 4)
            views = [g.region(i).view(tdt).view(shape) for i in range(4)]
            for t, src in zip(views[:3], (q0, k0, v0)):
                t.copy_((src if layout == "head_major" else src.permute(0, 2, 1, 3)).to(tdt))
            q, k, v, y = views
            originals = [t.clone() for t in (q, k, v)]
            for variant in _variants(N, d):
                op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant=variant, layout=layout, dtype=dtype)
                nbytes = attn.linfusion_attn_workspace_bytes(op.desc, sm)
                ws = Guarded(nbytes, 1)
                op.set_workspace(ws.region(0))
                y.fill_(float("nan"))
                op.forward(q, k, v, y)
                torch.cuda.synchronize()
                what = f"{dims} {dtype} {layout} {variant}"
                assert op.status() == attn.OK, what
                assert g.guards_intact(), f"{what}: a guard band around Q/K/V/Y was written"
                assert ws.guards_intact(), f"{what}: a guard band around the workspace was written"
                for t, o in zip((q, k, v), originals):
                    assert torch.equal(t.view(torch.int16), o.view(torch.int16)), f"{what}: an input changed"
                yy = y if layout == "head_major" else y.permute(0, 2, 1, 3)
                assert_parity(yy, ref_d, what)                      # finite everywhere: Y was written in full
                op.close()
            # the allocation-free entry point (its scratch is the library's own array)
            if 2 * B * H * d * (d + 1) * 4 + 512 <= 16 << 20:
                y.fill_(float("nan"))
                desc = attn.make_desc(B, H, N, d, eps=EPS, layout=layout, dtype=dtype)
                attn.linfusion_attn_forward_noalloc(desc, q.data_ptr(), k.data_ptr(), v.data_ptr(), y.data_ptr(),
                                                    torch.cuda.current_stream().cuda_stream)
                torch.cuda.synchronize()
                assert g.guards_intact(), f"{dims} {dtype} {layout} noalloc: a guard band was written"
                yy = y if layout == "head_major" else y.permute(0, 2, 1, 3)
                assert_parity(yy, ref_d, f"{dims} {dtype} {layout} noalloc")


def test_a_handle_created_while_the_default_stream_is_busy_serves_a_side_stream_at_once():
    """create() clears part of the workspace; a forward enqueued right afterwards on a non-blocking
    side stream must neither see stale contents nor be overtaken by the clear."""
    shape = wl.find_shape("sdxl_2048_L2")
    q, k, v = wl.make_qkv(shape, seed=71, device="cuda")
    ref_op = attn.LinFusionAttention(shape.B, shape.H, shape.N, shape.d, variant="stream")
    want = ref_op.forward(q, k, v).clone()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    junk = torch.empty(1 << 28, dtype=torch.uint8, device="cuda")
    for variant in ("stream", "split"):
        for _ in range(8):                       # keep the legacy default stream busy
            junk.fill_(1)
        op = attn.LinFusionAttention(shape.B, shape.H, shape.N, shape.d, variant=variant)
        y = torch.empty_like(q)
        op.forward(q, k, v, y, stream=side.cuda_stream)
        side.synchronize()
        torch.cuda.synchronize()
        assert op.status() == attn.OK
        if variant == "stream":
            assert torch.equal(y.view(torch.int16), want.view(torch.int16))
        else:
            assert_parity(y, oracle_y(q, k, v), "side stream, split")
        # the same after lending a workspace
        nbytes = attn.linfusion_attn_workspace_bytes(op.desc, torch.cuda.get_device_properties(0).multi_processor_count)
        ws = torch.full((nbytes + 256,), 0xFF, dtype=torch.uint8, device="cuda")
        off = (-ws.data_ptr()) % 256
        for _ in range(8):
            junk.fill_(2)
        op.set_workspace(ws[off:off + nbytes])
        y2 = torch.empty_like(q)
        op.forward(q, k, v, y2, stream=side.cuda_stream)
        side.synchronize()
        torch.cuda.synchronize()
        assert op.status() == attn.OK
        assert torch.equal(y2.view(torch.int16), y.view(torch.int16))
        op.close()
    ref_op.close()
