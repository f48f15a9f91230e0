"""The allocation-free entry point against the handle-based one.

``linfusion_attn_forward_noalloc`` serves hosts that cannot let a library allocate device memory
(a server that gave all of it to its own arena at start-up; a pipeline that cannot take the
device-wide synchronization of cudaMalloc).  Its scratch is a fixed array inside the library, which
every call shares and which keeps the previous call's contents, so the check is done on two calls
in a row, with different inputs, through the C ABI.  This file is named to be collected last.
"""
import numpy as np
import pytest
import torch

from paper_2409_02097_b200 import attn, workloads as wl

import oracle

from _util import EPS, MAX_ABS_TOL, MEAN_ABS_TOL, REL_FRO_TOL, assert_parity, oracle_y, to_f64

pytestmark = pytest.mark.gpu


def _compare(y_new, y_old, what):
    a, b = y_new.double(), y_old.double()
    diff = (a - b).abs()
    rel = (a - b).norm() / b.norm()
    assert torch.isfinite(a).all(), what
    assert diff.max().item() <= MAX_ABS_TOL and diff.mean().item() <= MEAN_ABS_TOL, what
    assert rel.item() <= REL_FRO_TOL, f"{what}: rel_fro={rel.item():.3e}"


@pytest.mark.parametrize("dims", [(2, 8, 4096, 40), (2, 10, 2304, 64), (2, 8, 257, 160)],
                         ids=lambda d: "x".join(map(str, d)))
def test_noalloc_matches_handle_forward_twice_in_a_row(dims):
    B, H, N, d = dims
    op = attn.LinFusionAttention(B, H, N, d, variant="split")
    desc = attn.make_desc(B, H, N, d)
    stream = torch.cuda.current_stream().cuda_stream
    outputs = []
    for call, seed in enumerate((41, 42)):
        q, k, v = wl.make_small(B, H, N, d, seed=seed, device="cuda")
        y_old = op.forward(q, k, v)
        y_new = torch.full_like(q, float("nan"))
        attn.linfusion_attn_forward_noalloc(desc, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                            y_new.data_ptr(), stream)
        torch.cuda.synchronize()
        _compare(y_new, y_old, f"{dims} call {call}")
        assert_parity(y_new, oracle_y(q, k, v), f"noalloc vs oracle {dims} call {call}")
        outputs.append((q, k, v, y_new))
    # the same inputs again give the same bits, whatever an earlier call left in the array
    q, k, v, y_first = outputs[0]
    y_again = torch.empty_like(q)
    attn.linfusion_attn_forward_noalloc(desc, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                        y_again.data_ptr(), stream)
    torch.cuda.synchronize()
    assert torch.equal(y_again.view(torch.int16), y_first.view(torch.int16))
    op.close()


def test_noalloc_rejects_what_does_not_fit_and_bad_arguments():
    q, k, v = wl.make_small(1, 1, 64, 160, seed=1, device="cuda")
    y = torch.empty_like(q)
    ptrs = (q.data_ptr(), k.data_ptr(), v.data_ptr(), y.data_ptr())
    # d = 160 with 100 slabs: the state alone needs 2 * 100 * 160 * 161 * 4 bytes > 16 MiB.
    # Rejected from the descriptor, before any pointer is used.
    with pytest.raises(attn.LinFusionError) as e:
        attn.linfusion_attn_forward_noalloc(attn.make_desc(1, 100, 64, 160), *ptrs)
    assert e.value.code == attn.ERR_ALLOC
    with pytest.raises(attn.LinFusionError) as e:
        attn.linfusion_attn_forward_noalloc(attn.make_desc(1, 1, 64, 160, variant="cluster"), *ptrs)
    assert e.value.code == attn.ERR_UNSUPPORTED
    with pytest.raises(attn.LinFusionError) as e:
        attn.linfusion_attn_forward_noalloc(attn.make_desc(1, 1, 64, 160), ptrs[0], ptrs[1], ptrs[2], 0)
    assert e.value.code == attn.ERR_INVALID_ARG
    with pytest.raises(attn.LinFusionError) as e:
        attn.linfusion_attn_forward_noalloc(attn.make_desc(1, 1, 64, 160), ptrs[0], ptrs[1], ptrs[2], ptrs[0])
    assert e.value.code == attn.ERR_INVALID_ARG


@pytest.mark.parametrize("dims", [(2, 32, 4096, 160), (1, 32, 2000, 160), (2, 40, 1500, 128)],
                         ids=lambda d: "x".join(map(str, d)))
def test_noalloc_when_the_array_limits_the_split_of_n(dims):
    """Shapes whose planned split of N does not fit the 16 MiB array: the entry point uses fewer
    chunks, which moves the state's offset.  Checked against the oracle, against the layout the
    library reports, and for the same bits on a second call."""
    B, H, N, d = dims
    desc = attn.make_desc(B, H, N, d)
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    chunks, off, used, cap = attn.linfusion_attn_noalloc_layout(desc, sm)
    planned = min(-(-2 * sm // (B * H)), -(-N // 64))
    assert 1 <= chunks < planned, (chunks, planned)          # the array, not the plan, set the count
    assert used <= cap and off % 256 == 0
    q, k, v = wl.make_small(B, H, N, d, seed=43, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    ys = []
    for _ in range(2):
        y = torch.full_like(q, float("nan"))
        attn.linfusion_attn_forward_noalloc(desc, q.data_ptr(), k.data_ptr(), v.data_ptr(), y.data_ptr(), stream)
        torch.cuda.synchronize()
        ys.append(y)
    assert torch.equal(ys[0].view(torch.int16), ys[1].view(torch.int16))
    assert_parity(ys[0], oracle_y(q, k, v), f"noalloc clamped {dims}")


def test_noalloc_follows_the_layout_and_normalizer_flags():
    B, H, N, d = 2, 4, 1111, 80
    q, k, v = wl.make_small(B, H, N, d, seed=44, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    # token-major [B, N, H, d]
    qt, kt, vt = (t.permute(0, 2, 1, 3).contiguous() for t in (q, k, v))
    yt = torch.full_like(qt, float("nan"))
    attn.linfusion_attn_forward_noalloc(attn.make_desc(B, H, N, d, layout="token_major"), qt.data_ptr(),
                                        kt.data_ptr(), vt.data_ptr(), yt.data_ptr(), stream)
    torch.cuda.synchronize()
    assert_parity(yt.permute(0, 2, 1, 3), oracle_y(q, k, v), "noalloc token-major")
    # the operator without its normalizer: |Y| grows with N, gates relative to max|Y|
    yu = torch.full_like(q, float("nan"))
    attn.linfusion_attn_forward_noalloc(attn.make_desc(B, H, N, d, normalize=False), q.data_ptr(),
                                        k.data_ptr(), v.data_ptr(), yu.data_ptr(), stream)
    torch.cuda.synchronize()
    ref = oracle.linear_unnormalized(to_f64(q), to_f64(k), to_f64(v))
    scale = np.abs(ref).max()
    diff = np.abs(to_f64(yu) - ref)
    assert diff.max() <= MAX_ABS_TOL * scale and diff.mean() <= MEAN_ABS_TOL * scale
    assert np.linalg.norm(diff) <= REL_FRO_TOL * np.linalg.norm(ref)
