"""The bounds-checked debugging build (-DLF_CHECKED) in place of a memory checker: every global-memory
address the split / cluster kernels compute is compared with the buffers of the call; an access
outside them is counted and skipped.  The ragged shapes, both layouts, both storage types, two widths,
the allocation-free entry point and the token-sharded halves must run with a count of zero and still
match the oracle.  The checked library is loaded in a child process (a process holds one build)."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import sys
import numpy as np
import torch
sys.path.insert(0, sys.argv[1]); sys.path.insert(0, sys.argv[1] + "/tests")
import oracle
from paper_2409_02097_b200 import attn, workloads as wl
from _util import EPS, assert_parity, oracle_y, to_f64

assert attn.checked_build(), "not the checked build"
attn.checked_violations(0, reset=True)
RAGGED = [(1, 1, 1, 64), (2, 1, 63, 64), (1, 2, 65, 64), (1, 1, 127, 64), (1, 3, 129, 64), (1, 2, 4097, 64),
          (1, 3, 1, 40), (2, 2, 65, 40), (1, 2, 4097, 40), (1, 1, 63, 160), (1, 3, 129, 160), (1, 2, 4097, 160),
          (1, 2, 127, 80), (1, 1, 129, 128), (2, 8, 64, 160), (2, 20, 144, 64)]
runs = 0
for (B, H, N, d) in RAGGED:
    q, k, v = wl.make_small(B, H, N, d, seed=57, device="cuda")
    ref = oracle_y(q, k, v)
    for layout in ("head_major", "token_major"):
        cv = (lambda t: t) if layout == "head_major" else (lambda t: t.permute(0, 2, 1, 3).contiguous())
        for dtype in ("bf16", "fp16"):
            tdt = torch.bfloat16 if dtype == "bf16" else torch.float16
            qq, kk, vv = (cv(t).to(tdt) for t in (q, k, v))
            r = ref if dtype == "bf16" else oracle_y(q.half(), k.half(), v.half())
            for variant in ("split", "cluster"):
                op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant=variant, layout=layout, dtype=dtype)
                y = op.forward(qq, kk, vv)
                torch.cuda.synchronize()
                assert op.status() == attn.OK
                yy = y if layout == "head_major" else y.permute(0, 2, 1, 3)
                assert_parity(yy, r, f"checked {(B, H, N, d)} {layout} {dtype} {variant}",
                              rel_fro_tol=1e-2 if dtype == "bf16" else 1e-3)
                n = attn.checked_violations(0)
                assert n == 0, f"{n} accesses outside the call's buffers: {(B, H, N, d)} {layout} {dtype} {variant}"
                op.close()
                runs += 1
    # the allocation-free entry point (the fixed array is its workspace)
    y = torch.empty_like(q)
    attn.linfusion_attn_forward_noalloc(attn.make_desc(B, H, N, d, eps=EPS), q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                        y.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert_parity(y, ref, f"checked noalloc {(B, H, N, d)}")
    assert attn.checked_violations(0) == 0
# two widths
for dk, dv in ((128, 64), (80, 40), (32, 64)):
    q, k, _ = wl.make_small(2, 3, 777, dk, seed=58, device="cuda")
    _, _, v = wl.make_small(2, 3, 777, dv, seed=59, device="cuda")
    ref = oracle.linear(to_f64(q), to_f64(k), to_f64(v), EPS)
    for variant in ("split", "cluster"):
        op = attn.LinFusionAttention(2, 3, 777, dv, eps=EPS, variant=variant, d_qk=dk)
        y = op.forward(q, k, v)
        torch.cuda.synchronize()
        assert_parity(y, ref, f"checked dk={dk} dv={dv} {variant}")
        assert attn.checked_violations(0) == 0
        op.close()
# token-sharded halves with the peer-summed apply
q, k, v = wl.make_small(1, 2, 1500, 40, seed=60, device="cuda")
ref = oracle_y(q, k, v)
ops = []
for lo, hi in ((0, 700), (700, 1500)):
    op = attn.LinFusionAttention(1, 2, hi - lo, 40, eps=EPS, variant="split")
    op.state(k[:, :, lo:hi].contiguous(), v[:, :, lo:hi].contiguous())
    ops.append(op)
torch.cuda.synchronize()
ptrs = [op.state_buffer()[0] for op in ops]
outs = [op.apply_peers(q[:, :, lo:hi].contiguous(), ptrs) for op, (lo, hi) in zip(ops, ((0, 700), (700, 1500)))]
torch.cuda.synchronize()
assert_parity(torch.cat(outs, dim=2), ref, "checked two shards")
assert attn.checked_violations(0) == 0
# the check itself: with the registered range of Y cut short by its last 3 rows, exactly the stores to those
# rows are reported and skipped (they keep their NaN), everything else is written as before
B, H, N, d = 1, 1, 300, 40
q, k, v = wl.make_small(B, H, N, d, seed=61, device="cuda")
ref = oracle_y(q, k, v)
op = attn.LinFusionAttention(B, H, N, d, eps=EPS, variant="split")
y = torch.full_like(q, float("nan"))
attn.checked_shrink_y(3 * d * 2)
op.forward(q, k, v, y)
torch.cuda.synchronize()
n = attn.checked_violations(0)
attn.checked_shrink_y(0)
assert n == 3 * d // 2, n            # one 4-byte store per pair of channels of the three rows
assert torch.isnan(y[0, 0, N - 3:].float()).all() and not torch.isnan(y[0, 0, :N - 3].float()).any()
assert_parity(y[:, :, :N - 3], ref[:, :, :N - 3], "rows inside the shortened range")
op.forward(q, k, v, y)
torch.cuda.synchronize()
assert attn.checked_violations(0) == 0 and not torch.isnan(y.float()).any()
op.close()
print("CHECKED_OK", runs)
'''


def test_checked_build_finds_no_access_outside_the_buffers():
    from paper_2409_02097_b200 import build
    lib = build.build_library(checked=True)
    env = dict(os.environ, LINFUSION_ATTN_LIB=lib)
    out = subprocess.run([sys.executable, "-c", CHILD, ROOT], env=env, capture_output=True, text=True, timeout=900)
    assert out.returncode == 0 and "CHECKED_OK" in out.stdout, out.stdout[-2000:] + out.stderr[-4000:]
