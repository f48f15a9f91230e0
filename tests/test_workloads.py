"""The synthetic input generator: shapes of the five workload families, determinism, recipe."""
import torch

from paper_2409_02097_b200 import workloads as wl


def test_config_table_matches_the_workload_families():
    shapes = wl.all_shapes()
    assert len(shapes) == 13 and len({s.name for s in shapes}) == 12
    assert [len(c) for c in wl.CONFIGS] == [1, 4, 4, 2, 2]
    for s in shapes:
        assert s.B == 2 and s.C in (320, 640, 1280)
    big = wl.find_shape("sdxl_16k_L1")
    assert (big.N, big.H, big.d, big.C) == (1024 * 512, 10, 64, 640)
    assert big.min_bytes == 4 * 2 * 524288 * 640 * 2 == 5368709120
    assert wl.find_shape("sdxl_16k_L2").min_bytes == 2684354560
    assert wl.find_shape("sd15_512_L1").flops == 4 * 2 * 4096 * 320 * 40


def test_generator_is_deterministic_and_bf16():
    s = wl.AttnShape("t", 2, 3, 100, 40)
    a = wl.make_qkv(s, seed=7)
    b = wl.make_qkv(s, seed=7)
    c = wl.make_qkv(s, seed=8)
    for x, y in zip(a, b):
        assert x.dtype == torch.bfloat16 and x.shape == (2, 3, 100, 40)
        assert torch.equal(x, y)
    assert not torch.equal(a[0], c[0])
    assert not torch.equal(a[0], a[1]) and not torch.equal(a[1], a[2])


def test_values_are_standard_normal():
    q, k, v = wl.make_qkv(wl.AttnShape("t", 2, 4, 4096, 64), seed=1)
    for t in (q, k, v):
        f = t.float()
        assert abs(f.mean().item()) < 0.01 and abs(f.std().item() - 1.0) < 0.01
    _, _, v1 = wl.make_qkv(wl.AttnShape("t", 2, 4, 4096, 64), seed=1, v_mean=1.0)
    assert abs(v1.float().mean().item() - 1.0) < 0.01


def test_outlier_rows_hit_all_three_tensors_and_all_heads():
    s = wl.AttnShape("t", 2, 4, 8192, 64, outlier_frac=0.01, outlier_scale=8.0)
    q, k, v = wl.make_qkv(s, seed=3)
    plain = wl.make_qkv(wl.AttnShape("t", 2, 4, 8192, 64), seed=3)
    del plain
    rms = lambda t: t.float().pow(2).mean(dim=(1, 3)).sqrt()      # [B, N]
    hot = rms(q) > 4.0
    frac = hot.float().mean().item()
    assert 0.005 < frac < 0.02
    assert torch.equal(hot, rms(k) > 4.0) and torch.equal(hot, rms(v) > 4.0)
    per_head = q.float().pow(2).mean(dim=3).sqrt()               # [B, H, N]
    assert ((per_head > 4.0) == hot[:, None, :]).all()


def test_generated_inputs_match_the_committed_checksums():
    """The recipe is pinned: the CPU generator must reproduce, bit for bit, the inputs whose checksums are
    committed (a change of the generator's stream, of the draw order or of the rounding shows up here)."""
    import importlib.util
    import json
    import os
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_workload_checksums", os.path.join(here, "make_workload_checksums.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    with open(os.path.join(here, "workload_checksums.json")) as f:
        want = json.load(f)["cases"]
    got = mod.cases()
    assert got.keys() == want.keys()
    for name in want:
        assert got[name] == want[name], name
