"""The benchmark's reference arm runs without a GPU: it times the fp64 oracle on host cores and
prints one JSON line with the agreed keys."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, cwd=ROOT,
                         timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "linear_attn_tokens_per_s" and d["unit"] == "tokens/s"
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["dtype"] == "f64"
    assert d["value"] > 0 and d["steps"] == 1 and d["gpu_launches"] == 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"] == d["e2e"]["value"]
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert d["config"]["workload"] == "sdxl_16k"


def _load_bench():
    import importlib.util
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_gpus_n_outside_torchrun_starts_n_ranks(monkeypatch):
    bench = _load_bench()
    argv = ["--gpus", "2", "--steps", "7", "--warmup", "3"]
    cmd = bench.launcher_command(argv, 2)
    assert cmd[0] == sys.executable and cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--standalone" in cmd and "--nnodes=1" in cmd and "--nproc-per-node=2" in cmd
    assert cmd[cmd.index("--local-addr") + 1] == "127.0.0.1"
    assert cmd[-len(argv) - 1] == os.path.join(ROOT, "bench.py") and cmd[-len(argv):] == argv
    calls = []
    monkeypatch.setattr(bench.subprocess, "call", lambda c: calls.append(c) or 0)
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    import torch
    monkeypatch.setattr(torch.cuda, "device_count", lambda: 2)
    ran = []
    monkeypatch.setattr(bench, "run_cuda", lambda a: ran.append(a))
    bench.main(argv)                                   # re-launches, does not run in this process
    assert calls == [cmd] and ran == []
    bench.main(["--gpus", "1", "--steps", "7"])        # one GPU: runs here
    assert len(calls) == 1 and len(ran) == 1
    monkeypatch.setenv("WORLD_SIZE", "2")              # already under a launcher: runs here
    bench.main(argv)
    assert len(calls) == 1 and len(ran) == 2
    monkeypatch.delenv("WORLD_SIZE")
    monkeypatch.setattr(torch.cuda, "device_count", lambda: 1)       # fewer devices than ranks: says so
    try:
        bench.main(argv)
        raise AssertionError("must refuse to start 2 ranks on 1 device")
    except SystemExit as e:
        assert "needs 2 CUDA devices" in str(e.code)
    monkeypatch.setattr(torch.cuda, "device_count", lambda: 2)
    monkeypatch.setattr(bench.subprocess, "call", lambda c: 3)
    try:
        bench.main(argv)
        raise AssertionError("a failing launcher must fail the benchmark")
    except SystemExit as e:
        assert e.code == 3


def test_rank_count_that_contradicts_gpus_is_an_error():
    env = dict(os.environ, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"],
                         capture_output=True, text=True, cwd=ROOT, env=env, timeout=600)
    assert out.returncode != 0
    assert "--gpus 2 but the launcher started 1 rank" in out.stderr
