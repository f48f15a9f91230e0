#!/usr/bin/env python
"""Benchmark of the normalized non-causal linear attention at the SD-XL 16K-image shapes.

    python bench.py --gpus N --steps K --warmup W            # the CUDA library
    python bench.py --impl reference --steps K --warmup W    # the fp64 CPU oracle, on host cores

One step = one forward of each attention level of the 16384x8192 SD-XL workload
(N = 524288, C = 640, H = 10 and N = 131072, C = 1280, H = 20; B = 2, d = 64, bf16), i.e. every
stage of the path (split-N state, fixed-order reduction, apply) over one batch.  Prints ONE JSON
line: tokens/s over all GPUs with inputs resident in HBM, the same through the host-buffer entry
point (copies inside the timed region), the roofline of the slowest kernel, and the oracle timed
on a bounded sample as a CPU baseline.

With N > 1 there is one rank per GPU (started by torchrun, or by this script itself when it is run
plainly with --gpus N).  Default there is the token-sharded forward of Sec. 4.3: every rank owns
the N tokens of the two levels as its run of a sequence of world x N tokens, builds the state of its
own K/V tokens, the ranks sum their states (one all-reduce of B*H*d*(d+1) fp32 per level, whatever
N is) and every rank applies the sum to its own Q tokens: per-GPU work is fixed, the exchange is
the constant-size one the paper points out (weak scaling).  `--parallelism replicas` runs
independent batches instead (no data-path collective); `--parallelism token_sharded_peers` lets the
apply step read the peers' states itself over NVLink (symmetric memory, plain loads).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "linear_attn_tokens_per_s"
UNIT = "tokens/s"
WORKLOAD = "sdxl_16k"          # both attention levels of the 16384x8192 SD-XL workload
KERNEL_TIMING_STRIDE = 8
NOMINAL_HBM_GBS = 8000.0


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def recorded_traffic(kernel: str, shape: str):
    """DRAM bytes per launch from the committed ncu summary, or None when the kernel sources
    have changed since the counters were taken."""
    import hashlib
    try:
        csrc = os.path.join(ROOT, "paper_2409_02097_b200", "csrc")
        h = hashlib.sha256()
        for name in ("common.cuh", "stream_kernels.cuh"):
            with open(os.path.join(csrc, name), "rb") as f:
                h.update(f.read())
        sha = h.hexdigest()[:16]
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            for line in f:
                parts = line.split()
                if len(parts) == 4 and parts[0] == kernel and parts[1] == shape and parts[3] == sha:
                    return int(parts[2])
    except Exception:
        pass
    return None


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the benchmark runs (read-only)."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_ms: int = 50):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", str(period_ms), "-i", str(gpu_index)],
                stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, windows):
        """`windows`: name -> (t0, t1) in time.time() seconds; returns name -> summary."""
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        rows = []
        try:
            self.file.flush()
            with open(self.file.name) as f:
                for line in f:
                    parts = [p.strip() for p in line.split(",")]
                    if len(parts) < 9:
                        continue
                    try:
                        ts = time.mktime(time.strptime(parts[0].split(".")[0], "%Y/%m/%d %H:%M:%S"))
                        ts += float("0." + parts[0].split(".")[1]) if "." in parts[0] else 0.0
                        rows.append((ts, float(parts[1]), float(parts[2]), float(parts[3]), parts[4:9]))
                    except Exception:
                        continue
            os.unlink(self.file.name)
        except Exception:
            pass
        return {name: self._summarize(rows, t0, t1, name) for name, (t0, t1) in windows.items()}

    @staticmethod
    def _summarize(rows, t0, t1, name):
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        inside = [r for r in rows if t0 - 0.05 <= r[0] <= t1 + 0.05]
        window = name + "_region"
        if len(inside) < 3:
            # Too short a region for the sampler: use the samples taken under load in this run.
            pmax = max(r[3] for r in rows)
            inside = [r for r in rows if r[3] >= 0.5 * pmax]
            window = "whole_run_under_load"
        sm = sorted(r[1] for r in inside)
        reasons = set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in inside:
            for name, val in zip(names, r[4][1:]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": inside[0][2], "reasons": sorted(reasons),
                "samples": len(inside), "window": window,
                "power_w_max": max(r[3] for r in inside)}


def time_oracle_sample(max_seconds: float = 15.0):
    """Time the oracle, as it stands, on (batch, head) slabs of the larger 16K level, one slab after
    another until about `max_seconds` of oracle time have been spent (or, if one slab alone would
    take longer, on a leading run of its tokens).  Input generation is not timed.  Returns a dict."""
    import numpy as np
    import torch
    import oracle
    from paper_2409_02097_b200 import workloads as wl

    shape = wl.find_shape("sdxl_16k_L1")
    g = torch.Generator().manual_seed(wl.BASE_SEED)
    probe_n = 16384
    def draw(n):
        return [torch.randn((n, shape.d), generator=g).bfloat16().double().numpy() for _ in range(3)]
    q, k, v = draw(probe_n)
    oracle.linear(q, k, v, 1e-6)                      # load the library, warm the threads
    t = time.perf_counter()
    oracle.linear(q, k, v, 1e-6)
    per_token = (time.perf_counter() - t) / probe_n
    n = int(min(shape.N, max(probe_n, max_seconds / max(per_token, 1e-12))))
    slabs, dt = 0, 0.0
    q, k, v = draw(n)                                 # the oracle's time does not depend on the values
    while slabs < shape.B * shape.H and (slabs == 0 or dt + dt / slabs <= max_seconds):
        t = time.perf_counter()
        y = oracle.linear(q, k, v, 1e-6)
        dt += time.perf_counter() - t
        slabs += 1
        assert np.isfinite(y).all()
    # A slab carries one of H heads of every token: n slab-rows are n / H tokens of the layer.
    tokens = slabs * n / shape.H
    return {"value": tokens / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{slabs} of {shape.B * shape.H} (b,h) slabs of sdxl_16k_L1, {n} of {shape.N} "
                      f"tokens each, fp64, {dt:.2f} s of oracle time",
            "seconds": dt, "n": n, "slabs": slabs}


def run_reference(args):
    """The reference arm: the CPU oracle on a bounded sample per step."""
    import numpy as np
    import torch
    import oracle
    from paper_2409_02097_b200 import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    shape = wl.find_shape("sdxl_16k_L1")
    probe = time_oracle_sample(max_seconds=2.0)
    per_token_row = probe["seconds"] / (probe["n"] * probe["slabs"])
    budget = 150.0 / max(1, args.steps + args.warmup)
    n = int(min(shape.N, max(4096, budget / per_token_row)))
    g = torch.Generator().manual_seed(wl.BASE_SEED)
    q, k, v = [torch.randn((n, shape.d), generator=g).bfloat16().double().numpy() for _ in range(3)]
    for _ in range(args.warmup):
        oracle.linear(q, k, v, 1e-6)
    t = time.perf_counter()
    for _ in range(args.steps):
        y = oracle.linear(q, k, v, 1e-6)
    dt = time.perf_counter() - t
    assert np.isfinite(y).all()
    value = (n / shape.H) * args.steps / dt
    sample = (f"per step: {n} of {shape.N} tokens of one (b,h) slab of sdxl_16k_L1, fp64 oracle "
              f"on host cores")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def launcher_command(argv, gpus):
    """The command that starts one rank per GPU on this node for `python bench.py <argv>`."""
    return [sys.executable, "-m", "torch.distributed.run", "--standalone", "--nnodes=1",
            f"--nproc-per-node={gpus}", "--local-addr", "127.0.0.1",
            os.path.join(ROOT, "bench.py")] + list(argv)


def maybe_relaunch(args, argv):
    """`python bench.py --gpus N` with N > 1 outside torchrun: start the N ranks ourselves.
    Returns True when this process was replaced by (and has waited for) the launcher."""
    if args.gpus <= 1 or "WORLD_SIZE" in os.environ:
        return False
    if args.impl == "cuda":
        import torch
        if torch.cuda.device_count() < args.gpus:
            raise SystemExit(f"bench.py: --gpus {args.gpus} needs {args.gpus} CUDA devices on this node, "
                             f"{torch.cuda.device_count()} visible")
    rc = subprocess.call(launcher_command(argv, args.gpus))
    if rc != 0:
        raise SystemExit(rc)
    return True


def run_cuda(args):
    import torch
    from paper_2409_02097_b200 import attn, build, sharding, workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention has no CPU path")
    if torch.cuda.device_count() < (int(os.environ.get("LOCAL_WORLD_SIZE", world))):
        raise SystemExit(f"bench.py: --gpus {args.gpus} needs {world} CUDA devices on this node, "
                         f"{torch.cuda.device_count()} visible")
    parallelism = args.parallelism
    if parallelism == "auto":
        parallelism = "token_sharded" if world > 1 else "single"
    if parallelism != "single" and (args.layout != "head_major"):
        raise SystemExit("bench.py: the token-sharded modes time the head-major layout")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build.build_library()
    if dist is not None:
        dist.barrier()
    attn.load_library()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    shapes = wl.CONFIGS[4]
    if args.workload == "sdxl_16k_eighth":
        # Same layers at one eighth of the tokens: small enough for a multi-pass profiler capture,
        # still several times the L2 capacity.  Not a benchmark workload.
        shapes = [wl.AttnShape(s.name + "_eighth", s.B, s.H, s.N // 8, s.d) for s in shapes]
    elif args.workload == "sdxl_16k_L2":
        # The smaller of the two levels alone, full size (2.7 GB on the device): for profiler
        # captures of DRAM counters over whole launches.  Not a benchmark workload.
        shapes = shapes[1:]
    eps = 1e-6
    layers = []
    sharded = parallelism in ("token_sharded", "token_sharded_peers")
    symm = None
    for i, s in enumerate(shapes):
        q, k, v = wl.make_qkv(s, seed=wl.BASE_SEED + 100 * rank + i, device=f"cuda:{local_rank}")
        if args.layout == "token_major":          # [B, N, H, d]: what a UNet holds before splitting heads
            q, k, v = (t.permute(0, 2, 1, 3).contiguous() for t in (q, k, v))
        if args.dtype == "fp16":
            q, k, v = (t.half() for t in (q, k, v))
        y = torch.empty_like(q)
        if sharded:
            # This rank's run of a sequence of world * N tokens (its own seeded tokens).
            sh = sharding.TokenShardedAttention(s.B, s.H, s.N, s.d, eps=eps, device=local_rank,
                                                variant="stream", dtype=args.dtype,
                                                symmetric=(parallelism == "token_sharded_peers"))
            layers.append((s, sh.op, q, k, v, y, sh))
        else:
            op = attn.LinFusionAttention(s.B, s.H, s.N, s.d, eps=eps, device=local_rank, layout=args.layout,
                                         dtype=args.dtype)
            layers.append((s, op, q, k, v, y, None))
    tokens_per_step = sum(s.tokens for s in shapes)
    launches_per_step = sum((4 if sh is not None else op.launches_per_forward) for _, op, *_, sh in layers)

    # The all-reduce (or the peers' barrier) of every KERNEL_TIMING_STRIDE-th step is bracketed
    # with events so that the exchange's share of the step can be reported.
    exchange_events = []
    step_index = [0]

    def step():
        sample = sharded and step_index[0] % KERNEL_TIMING_STRIDE == 0
        step_index[0] += 1
        for _, op, q, k, v, y, sh in layers:
            if sh is None:
                op.forward(q, k, v, y)
            else:
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)] if sample else None
                if parallelism == "token_sharded":
                    sh.forward(q, k, v, y, events=ev)
                else:
                    sh.forward_symmetric(q, k, v, y, events=ev)
                if ev is not None:
                    exchange_events.append((_.name, ev))

    sampler = ClockSampler(local_rank) if rank == 0 else None
    for _ in range(max(args.warmup, 3)):
        step()
    exchange_events.clear()
    step_index[0] = 0
    # Per-kernel durations: CUDA events around each kernel of every KERNEL_TIMING_STRIDE-th step of
    # the timed region (an event record between two kernels undoes their chained launch, so timing
    # every step would slow the steps it measures).
    if not sharded:
        for _, op, *_ in layers:
            op.enable_kernel_timing(min(args.steps, 4096))
            op.set_kernel_timing_stride(KERNEL_TIMING_STRIDE)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    barrier()
    t1 = time.time()
    ms = ev0.elapsed_time(ev1)
    for _, op, *_ in layers:
        assert op.status() == attn.OK, "a device-side wait expired"
    if dist is not None:
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    value = world * tokens_per_step * args.steps / (ms * 1e-3)
    exchange = None
    if sharded:
        state_bytes = sum(s.B * s.H * s.d * (s.d + 1) * 4 for s in shapes)
        exchange = {"kind": "nccl all_reduce (sum) of S|z" if parallelism == "token_sharded"
                            else "peers' S|z read by the apply step (symmetric memory, plain loads)",
                    "bytes_per_step_per_rank": state_bytes, "independent_of_N": True}
        if exchange_events:
            n_sampled = len(exchange_events) // len(shapes)
            ex_ms = sum(ev[1].elapsed_time(ev[2]) for _, ev in exchange_events) / n_sampled
            exchange["ms_per_step"] = ex_ms
            exchange["share_of_step"] = ex_ms / (ms / args.steps)
            exchange["sampled_steps"] = n_sampled

    kernel_times_taken = {}
    if not sharded:
        for s_, op, *_ in layers:
            kernel_times_taken[s_.name] = op.kernel_times()
    # A second, longer region of back-to-back steps: the board reaches its power limit within a
    # few hundred milliseconds and the SM clock settles below its maximum, so the burst above and
    # the steady state differ.  Timed the same way; its clock samples come from inside its window.
    sustained = None
    if args.sustained_seconds > 0:
        n_sus = max(args.steps, int(args.sustained_seconds / max(ms / args.steps * 1e-3, 1e-6)) + 1)
        if not sharded:
            for _, op, *_ in layers:
                op.enable_kernel_timing(0)          # undisturbed chained launches
        barrier()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ts0 = time.time()
        s0.record()
        for _ in range(n_sus):
            step()
        s1.record()
        barrier()
        ts1 = time.time()
        ms_sus = s0.elapsed_time(s1)
        if dist is not None:
            t = torch.tensor([ms_sus], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms_sus = float(t.item())
        step_bytes_ = sum(s.min_bytes for s in shapes)
        sustained = {"steps": n_sus, "ms_per_step": ms_sus / n_sus, "seconds": ms_sus * 1e-3,
                     "value": world * tokens_per_step * n_sus / (ms_sus * 1e-3), "unit": UNIT,
                     "hbm_gbs_whole_path": step_bytes_ * n_sus / (ms_sus * 1e-3) / 1e9,
                     "hbm_frac_of_nominal_8TBps": step_bytes_ * n_sus / (ms_sus * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                     "window": (ts0, ts1)}

    # Per-kernel durations recorded inside the timed region.
    peak, peak_kind = measured_peak_gbs()
    kernels = []
    names = ["stream_state_kernel", "stream_reduce_kernel", "stream_apply_kernel"]
    if sharded:
        # The two halves, each bracketed as a whole on the sampled steps (state kernel + reduction;
        # operand packing + apply kernel).
        for s in shapes:
            evs = [ev for name, ev in exchange_events if name == s.name]
            for label, i in (("stream_state_kernel+stream_reduce_kernel", 0), ("stream_pack_kernel+stream_apply_kernel", 2)):
                if not evs:
                    continue
                avg_ms = sum(ev[i].elapsed_time(ev[i + 1]) for ev in evs) / len(evs)
                algo = 2 * s.B * s.N * s.C * 2
                kernels.append({"kernel": label, "shape": s.name, "avg_ms": avg_ms, "algorithmic_bytes": algo,
                                "gbs": algo / (avg_ms * 1e-3) / 1e9})
    for s, op, *_ in layers:
        if sharded or kernel_times_taken.get(s.name) is None:
            continue
        sums, calls = kernel_times_taken[s.name]
        # three launches: state, reduction, apply; two when the apply kernel takes over the reduction
        op_names = names if op.launches_per_forward == 3 else [names[0], names[2]]
        for name, total in zip(op_names, sums):
            if calls == 0:
                continue
            avg_ms = total / calls
            algo = 2 * s.B * s.N * s.C * 2 if name != "stream_reduce_kernel" else 0
            kernels.append({"kernel": name, "shape": s.name, "avg_ms": avg_ms,
                            "algorithmic_bytes": algo,
                            "gbs": (algo / (avg_ms * 1e-3) / 1e9) if avg_ms > 0 else None})
    dominant = max(kernels, key=lambda r: r["avg_ms"]) if kernels else None
    roofline = None
    if dominant is not None:
        roofline = {"bound": "hbm", "kernel": dominant["kernel"], "shape": dominant["shape"],
                    "achieved": dominant["gbs"], "peak": peak, "peak_kind": f"of {peak_kind}",
                    "unit": "GB/s", "frac": dominant["gbs"] / peak,
                    "traffic": recorded_traffic(dominant["kernel"], dominant["shape"]),
                    "frac_of_nominal_8TBps": dominant["gbs"] / NOMINAL_HBM_GBS}
    step_bytes = sum(s.min_bytes for s in shapes)
    path_gbs = step_bytes * args.steps / (ms * 1e-3) / 1e9

    # End to end through the host-buffer entry point: H2D of Q, K, V and D2H of Y every step.
    e2e = None
    if not args.no_e2e and not sharded:
        host = []
        for s, op, q, k, v, y, _ in layers:
            hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
            hy = torch.empty_like(hq).pin_memory()
            host.append((op, hq, hk, hv, hy))
        def e2e_step():
            for op, hq, hk, hv, hy in host:
                op.forward_host(hq, hk, hv, hy)
        e2e_step()                      # allocates the staging buffers
        e2e_step()
        barrier()
        k_e2e = max(1, min(args.steps, args.e2e_steps))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(k_e2e):
            e2e_step()
        e1.record()
        barrier()
        ms_e2e = e0.elapsed_time(e1)
        if dist is not None:
            t = torch.tensor([ms_e2e], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms_e2e = float(t.item())
        h2d = sum(3 * s.B * s.N * s.C * 2 for s in shapes)
        d2h = sum(s.B * s.N * s.C * 2 for s in shapes)
        e2e = {"value": world * tokens_per_step * k_e2e / (ms_e2e * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": k_e2e,
               "ms_per_step": ms_e2e / k_e2e}
        del host

    clocks = None
    if sampler is not None:
        # The timed region is often shorter than the sampler's period; the sustained region follows
        # it directly, so the two together are the window the clock record describes.
        windows = {"timed": (t0, t1)}
        if sustained is not None:
            windows["sustained"] = sustained["window"]
            windows["timed"] = (t0, sustained["window"][1])
        rec = sampler.stop(windows)
        clocks = rec["timed"]
        if sustained is not None:
            sc = rec["sustained"]
            sustained.update({"sm_mhz_median": sc["sm_mhz"], "sm_max_mhz": sc["sm_max_mhz"], "reasons": sc["reasons"],
                              "clock_samples": sc["samples"], "power_w_max": sc.get("power_w_max"),
                              "ms_per_step_x_sm_mhz": (sustained["ms_per_step"] * sc["sm_mhz"]) if sc["sm_mhz"] else None})
    if sustained is not None:
        sustained.pop("window", None)

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cb = time_oracle_sample(15.0)
        cpu_baseline = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": args.dtype, "data": "synthetic",
            "config": {"workload": args.workload,
                       "shapes": [{"name": s.name, "B": s.B, "H": s.H, "N": s.N, "d": s.d}
                                  for s in shapes],
                       "variant": [op.variant for _, op, *_ in layers],
                       "l2": "inputs larger than L2 (%.2f GB touched per step)" % (step_bytes / 1e9),
                       "layout": args.layout,
                       "parallelism": {"single": "one GPU",
                                       "replicas": f"independent batches x{world} (no data-path collective)",
                                       "token_sharded": f"token-sharded x{world}: each rank owns N tokens of a "
                                                        f"{world}xN-token sequence; one all-reduce of S|z per level",
                                       "token_sharded_peers": f"token-sharded x{world}: the apply step sums the "
                                                              f"peers' S|z itself over NVLink"}[parallelism],
                       "exchange": exchange},
            "tokens_per_s_per_gpu": value / world,
            "hbm_gbs_whole_path": path_gbs,
            "hbm_frac_of_nominal_8TBps": path_gbs / NOMINAL_HBM_GBS,
            "hbm_frac_of_measured_copy": path_gbs / peak,
            "sustained": sustained,
            "roofline": roofline, "kernels": kernels,
            "kernel_timing": f"CUDA events around each kernel of every {KERNEL_TIMING_STRIDE}th step of the timed region",
            "cpu_baseline": cpu_baseline, "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def run_sweep(args):
    """Every attention level of the five workload families, every kernel variant that serves it.
    Shapes smaller than the L2 cache are cycled through enough distinct buffer sets to exceed it;
    one JSON line per (shape, variant), `effective_gbs` = minimum traffic / time."""
    import torch
    from paper_2409_02097_b200 import attn, build, workloads as wl

    build.build_library()
    torch.cuda.set_device(0)
    peak, _ = measured_peak_gbs()
    seen = set()
    configs = list(wl.CONFIGS)
    if args.shape:
        # extra shapes given on the command line (beyond the five workload families): B,H,N,d each
        extra = []
        for spec in args.shape:
            B, H, N, d = (int(x) for x in spec.split(","))
            extra.append(wl.AttnShape(f"B{B}_H{H}_N{N}_d{d}", B, H, N, d))
        configs = [extra]
    for cfg_idx, cfg in enumerate(configs):
        for s in cfg:
            if s.name in seen or (args.only and s.name != args.only):
                continue
            seen.add(s.name)
            sets = max(1, min(64, -(-400_000_000 // s.min_bytes)))
            if s.min_bytes > (2 << 30):
                sets = 1
            bufs = []
            for r in range(sets):
                q, k, v = wl.make_qkv(s, seed=wl.BASE_SEED + r, device="cuda:0")
                if args.layout == "token_major":
                    q, k, v = (t.permute(0, 2, 1, 3).contiguous() for t in (q, k, v))
                if args.dtype == "fp16":
                    q, k, v = (t.half() for t in (q, k, v))
                bufs.append((q, k, v, torch.empty_like(q)))
            variants = ["auto", "split"] + (["stream"] if s.d == 64 else []) + \
                       (["fused"] if s.d in (40, 64, 80, 160) else []) + (["cluster"] if s.N <= 16384 else [])
            for variant in variants:
                op = attn.LinFusionAttention(s.B, s.H, s.N, s.d, device=0, variant=variant, layout=args.layout,
                                             dtype=args.dtype)
                steps = max(20, min(args.steps, int(2e10 // s.min_bytes)))
                for i in range(5):
                    op.forward(*bufs[i % sets])
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for i in range(steps):
                    op.forward(*bufs[i % sets])
                e1.record()
                torch.cuda.synchronize()
                assert op.status() == attn.OK
                us = 1e3 * e0.elapsed_time(e1) / steps
                gbs = s.min_bytes / (us * 1e-6) / 1e9
                print(json.dumps({
                    "config": cfg_idx + 1, "shape": s.name, "B": s.B, "H": s.H, "N": s.N, "d": s.d,
                    "requested": variant, "variant": op.variant, "launches": op.launches_per_forward,
                    "layout": args.layout, "dtype": args.dtype,
                    "us_per_forward": us, "tokens_per_s": s.tokens / (us * 1e-6),
                    "effective_gbs": gbs, "frac_of_nominal_8TBps": gbs / NOMINAL_HBM_GBS,
                    "frac_of_measured_copy": gbs / peak, "buffer_sets": sets,
                    "hbm_resident": ("no: cycled through %d buffer sets (%.0f MB) to exceed L2"
                                     % (sets, sets * s.min_bytes / 1e6)) if sets > 1 else
                                    "single set, larger than L2",
                    "roofline_us_at_8TBps": s.min_bytes / 8e12 * 1e6}), flush=True)
                op.close()
            del bufs
            torch.cuda.empty_cache()


def measured_tensor_peaks():
    """(burst, sustained) dense bf16 TFLOP/s from MEASURED_PEAKS.json, else the stated fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"]), "measured"
    except Exception:
        return 1590.0, 1400.0, "fallback"


def run_from_x(args):
    """The module fed from the layer input X (projections fused into the state and apply kernels),
    one JSON line per shape: each kernel's time and tensor-core rate, the whole forward with and
    without the non-linear branches, and beside it the un-fused route — Q, K, V from a library GEMM
    (torch.matmul), written to and read back from device memory, then the attention kernels."""
    import torch
    from paper_2409_02097_b200 import attn, build, workloads as wl

    build.build_library()
    torch.cuda.set_device(0)
    burst, sustained, kind = measured_tensor_peaks()
    names = ("q_lin", "q_w1", "b_q", "g_q", "e_q", "k_lin", "k_w1", "b_k", "g_k", "e_k", "v")
    shapes = [wl.find_shape(n) for n in (args.only.split(",") if args.only else
                                         ["sdxl_2048_L1", "sdxl_2048_L2", "sdxl_16k_L2", "sdxl_16k_L1"])]
    for s in shapes:
        assert s.d == 64
        B, H, N, C = s.B, s.H, s.N, s.C
        x, w = wl.make_producer_inputs(B, H, N, 64, seed=wl.BASE_SEED, names=names, device="cuda:0")
        w = dict(w)
        for side in ("q", "k"):
            w[f"{side}_b1"], w[f"{side}_gamma"], w[f"{side}_beta"] = w.pop(f"b_{side}"), w.pop(f"g_{side}"), w.pop(f"e_{side}")
        w_lin = {"q_lin": w["q_lin"], "k_lin": w["k_lin"], "v": w["v"]}
        op = attn.LinFusionAttention(B, H, N, 64, device=0, variant="stream", layout="token_major")
        y = torch.empty_like(x)
        t = torch.empty_like(x)
        tokens = B * N
        steps = max(5, min(args.steps, int(4e13 // (tokens * 10 * C * C))))

        def timed(fn):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(steps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / steps

        ms_state = timed(lambda: op.state_x(x, w["k_lin"], w["v"]))
        ms_apply = timed(lambda: op.apply_x(x, w["q_lin"], None, y))
        ms_branch = timed(lambda: op.branch_x(x, w["k_w1"], w["k_b1"], w["k_gamma"], w["k_beta"], 1e-5, 0.01, t))
        ms_lin = timed(lambda: op.forward_x(x, w_lin, y=y))
        ms_full = timed(lambda: op.forward_x(x, w, y=y))
        assert op.status() == attn.OK
        # un-fused: library GEMMs produce Q, K, V in device memory, then the three attention kernels
        q = torch.empty_like(x)
        k = torch.empty_like(x)
        v = torch.empty_like(x)
        x2 = x.view(B * N, C)

        def unfused():
            torch.matmul(x2, w["q_lin"], out=q.view(B * N, C))
            torch.matmul(x2, w["k_lin"], out=k.view(B * N, C))
            torch.matmul(x2, w["v"], out=v.view(B * N, C))
            op.forward(q.view(B, N, H, 64), k.view(B, N, H, 64), v.view(B, N, H, 64), y.view(B, N, H, 64))
        ms_unfused = timed(unfused)
        ms_gemm = timed(lambda: torch.matmul(x2, w["v"], out=v.view(B * N, C)))
        proj = 2.0 * tokens * C * C             # flops of one C x C projection
        attn_half = 2.0 * tokens * C * 64       # flops of the state (or the apply) contraction
        tf = lambda flops, ms: flops / (ms * 1e-3) / 1e12
        line = {
            "mode": "from_x", "shape": s.name, "B": B, "H": H, "N": N, "C": C, "dtype": "bf16", "steps": steps,
            "peak_tflops": {"burst": burst, "sustained": sustained, "kind": "of " + kind},
            "kernels": {
                "producer_state2_kernel+reduce": {"ms": ms_state, "tflops": tf(2 * proj + attn_half, ms_state)},
                "pack+producer_apply_kernel": {"ms": ms_apply, "tflops": tf(proj + attn_half, ms_apply)},
                "producer_hidden_kernel+norm (one branch)": {"ms": ms_branch, "tflops": tf(proj, ms_branch)},
            },
            "forward_x_linear_branches": {"ms": ms_lin, "tflops": tf(3 * proj + 2 * attn_half, ms_lin),
                                          "tokens_per_s": tokens / (ms_lin * 1e-3)},
            "forward_x_with_non_linear_branches": {"ms": ms_full, "tflops": tf(5 * proj + 2 * attn_half, ms_full),
                                                   "tokens_per_s": tokens / (ms_full * 1e-3)},
            "unfused_library_gemm_then_attention": {"ms": ms_unfused, "tokens_per_s": tokens / (ms_unfused * 1e-3),
                                                    "one_library_gemm_ms": ms_gemm, "one_library_gemm_tflops": tf(proj, ms_gemm)},
            "roofline": {"bound": "tensor", "kernel": "producer_state2_kernel", "achieved": tf(2 * proj + attn_half, ms_state),
                         "peak": sustained, "peak_kind": "of " + kind + " (sustained bf16)", "unit": "TFLOP/s",
                         "frac": tf(2 * proj + attn_half, ms_state) / sustained, "traffic": None},
        }
        print(json.dumps(line), flush=True)
        op.close()
        del x, w, y, t, q, k, v
        torch.cuda.empty_cache()


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default=WORKLOAD, choices=[WORKLOAD, "sdxl_16k_eighth", "sdxl_16k_L2"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--sustained-seconds", type=float, default=2.5,
                    help="length of the second, back-to-back region timed after the --steps region (0: none)")
    ap.add_argument("--parallelism", default="auto",
                    choices=["auto", "single", "replicas", "token_sharded", "token_sharded_peers"],
                    help="auto: token_sharded when --gpus > 1")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layout", default="head_major", choices=["head_major", "token_major"],
                    help="[B,H,N,d] (default, the benchmark's layout) or [B,N,H,d]")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp16"],
                    help="storage type of Q, K, V, Y (the headline number is bf16)")
    ap.add_argument("--sweep", action="store_true",
                    help="time every shape of the five workload families with every variant")
    ap.add_argument("--only", default="", help="with --sweep / --from-x: restrict to one shape, e.g. sd15_512_L1")
    ap.add_argument("--shape", action="append", default=[], metavar="B,H,N,d",
                    help="with --sweep: time this shape instead of the workload families (may be given several times)")
    ap.add_argument("--from-x", action="store_true",
                    help="time the module fed from the layer input X (fused projections) beside the un-fused route")
    argv = sys.argv[1:] if argv is None else argv
    args = ap.parse_args(argv)
    if args.from_x:
        return run_from_x(args)
    if args.sweep:
        run_sweep(args)
    elif maybe_relaunch(args, argv):
        return
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
