"""Writes tests/golden/workload_checksums.json: checksums of the seeded synthetic inputs that
``paper_2409_02097_b200.workloads`` generates on the CPU, which pin the input recipe (the generator's
stream, the draw order of the tensors, the outlier mask, the rounding to 16 bits) across library
versions.  Calls the input generator only — none of the attention arithmetic, neither the oracle nor
the CUDA library.

    python tests/golden/make_workload_checksums.py
"""
import hashlib
import json
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from paper_2409_02097_b200 import workloads as wl  # noqa: E402


def digest(t: torch.Tensor) -> str:
    """sha256 of the tensor's 16-bit words in memory order (little endian)."""
    return hashlib.sha256(t.contiguous().view(torch.int16).numpy().tobytes()).hexdigest()[:32]


def cases():
    out = {}
    # the small workload family whole; one slab-sized piece of a mid-size one with outlier rows; the producers' inputs
    for name, shape, seed in [("sd15_512_L4", wl.find_shape("sd15_512_L4"), wl.BASE_SEED),
                              ("sd21_768_L4", wl.find_shape("sd21_768_L4"), wl.BASE_SEED + 2),
                              ("outliers_2x2x4096x64", wl.AttnShape("t", 2, 2, 4096, 64, outlier_frac=0.01, outlier_scale=8.0),
                               wl.BASE_SEED + 3)]:
        q, k, v = wl.make_qkv(shape, seed=seed, device="cpu")
        out[name] = {"seed": seed, "shape": [shape.B, shape.H, shape.N, shape.d], "q": digest(q), "k": digest(k), "v": digest(v),
                     "q_first4": [float(x) for x in q.flatten()[:4]]}
    q, k, v = wl.make_small(1, 2, 65, 40, seed=11, device="cpu", v_mean=1.0)
    out["small_1x2x65x40_vmean1"] = {"seed": 11, "q": digest(q), "k": digest(k), "v": digest(v)}
    x, w = wl.make_producer_inputs(1, 2, 33, 64, seed=13, names=("q_lin", "b_q", "g_q", "e_q", "tq"), device="cpu")
    out["producer_1x2x33x64"] = {"seed": 13, "x": digest(x), **{n: digest(t) for n, t in w.items()}}
    return out


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "workload_checksums.json")
    data = {"_about": "sha256 (first 32 hex digits) of the 16-bit words of the CPU-generated synthetic inputs; "
                      "written by tests/golden/make_workload_checksums.py, which calls the input generator only",
            "torch": torch.__version__.split("+")[0], "cases": cases()}
    with open(path, "w") as f:
        json.dump(data, f, indent=1)
    print(path)
