"""Seeded synthetic Q, K, V tensors shaped like Stable Diffusion self-attention layers.

This module only produces inputs.  It holds none of the attention arithmetic and
is the one piece shared by the tests of the CPU oracle and of the CUDA library,
so that both sides see identical bits.

The paper evaluates on SD-v1.5 / SD-v2.1 / SD-XL activations driven by COCO and
LAION prompts; those models and datasets are not used here.  The stand-ins are
iid N(0, 1) tensors with the layers' shapes (B = 2 is the classifier-free
guidance pair), drawn in fp32 from a seeded generator and rounded to bf16
(round-to-nearest-even).  The "outlier" workloads scale 1 % of the tokens by 8
in Q, K and V alike (one Bernoulli(0.01) mask over (batch, token), shared by all
heads), the way a hidden-state outlier would hit all three projections.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import torch

BASE_SEED = 20240902


@dataclass(frozen=True)
class AttnShape:
    """One attention layer: tokens N = h*w, channels C = H*d, laid out [B, H, N, d]."""
    name: str
    B: int
    H: int
    N: int
    d: int
    outlier_frac: float = 0.0
    outlier_scale: float = 1.0

    @property
    def C(self) -> int:
        return self.H * self.d

    @property
    def tokens(self) -> int:
        return self.B * self.N

    @property
    def min_bytes(self) -> int:
        """Q, K, V read once and Y written once, bf16: 4 * B * N * C * 2 bytes."""
        return 4 * self.B * self.N * self.C * 2

    @property
    def flops(self) -> int:
        return 4 * self.B * self.N * self.C * self.d


def _s(name, H, N, d, **kw):
    return AttnShape(name=name, B=2, H=H, N=N, d=d, **kw)


# The five workload families; index 0 is the small case, index 4 the 16K-image case.
CONFIGS: List[List[AttnShape]] = [
    [_s("sd15_512_L1", 8, 4096, 40)],
    [_s("sd15_512_L1", 8, 4096, 40), _s("sd15_512_L2", 8, 1024, 80),
     _s("sd15_512_L3", 8, 256, 160), _s("sd15_512_L4", 8, 64, 160)],
    [_s("sd21_768_L1", 5, 9216, 64), _s("sd21_768_L2", 10, 2304, 64),
     _s("sd21_768_L3", 20, 576, 64), _s("sd21_768_L4", 20, 144, 64)],
    [_s("sdxl_2048_L1", 10, 16384, 64, outlier_frac=0.01, outlier_scale=8.0),
     _s("sdxl_2048_L2", 20, 4096, 64, outlier_frac=0.01, outlier_scale=8.0)],
    [_s("sdxl_16k_L1", 10, 524288, 64), _s("sdxl_16k_L2", 20, 131072, 64)],
]


def all_shapes() -> List[AttnShape]:
    out = []
    for cfg in CONFIGS:
        out.extend(cfg)
    return out


def find_shape(name: str) -> AttnShape:
    for s in all_shapes():
        if s.name == name:
            return s
    raise KeyError(name)


def make_qkv(shape: AttnShape, seed: int = BASE_SEED, device: str = "cpu",
             v_mean: float = 0.0):
    """Return bf16 (q, k, v), each [B, H, N, d] on ``device``, a pure function of
    (shape, seed, device type, v_mean).  ``v_mean`` shifts V so that |Y| ~ 1 cases can be made.
    """
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed))
    dims = (shape.B, shape.H, shape.N, shape.d)
    mask = None
    if shape.outlier_frac > 0.0:
        u = torch.rand((shape.B, 1, shape.N, 1), generator=g, device=dev, dtype=torch.float32)
        mask = torch.where(u < shape.outlier_frac,
                           torch.tensor(shape.outlier_scale, device=dev),
                           torch.tensor(1.0, device=dev))
    out = []
    for idx in range(3):
        t = torch.randn(dims, generator=g, device=dev, dtype=torch.float32)
        if idx == 2 and v_mean != 0.0:
            t += v_mean
        if mask is not None:
            t *= mask
        out.append(t.to(torch.bfloat16))
        del t
    return tuple(out)


def make_small(B: int, H: int, N: int, d: int, seed: int = BASE_SEED, device: str = "cpu",
               v_mean: float = 0.0, scale: float = 1.0):
    """Free-form shape for edge cases (ragged N, tiny N, odd head counts)."""
    q, k, v = make_qkv(AttnShape("adhoc", B, H, N, d), seed=seed, device=device, v_mean=v_mean)
    if scale != 1.0:
        q, k, v = (q.float() * scale).bfloat16(), (k.float() * scale).bfloat16(), \
                  (v.float() * scale).bfloat16()
    return q, k, v


def make_producer_inputs(B: int, H: int, N: int, d: int, seed: int = BASE_SEED, names=("q", "k", "v"),
                         device: str = "cpu", dtype=torch.bfloat16, x_mean: float = 0.0):
    """Layer input and module parameters for the attention fed from X (Sec. 3.1 implementation
    details; the trained weights the paper uses are not available, these are their stand-ins).

    Returns ``(x, w)``: ``x`` [B, N, C] ~ N(x_mean, 1) with C = H * d, and ``w[name]`` for every name asked
    for.  A name that starts with "t" gives a [B, N, C] tensor ~ N(0, 0.25) (a stand-in for the output
    of a non-linear branch); "b..." a bias [C] ~ N(0, 0.25); "g..." a LayerNorm scale [C] ~ N(1, 0.04);
    "e..." a LayerNorm shift [C] ~ N(0, 0.04); any other name a weight matrix [C, C] (row = input
    channel) ~ N(0, 1/C), so that x @ w is ~ N(0, 1) per element like the Q, K, V of the other
    workloads.  Everything is drawn in fp32 from one seeded generator and rounded to ``dtype``."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed))
    C = H * d
    x = (torch.randn((B, N, C), generator=g, device=dev, dtype=torch.float32) + x_mean).to(dtype)
    w = {}
    for name in names:
        if name.startswith("t"):
            t = 0.5 * torch.randn((B, N, C), generator=g, device=dev, dtype=torch.float32)
        elif name.startswith("b"):
            t = 0.5 * torch.randn((C,), generator=g, device=dev, dtype=torch.float32)
        elif name.startswith("g"):
            t = 1.0 + 0.2 * torch.randn((C,), generator=g, device=dev, dtype=torch.float32)
        elif name.startswith("e"):
            t = 0.2 * torch.randn((C,), generator=g, device=dev, dtype=torch.float32)
        else:
            t = torch.randn((C, C), generator=g, device=dev, dtype=torch.float32) / (C ** 0.5)
        w[name] = t.to(dtype)
    return x, w
