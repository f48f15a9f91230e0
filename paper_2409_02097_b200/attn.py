"""ctypes binding over the C ABI in ``include/linfusion_attn.h``.

Argument marshalling only: every step of the attention runs in the CUDA library.  There is no
CPU fallback; loading fails loudly when ``liblinfusion_attn.so`` has not been built
(``python -m paper_2409_02097_b200.build``).  PyTorch is used for device memory and streams.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_PKG = os.path.dirname(os.path.abspath(__file__))
# LINFUSION_ATTN_LIB selects another build of the same library (the bounds-checked debugging build)
LIB_PATH = os.environ.get("LINFUSION_ATTN_LIB") or os.path.join(_PKG, "liblinfusion_attn.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALLOC, ERR_CUDA, ERR_TIMEOUT = range(6)
PHI_ELU_PLUS_ONE, PHI_IDENTITY = 0, 1
VARIANT_AUTO, VARIANT_SPLIT, VARIANT_STREAM, VARIANT_CLUSTER, VARIANT_FUSED = 0, 1, 2, 3, 4
VARIANTS = {"auto": VARIANT_AUTO, "split": VARIANT_SPLIT, "stream": VARIANT_STREAM,
            "cluster": VARIANT_CLUSTER, "fused": VARIANT_FUSED}

EXPORTED = [
    "linfusion_attn_create", "linfusion_attn_forward", "linfusion_attn_forward_host",
    "linfusion_attn_destroy", "linfusion_status_string", "linfusion_attn_workspace_bytes",
    "linfusion_attn_set_workspace", "linfusion_attn_status", "linfusion_attn_read_state",
    "linfusion_attn_variant_name", "linfusion_attn_launches_per_forward",
    "linfusion_attn_enable_kernel_timing", "linfusion_attn_kernel_times",
    "linfusion_attn_set_kernel_timing_stride",
    "linfusion_attn_forward_noalloc", "linfusion_attn_noalloc_layout",
    "linfusion_attn_state", "linfusion_attn_apply", "linfusion_attn_state_buffer",
    "linfusion_attn_apply_peers", "linfusion_attn_selftest_wait", "linfusion_attn_selftest_counter_wait",
    "linfusion_attn_state_x", "linfusion_attn_apply_x", "linfusion_attn_branch_x", "linfusion_attn_forward_x",
    "linfusion_attn_checked_build", "linfusion_attn_checked_violations", "linfusion_attn_checked_shrink_y",
]


class Desc(ctypes.Structure):
    """Mirror of ``linfusion_attn_desc_t``."""
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("N", ctypes.c_int32),
                ("d", ctypes.c_int32), ("phi", ctypes.c_int32), ("eps", ctypes.c_float),
                ("device", ctypes.c_int32), ("flags", ctypes.c_uint32), ("d_qk", ctypes.c_int32)]


class MlpWeights(ctypes.Structure):
    """Mirror of ``linfusion_mlp_weights_t``."""
    _fields_ = [("w_lin", ctypes.c_void_p), ("w_1", ctypes.c_void_p), ("b_1", ctypes.c_void_p),
                ("gamma", ctypes.c_void_p), ("beta", ctypes.c_void_p)]


class ModuleWeights(ctypes.Structure):
    """Mirror of ``linfusion_module_weights_t``."""
    _fields_ = [("q", MlpWeights), ("k", MlpWeights), ("w_v", ctypes.c_void_p),
                ("ln_eps", ctypes.c_float), ("leaky_slope", ctypes.c_float)]


class LinFusionError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {status_string(code)} (status {code})")


_lib = None


def load_library() -> ctypes.CDLL:
    """Load the CUDA library; raises if it is missing (there is no other implementation)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} not found: build it with `python -m paper_2409_02097_b200.build` "
            "(nvcc, sm_100a).  This package has no CPU or PyTorch fallback.")
    lib = ctypes.CDLL(LIB_PATH)
    vp, st = ctypes.c_void_p, ctypes.c_int
    lib.linfusion_attn_create.restype = st
    lib.linfusion_attn_create.argtypes = [ctypes.POINTER(Desc), ctypes.POINTER(vp)]
    lib.linfusion_attn_forward.restype = st
    lib.linfusion_attn_forward.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.linfusion_attn_forward_host.restype = st
    lib.linfusion_attn_forward_host.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.linfusion_attn_destroy.restype = st
    lib.linfusion_attn_destroy.argtypes = [vp]
    lib.linfusion_status_string.restype = ctypes.c_char_p
    lib.linfusion_status_string.argtypes = [st]
    lib.linfusion_attn_plan.restype = st
    lib.linfusion_attn_plan.argtypes = [ctypes.POINTER(Desc), ctypes.c_int, ctypes.POINTER(ctypes.c_int32),
                                        ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
    lib.linfusion_attn_workspace_bytes.restype = st
    lib.linfusion_attn_workspace_bytes.argtypes = [ctypes.POINTER(Desc), ctypes.c_int,
                                                   ctypes.POINTER(ctypes.c_size_t)]
    lib.linfusion_attn_set_workspace.restype = st
    lib.linfusion_attn_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
    lib.linfusion_attn_status.restype = st
    lib.linfusion_attn_status.argtypes = [vp]
    lib.linfusion_attn_read_state.restype = st
    lib.linfusion_attn_read_state.argtypes = [vp, vp, vp]
    lib.linfusion_attn_variant_name.restype = ctypes.c_char_p
    lib.linfusion_attn_variant_name.argtypes = [vp]
    lib.linfusion_attn_launches_per_forward.restype = ctypes.c_int32
    lib.linfusion_attn_launches_per_forward.argtypes = [vp]
    lib.linfusion_attn_enable_kernel_timing.restype = st
    lib.linfusion_attn_enable_kernel_timing.argtypes = [vp, ctypes.c_int32]
    lib.linfusion_attn_set_kernel_timing_stride.restype = st
    lib.linfusion_attn_set_kernel_timing_stride.argtypes = [vp, ctypes.c_int32]
    lib.linfusion_attn_kernel_times.restype = st
    lib.linfusion_attn_kernel_times.argtypes = [vp, ctypes.POINTER(ctypes.c_float),
                                                ctypes.POINTER(ctypes.c_int32)]
    lib.linfusion_attn_forward_noalloc.restype = st
    lib.linfusion_attn_forward_noalloc.argtypes = [ctypes.POINTER(Desc), vp, vp, vp, vp, vp]
    lib.linfusion_attn_noalloc_layout.restype = st
    lib.linfusion_attn_noalloc_layout.argtypes = [ctypes.POINTER(Desc), ctypes.c_int,
                                                  ctypes.POINTER(ctypes.c_int32)] + \
                                                 [ctypes.POINTER(ctypes.c_size_t)] * 3
    lib.linfusion_attn_state.restype = st
    lib.linfusion_attn_state.argtypes = [vp, vp, vp, vp]
    lib.linfusion_attn_apply.restype = st
    lib.linfusion_attn_apply.argtypes = [vp, vp, vp, vp]
    lib.linfusion_attn_selftest_wait.restype = st
    lib.linfusion_attn_selftest_wait.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    lib.linfusion_attn_selftest_counter_wait.restype = st
    lib.linfusion_attn_selftest_counter_wait.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    lib.linfusion_attn_apply_peers.restype = st
    lib.linfusion_attn_apply_peers.argtypes = [vp, vp, vp, ctypes.POINTER(ctypes.c_void_p), ctypes.c_int32, vp]
    lib.linfusion_attn_state_buffer.restype = st
    lib.linfusion_attn_state_buffer.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(ctypes.c_size_t)]
    lib.linfusion_attn_state_x.restype = st
    lib.linfusion_attn_state_x.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.linfusion_attn_apply_x.restype = st
    lib.linfusion_attn_apply_x.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.linfusion_attn_branch_x.restype = st
    lib.linfusion_attn_branch_x.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_float, ctypes.c_float, vp, vp]
    lib.linfusion_attn_forward_x.restype = st
    lib.linfusion_attn_forward_x.argtypes = [vp, vp, ctypes.POINTER(ModuleWeights), vp, vp]
    lib.linfusion_attn_checked_build.restype = ctypes.c_int32
    lib.linfusion_attn_checked_build.argtypes = []
    lib.linfusion_attn_checked_violations.restype = st
    lib.linfusion_attn_checked_violations.argtypes = [ctypes.c_int32, ctypes.POINTER(ctypes.c_uint32), ctypes.c_int32]
    lib.linfusion_attn_checked_shrink_y.restype = st
    lib.linfusion_attn_checked_shrink_y.argtypes = [ctypes.c_size_t]
    _lib = lib
    return lib


def checked_build() -> bool:
    """True when the loaded library is the bounds-checked debugging build."""
    return bool(load_library().linfusion_attn_checked_build())


def checked_shrink_y(nbytes: int) -> None:
    """Self-test of the checked build: register Y ``nbytes`` short, so that its last rows count as out of range."""
    rc = load_library().linfusion_attn_checked_shrink_y(int(nbytes))
    if rc != OK:
        raise LinFusionError(rc, "linfusion_attn_checked_shrink_y")


def checked_violations(device: int = 0, reset: bool = True) -> int:
    """Global-memory accesses the checked build found outside the buffers of their call (and skipped)."""
    n = ctypes.c_uint32(0)
    rc = load_library().linfusion_attn_checked_violations(int(device), ctypes.byref(n), 1 if reset else 0)
    if rc != OK:
        raise LinFusionError(rc, "linfusion_attn_checked_violations")
    return int(n.value)


def status_string(code: int) -> str:
    return load_library().linfusion_status_string(int(code)).decode()


LAYOUT_TOKEN_MAJOR = 0x10   # tensors are [B, N, H, d] instead of [B, H, N, d]
FLAG_UNNORMALIZED = 0x20    # Y_i = phi(Q_i) S, without the division by phi(Q_i) . z + eps
DTYPE_FP16 = 0x40           # Q, K, V, Y are fp16 instead of bf16


def make_desc(B, H, N, d, phi=PHI_ELU_PLUS_ONE, eps=1e-6, device=0, variant="auto",
              layout="head_major", normalize=True, dtype="bf16", d_qk=0) -> Desc:
    """``d`` is the width of V and Y; ``d_qk`` the feature width d' of Q and K when it differs
    (Prop. 3), 0 meaning the same."""
    flags = VARIANTS[variant] if isinstance(variant, str) else int(variant)
    if not normalize:
        flags |= FLAG_UNNORMALIZED
    if dtype == "fp16":
        flags |= DTYPE_FP16
    elif dtype != "bf16":
        raise ValueError("dtype must be 'bf16' or 'fp16'")
    if layout == "token_major":
        flags |= LAYOUT_TOKEN_MAJOR
    elif layout != "head_major":
        raise ValueError("layout must be 'head_major' or 'token_major'")
    return Desc(int(B), int(H), int(N), int(d), int(phi), float(eps), int(device), flags, int(d_qk))


def linfusion_attn_workspace_bytes(desc: Desc, sm_count: int = 0) -> int:
    out = ctypes.c_size_t(0)
    rc = load_library().linfusion_attn_workspace_bytes(ctypes.byref(desc), int(sm_count),
                                                       ctypes.byref(out))
    if rc != OK:
        raise LinFusionError(rc, "linfusion_attn_workspace_bytes")
    return int(out.value)


def linfusion_attn_plan(desc: Desc, sm_count: int = 0):
    """(variant name, launches per forward, CTAs of the largest one-dimensional grid) for ``desc``, no GPU needed."""
    variant, launches, ctas = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_int32(0)
    rc = load_library().linfusion_attn_plan(ctypes.byref(desc), int(sm_count), ctypes.byref(variant),
                                            ctypes.byref(launches), ctypes.byref(ctas))
    if rc != OK:
        raise LinFusionError(rc, "linfusion_attn_plan")
    names = {v: k for k, v in VARIANTS.items()}
    return names[variant.value], int(launches.value), int(ctas.value)


def linfusion_attn_create(desc: Desc) -> ctypes.c_void_p:
    handle = ctypes.c_void_p()
    rc = load_library().linfusion_attn_create(ctypes.byref(desc), ctypes.byref(handle))
    if rc != OK:
        raise LinFusionError(rc, "linfusion_attn_create")
    return handle


def linfusion_attn_forward(handle, q_ptr: int, k_ptr: int, v_ptr: int, y_ptr: int,
                           stream_ptr: int = 0) -> None:
    rc = load_library().linfusion_attn_forward(handle, q_ptr, k_ptr, v_ptr, y_ptr, stream_ptr)
    if rc != OK:
        raise LinFusionError(rc, "linfusion_attn_forward")


def linfusion_attn_forward_host(handle, q_ptr: int, k_ptr: int, v_ptr: int, y_ptr: int,
                                stream_ptr: int = 0) -> None:
    rc = load_library().linfusion_attn_forward_host(handle, q_ptr, k_ptr, v_ptr, y_ptr, stream_ptr)
    if rc != OK:
        raise LinFusionError(rc, "linfusion_attn_forward_host")


def linfusion_attn_forward_noalloc(desc: Desc, q_ptr: int, k_ptr: int, v_ptr: int, y_ptr: int,
                                   stream_ptr: int = 0) -> None:
    """Handle-free forward that allocates nothing: the split-N scratch is a fixed 16 MiB array
    inside the library's device image.  For hosts that cannot let a library call cudaMalloc.
    Calls that overlap on the GPU race on that array; problems whose state does not fit raise
    ``LinFusionError`` with ``ERR_ALLOC``."""
    rc = load_library().linfusion_attn_forward_noalloc(ctypes.byref(desc), q_ptr, k_ptr, v_ptr,
                                                       y_ptr, stream_ptr)
    if rc != OK:
        raise LinFusionError(rc, "linfusion_attn_forward_noalloc")


def linfusion_attn_noalloc_layout(desc: Desc, sm_count: int = 0):
    """(chunks, state_offset, bytes_used, capacity) of a problem in the allocation-free entry
    point's fixed array; raises ``LinFusionError`` (``ERR_ALLOC``) when it does not fit."""
    chunks = ctypes.c_int32(0)
    off, used, cap = ctypes.c_size_t(0), ctypes.c_size_t(0), ctypes.c_size_t(0)
    rc = load_library().linfusion_attn_noalloc_layout(ctypes.byref(desc), int(sm_count), ctypes.byref(chunks),
                                                      ctypes.byref(off), ctypes.byref(used), ctypes.byref(cap))
    if rc != OK:
        raise LinFusionError(rc, "linfusion_attn_noalloc_layout")
    return int(chunks.value), int(off.value), int(used.value), int(cap.value)


def linfusion_attn_destroy(handle) -> None:
    rc = load_library().linfusion_attn_destroy(handle)
    if rc != OK:
        raise LinFusionError(rc, "linfusion_attn_destroy")


class LinFusionAttention:
    """One handle per shape.  ``forward`` takes bf16 CUDA tensors [B, H, N, d] (or [B, N, H, d]
    with ``layout="token_major"``).  With ``d_qk`` (Prop. 3's feature width d') Q and K are
    [.., d_qk] while V and Y stay [.., d]."""

    def __init__(self, B, H, N, d, phi=PHI_ELU_PLUS_ONE, eps=1e-6, device=0, variant="auto",
                 layout="head_major", normalize=True, dtype="bf16", d_qk=0):
        self.desc = make_desc(B, H, N, d, phi, eps, device, variant, layout, normalize, dtype, d_qk)
        self.dtype = dtype
        dk = int(d_qk) if d_qk else int(d)
        self.dk = dk
        # V and Y are [B, H, N, d], or [B, N, H, d] in the token-major layout; Q and K have d' channels
        self.shape = (int(B), int(H), int(N), int(d)) if layout == "head_major" else \
                     (int(B), int(N), int(H), int(d))
        self.shape_qk = self.shape[:3] + (dk,)
        self._lib = load_library()
        self._h = linfusion_attn_create(self.desc)
        self._lent_ws = None

    # -- properties -------------------------------------------------------------------------
    @property
    def variant(self) -> str:
        return self._lib.linfusion_attn_variant_name(self._h).decode()

    @property
    def launches_per_forward(self) -> int:
        return int(self._lib.linfusion_attn_launches_per_forward(self._h))

    # -- calls ------------------------------------------------------------------------------
    def _check(self, t, name):
        import torch
        want = torch.float16 if self.dtype == "fp16" else torch.bfloat16
        shape = self.shape_qk if name in ("q", "k") else self.shape
        if tuple(t.shape) != shape or t.dtype != want or not t.is_contiguous():
            raise ValueError(f"{name}: expected contiguous {self.dtype} tensor of shape {shape}")

    def _new_y(self, like):
        import torch
        return torch.empty(self.shape, dtype=like.dtype, device=like.device)

    def forward(self, q, k, v, y=None, stream: Optional[int] = None):
        import torch
        for t, n in ((q, "q"), (k, "k"), (v, "v")):
            self._check(t, n)
            if not t.is_cuda:
                raise ValueError(f"{n}: expected a CUDA tensor")
        if y is None:
            y = self._new_y(q)
        else:
            self._check(y, "y")
        if stream is None:
            stream = torch.cuda.current_stream(q.device).cuda_stream
        linfusion_attn_forward(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), y.data_ptr(),
                               stream)
        return y

    def forward_host(self, q, k, v, y, stream: Optional[int] = None):
        """q, k, v, y: CPU (ideally pinned) bf16 tensors; y is valid after a stream sync."""
        import torch
        for t, n in ((q, "q"), (k, "k"), (v, "v"), (y, "y")):
            self._check(t, n)
            if t.is_cuda:
                raise ValueError(f"{n}: expected a host tensor")
        if stream is None:
            stream = torch.cuda.current_stream(self.desc.device).cuda_stream
        linfusion_attn_forward_host(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                    y.data_ptr(), stream)
        return y

    def status(self) -> int:
        return int(self._lib.linfusion_attn_status(self._h))

    def read_state(self):
        """(S [B,H,d',d], z [B,H,d']) of the last forward as fp32 numpy arrays."""
        import numpy as np
        B, H, d = self.desc.B, self.desc.H, self.desc.d
        S = np.empty((B, H, self.dk, d), dtype=np.float32)
        z = np.empty((B, H, self.dk), dtype=np.float32)
        rc = self._lib.linfusion_attn_read_state(self._h, S.ctypes.data, z.ctypes.data)
        if rc != OK:
            raise LinFusionError(rc, "linfusion_attn_read_state")
        return S, z

    # -- token-sharded use (Sec. 4.3): state of the local K/V, caller's sum, apply to the local Q --
    def state(self, k, v, stream: Optional[int] = None) -> None:
        import torch
        for t, n in ((k, "k"), (v, "v")):
            self._check(t, n)
        if stream is None:
            stream = torch.cuda.current_stream(k.device).cuda_stream
        rc = self._lib.linfusion_attn_state(self._h, k.data_ptr(), v.data_ptr(), stream)
        if rc != OK:
            raise LinFusionError(rc, "linfusion_attn_state")

    # -- fed from the layer input X [B, N, C] and the projection weights [C, C] (x @ w) ------------
    def _check_x(self, x, weights, extras=()):
        import torch
        want = torch.float16 if self.dtype == "fp16" else torch.bfloat16
        B, H, N, d = self.desc.B, self.desc.H, self.desc.N, self.desc.d
        C = H * d
        for t, n, shape in [(x, "x", (B, N, C))] + [(w, "weight", (C, C)) for w in weights] + \
                           [(t, "branch output", (B, N, C)) for t in extras if t is not None]:
            if tuple(t.shape) != shape or t.dtype != want or not t.is_contiguous() or not t.is_cuda:
                raise ValueError(f"{n}: expected contiguous CUDA {self.dtype} tensor of shape {shape}")

    def state_x(self, x, w_k, w_v, t_k=None, stream: Optional[int] = None) -> None:
        """S | z from the layer input: K = x @ w_k (+ t_k), V = x @ w_v computed inside the kernel."""
        import torch
        self._check_x(x, (w_k, w_v), (t_k,))
        if stream is None:
            stream = torch.cuda.current_stream(x.device).cuda_stream
        rc = self._lib.linfusion_attn_state_x(self._h, x.data_ptr(), w_k.data_ptr(), w_v.data_ptr(),
                                              t_k.data_ptr() if t_k is not None else None, stream)
        if rc != OK:
            raise LinFusionError(rc, "linfusion_attn_state_x")

    def branch_x(self, x, w_1, b_1, gamma, beta, ln_eps=1e-5, slope=0.01, t_out=None, stream: Optional[int] = None):
        """T = LeakyReLU(LayerNorm(x @ w_1 + b_1; gamma, beta)) [B, N, C]: one non-linear branch of f' / g'."""
        import torch
        self._check_x(x, (w_1,), (t_out,))
        if t_out is None:
            t_out = torch.empty_like(x)
        if stream is None:
            stream = torch.cuda.current_stream(x.device).cuda_stream
        rc = self._lib.linfusion_attn_branch_x(self._h, x.data_ptr(), w_1.data_ptr(),
                                               b_1.data_ptr() if b_1 is not None else None, gamma.data_ptr(),
                                               beta.data_ptr(), float(ln_eps), float(slope), t_out.data_ptr(), stream)
        if rc != OK:
            raise LinFusionError(rc, "linfusion_attn_branch_x")
        return t_out

    def forward_x(self, x, weights: dict, ln_eps=1e-5, slope=0.01, y=None, stream: Optional[int] = None):
        """The module from the layer input.  ``weights``: q_lin, k_lin, v ([C, C]) and, for each
        non-linear branch that is present, q_w1 / q_b1 / q_gamma / q_beta (and k_...)."""
        import torch
        self._check_x(x, (weights["q_lin"], weights["k_lin"], weights["v"]), (y,))
        if y is None:
            y = torch.empty_like(x)
        if stream is None:
            stream = torch.cuda.current_stream(x.device).cuda_stream
        ptr = lambda name: weights[name].data_ptr() if weights.get(name) is not None else None
        mw = ModuleWeights()
        for side, name in ((mw.q, "q"), (mw.k, "k")):
            side.w_lin, side.w_1, side.b_1 = ptr(name + "_lin"), ptr(name + "_w1"), ptr(name + "_b1")
            side.gamma, side.beta = ptr(name + "_gamma"), ptr(name + "_beta")
        mw.w_v, mw.ln_eps, mw.leaky_slope = ptr("v"), float(ln_eps), float(slope)
        self._weights_alive = weights
        rc = self._lib.linfusion_attn_forward_x(self._h, x.data_ptr(), ctypes.byref(mw), y.data_ptr(), stream)
        if rc != OK:
            raise LinFusionError(rc, "linfusion_attn_forward_x")
        return y

    def apply_x(self, x, w_q, t_q=None, y=None, stream: Optional[int] = None):
        """Y [B, N, C] from the layer input and the current state: Q = x @ w_q (+ t_q) inside the kernel."""
        import torch
        self._check_x(x, (w_q,), (t_q, y))
        if y is None:
            y = torch.empty_like(x)
        if stream is None:
            stream = torch.cuda.current_stream(x.device).cuda_stream
        rc = self._lib.linfusion_attn_apply_x(self._h, x.data_ptr(), w_q.data_ptr(),
                                              t_q.data_ptr() if t_q is not None else None, y.data_ptr(), stream)
        if rc != OK:
            raise LinFusionError(rc, "linfusion_attn_apply_x")
        return y

    def apply(self, q, y=None, stream: Optional[int] = None):
        import torch
        self._check(q, "q")
        if y is None:
            y = self._new_y(q)
        else:
            self._check(y, "y")
        if stream is None:
            stream = torch.cuda.current_stream(q.device).cuda_stream
        rc = self._lib.linfusion_attn_apply(self._h, q.data_ptr(), y.data_ptr(), stream)
        if rc != OK:
            raise LinFusionError(rc, "linfusion_attn_apply")
        return y

    def apply_peers(self, q, peer_state_ptrs, y=None, stream: Optional[int] = None):
        """Apply with the sum over devices done by the library: ``peer_state_ptrs`` lists the
        device addresses of every rank's state buffer (``state_buffer()[0]``, this rank's own
        included), readable from this device, in the same order on every rank."""
        import torch
        self._check(q, "q")
        if y is None:
            y = self._new_y(q)
        else:
            self._check(y, "y")
        if stream is None:
            stream = torch.cuda.current_stream(q.device).cuda_stream
        ptrs = (ctypes.c_void_p * len(peer_state_ptrs))(*[int(p) for p in peer_state_ptrs])
        rc = self._lib.linfusion_attn_apply_peers(self._h, q.data_ptr(), y.data_ptr(), ptrs,
                                                  len(peer_state_ptrs), stream)
        if rc != OK:
            raise LinFusionError(rc, "linfusion_attn_apply_peers")
        return y

    def state_buffer(self):
        """(device address, number of floats) of the fp32 S | z buffer: [B*H][d*d + d]."""
        ptr = ctypes.c_void_p()
        n = ctypes.c_size_t(0)
        rc = self._lib.linfusion_attn_state_buffer(self._h, ctypes.byref(ptr), ctypes.byref(n))
        if rc != OK:
            raise LinFusionError(rc, "linfusion_attn_state_buffer")
        return int(ptr.value or 0), int(n.value)

    def enable_kernel_timing(self, slots: int) -> None:
        rc = self._lib.linfusion_attn_enable_kernel_timing(self._h, int(slots))
        if rc != OK:
            raise LinFusionError(rc, "linfusion_attn_enable_kernel_timing")

    def selftest_wait(self):
        """(status code, milliseconds) of the bounded-wait self-test; ERR_TIMEOUT is the expected code."""
        ms = ctypes.c_float(0.0)
        rc = self._lib.linfusion_attn_selftest_wait(self._h, ctypes.byref(ms))
        return int(rc), float(ms.value)

    def selftest_counter_wait(self):
        """The same for the bounded poll of a global counter (the single-launch variant's wait)."""
        ms = ctypes.c_float(0.0)
        rc = self._lib.linfusion_attn_selftest_counter_wait(self._h, ctypes.byref(ms))
        return int(rc), float(ms.value)

    def set_kernel_timing_stride(self, stride: int) -> None:
        rc = self._lib.linfusion_attn_set_kernel_timing_stride(self._h, int(stride))
        if rc != OK:
            raise LinFusionError(rc, "linfusion_attn_set_kernel_timing_stride")

    def kernel_times(self):
        """([ms_state, ms_reduce, ms_apply] summed, calls) since the last call of this method."""
        ms = (ctypes.c_float * 3)()
        calls = ctypes.c_int32(0)
        rc = self._lib.linfusion_attn_kernel_times(self._h, ms, ctypes.byref(calls))
        if rc != OK:
            raise LinFusionError(rc, "linfusion_attn_kernel_times")
        return [float(x) for x in ms], int(calls.value)

    def set_workspace(self, tensor) -> None:
        rc = self._lib.linfusion_attn_set_workspace(self._h, tensor.data_ptr(),
                                                    tensor.numel() * tensor.element_size())
        if rc != OK:
            raise LinFusionError(rc, "linfusion_attn_set_workspace")
        self._lent_ws = tensor

    def close(self) -> None:
        if self._h is not None and self._h.value:
            linfusion_attn_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
