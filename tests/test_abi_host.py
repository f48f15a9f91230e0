"""Host-side checks of the C ABI that need no GPU: the library loads, exports every declared
symbol, and rejects bad descriptors before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2409_02097_b200 import attn, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return attn.load_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "linfusion_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(linfusion_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert "linfusion_attn_create" in names and "linfusion_attn_forward" in names
    assert "linfusion_attn_destroy" in names
    for name in names:
        assert hasattr(lib, name), f"{name} declared in the header but not exported"
    assert set(attn.EXPORTED) <= set(names)


def test_status_strings(lib):
    seen = set()
    for code in range(6):
        s = attn.status_string(code)
        assert s and s not in seen
        seen.add(s)
    assert attn.status_string(0) == "ok"
    assert "unknown" in attn.status_string(99)


def _ws(desc, sm=148):
    return attn.linfusion_attn_workspace_bytes(desc, sm)


def test_workspace_bytes_is_pure_host_and_monotone():
    small = _ws(attn.make_desc(2, 8, 4096, 40, variant="split"))
    assert small > 2 * 8 * 40 * 41 * 4
    # split: partials scale with the chunk count, never with N beyond the tile count
    a = _ws(attn.make_desc(2, 10, 524288, 64, variant="split"))
    b = _ws(attn.make_desc(2, 10, 2 * 524288, 64, variant="split"))
    assert a == b
    # stream: G * spans partials (one CTA per SM) + state + bf16 operand image + tile counters + status word
    s = _ws(attn.make_desc(2, 10, 524288, 64, variant="stream"))
    assert s == 148 * 2 * 4160 * 4 + 20 * 4160 * 4 + 20 * 80 * 128 + 256 + 256
    # cluster: no partials in global memory
    c = _ws(attn.make_desc(2, 8, 256, 160, variant="cluster"))
    assert c == (16 * 160 * 161 * 4 + 255) // 256 * 256 + 256
    # the single tcgen05 launch at widths 40 / 80 / 160: per_slab partials of [roundup16(d)][roundup16(d + 1)] floats
    # per slab (8 CTAs per slab at N = 4096 x 16 slabs, d = 40), state, two words per slab + control, status
    f = _ws(attn.make_desc(2, 8, 4096, 40, variant="fused"))
    assert f == (16 * 8 * 48 * 48 * 4 + 255) // 256 * 256 + (16 * 40 * 41 * 4 + 255) // 256 * 256 + 256 + 256 + 256
    # one CTA per slab (d = 160: a partial is 110 KB, so slabs are not shared): no partials at all
    assert _ws(attn.make_desc(2, 8, 256, 160, variant="fused")) == \
        (16 * 160 * 161 * 4 + 255) // 256 * 256 + 256 + 256 + 256
    # long runs with large partials: 8 CTAs per slab share the summing; partials, state, the 16-bit operand per
    # slab (3 atoms x 160 rows x 128 bytes), counters + control, status
    assert _ws(attn.make_desc(2, 8, 1024, 160, variant="fused")) == \
        (16 * 8 * 160 * 176 * 4 + 255) // 256 * 256 + (16 * 160 * 161 * 4 + 255) // 256 * 256 + \
        (16 * 3 * 160 * 128 + 255) // 256 * 256 + 256 + 256 + 256
    # more slabs than SMs: whole slabs per CTA, no partials either
    assert _ws(attn.make_desc(2, 100, 256, 40, variant="fused")) == \
        (200 * 40 * 41 * 4 + 255) // 256 * 256 + (200 * 8 + 255) // 256 * 256 + 256 + 256
    # the plan depends on the SM count it is given
    assert _ws(attn.make_desc(2, 10, 524288, 64, variant="stream"), 74) < s


@pytest.mark.parametrize("kw", [
    dict(B=0), dict(H=0), dict(N=0), dict(N=-5), dict(eps=-1.0), dict(eps=float("nan")),
    dict(eps=float("inf")), dict(device=-1),
])
def test_invalid_descriptors(kw):
    args = dict(B=2, H=8, N=4096, d=40, eps=1e-6, device=0)
    args.update(kw)
    desc = attn.make_desc(**args)
    with pytest.raises(attn.LinFusionError) as e:
        _ws(desc)
    assert e.value.code == attn.ERR_INVALID_ARG
    with pytest.raises(attn.LinFusionError) as e:
        attn.linfusion_attn_create(desc)
    assert e.value.code == attn.ERR_INVALID_ARG


@pytest.mark.parametrize("kw", [
    dict(d=40, variant="fused", H=80, N=128 * 513),        # more slabs than SMs and more than 512 tiles per slab
    dict(d=160, variant="fused", B=74, H=2, N=128 * 513),  # one CTA per slab, more than 512 tiles each
])
def test_shapes_the_single_launch_at_padded_widths_cannot_take(kw):
    args = dict(B=2, H=8, N=4096, d=64, eps=1e-6, device=0)
    args.update(kw)
    with pytest.raises(attn.LinFusionError) as e:
        _ws(attn.make_desc(**args))
    assert e.value.code == attn.ERR_UNSUPPORTED
    args["variant"] = "auto"                              # AUTO plans something else
    assert _ws(attn.make_desc(**args)) > 0


@pytest.mark.parametrize("kw", [
    dict(d=48), dict(d=7), dict(d=256), dict(phi=7), dict(variant=9), dict(variant=0x80),
    dict(d=40, variant="stream"), dict(d=128, variant="fused"), dict(d=32, variant="fused"),
])
def test_unsupported_descriptors(kw):
    args = dict(B=2, H=8, N=4096, d=64, eps=1e-6, device=0)
    args.update(kw)
    desc = attn.make_desc(**args)
    with pytest.raises(attn.LinFusionError) as e:
        _ws(desc)
    assert e.value.code == attn.ERR_UNSUPPORTED
    with pytest.raises(attn.LinFusionError) as e:
        attn.linfusion_attn_create(desc)
    assert e.value.code == attn.ERR_UNSUPPORTED


def test_null_arguments(lib):
    assert lib.linfusion_attn_create(None, None) == attn.ERR_INVALID_ARG
    out = ctypes.c_void_p()
    assert lib.linfusion_attn_create(None, ctypes.byref(out)) == attn.ERR_INVALID_ARG
    assert not out.value
    assert lib.linfusion_attn_forward(None, 16, 16, 16, 16, None) == attn.ERR_INVALID_ARG
    assert lib.linfusion_attn_forward_host(None, 16, 16, 16, 16, None) == attn.ERR_INVALID_ARG
    assert lib.linfusion_attn_destroy(None) == attn.OK
    assert lib.linfusion_attn_status(None) == attn.ERR_INVALID_ARG
    assert lib.linfusion_attn_read_state(None, None, None) == attn.ERR_INVALID_ARG
    assert lib.linfusion_attn_set_workspace(None, None, 0) == attn.ERR_INVALID_ARG
    assert lib.linfusion_attn_workspace_bytes(None, 0, None) == attn.ERR_INVALID_ARG
    assert lib.linfusion_attn_launches_per_forward(None) == 0
    assert lib.linfusion_attn_variant_name(None) == b""


def test_create_without_a_device_fails_cleanly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(attn.LinFusionError) as e:
        attn.linfusion_attn_create(attn.make_desc(2, 8, 4096, 40))
    assert e.value.code in (attn.ERR_CUDA, attn.ERR_INVALID_ARG)


def test_binding_has_no_fallback(monkeypatch):
    monkeypatch.setattr(attn, "_lib", None)
    monkeypatch.setattr(attn, "LIB_PATH", os.path.join(ROOT, "does_not_exist.so"))
    with pytest.raises(ImportError):
        attn.load_library()


def test_noalloc_layout_never_leaves_the_array():
    """Host arithmetic of the allocation-free entry point: over a sweep of descriptors and SM
    counts the partial states and the reduced state stay inside the fixed array, the state starts
    on a 256-byte boundary behind the last partial, and what cannot fit is refused."""
    fits = refused = clamped = 0
    for d in (32, 40, 64, 80, 128, 160):
        for slabs in (1, 2, 7, 16, 40, 64, 81, 82, 200, 1000, 4000, 65535):
            for N in (1, 63, 64, 65, 4096, 524288):
                for sm in (0, 1, 74, 148, 400):
                    desc = attn.make_desc(1, slabs, N, d)
                    per_chunk = slabs * d * (d + 1) * 4
                    try:
                        chunks, off, used, cap = attn.linfusion_attn_noalloc_layout(desc, sm)
                    except attn.LinFusionError as e:
                        assert e.code == attn.ERR_ALLOC
                        assert 2 * per_chunk + 256 > (16 << 20) - 256, (d, slabs)
                        refused += 1
                        continue
                    fits += 1
                    assert cap == 16 << 20
                    assert 1 <= chunks <= max(1, -(-N // 64))
                    assert off % 256 == 0 and off >= chunks * per_chunk
                    assert used == off + per_chunk and used <= cap
                    planned = min(max(1, -(-2 * (sm or 148) // slabs)), -(-N // 64))
                    clamped += chunks < planned
    assert fits > 500 and refused > 50 and clamped > 20
    with pytest.raises(attn.LinFusionError) as e:
        attn.linfusion_attn_noalloc_layout(attn.make_desc(1, 4, 64, 64, variant="cluster"))
    assert e.value.code == attn.ERR_UNSUPPORTED
    with pytest.raises(attn.LinFusionError) as e:
        attn.linfusion_attn_noalloc_layout(attn.make_desc(1, 70000, 64, 64))
    assert e.value.code == attn.ERR_UNSUPPORTED


def test_two_widths_in_the_descriptor():
    """Prop. 3: d_qk = d' is the width of Q and K, d that of V and Y; the state is d' x d."""
    # state floats follow d' * (d + 1): the cluster variant's workspace is state + status only
    sq = _ws(attn.make_desc(2, 4, 256, 64, variant="cluster"))
    wide = _ws(attn.make_desc(2, 4, 256, 64, variant="cluster", d_qk=128))
    narrow = _ws(attn.make_desc(2, 4, 256, 64, variant="cluster", d_qk=32))
    assert wide - sq == 8 * (128 - 64) * 65 * 4 and sq - narrow == 8 * (64 - 32) * 65 * 4
    assert _ws(attn.make_desc(2, 4, 256, 64, variant="split", d_qk=64)) == \
        _ws(attn.make_desc(2, 4, 256, 64, variant="split"))
    for kw in (dict(d=64, d_qk=48), dict(d=40, d_qk=128), dict(d=64, d_qk=128, variant="stream"),
               dict(d=64, d_qk=128, variant="fused")):
        with pytest.raises(attn.LinFusionError) as e:
            _ws(attn.make_desc(1, 1, 256, kw["d"], d_qk=kw["d_qk"], variant=kw.get("variant", "auto")))
        assert e.value.code == attn.ERR_UNSUPPORTED
    with pytest.raises(attn.LinFusionError) as e:
        _ws(attn.make_desc(1, 1, 256, 64, d_qk=-8))
    assert e.value.code == attn.ERR_INVALID_ARG
    # the allocation-free entry point sizes its array use by d' * (d + 1) too
    chunks, off, used, cap = attn.linfusion_attn_noalloc_layout(attn.make_desc(2, 8, 4096, 64, d_qk=128), 148)
    assert used - off == 16 * 128 * 65 * 4 and used <= cap and chunks >= 1


# (B, H, N, d) -> what AUTO resolves to on a 148-SM device (the crossovers measured on B200; the GPU tests check
# the same table against handles created on the device)
AUTO_POLICY = [
    ((2, 10, 524288, 64), "stream", 2), ((2, 20, 131072, 64), "stream", 2),
    ((2, 10, 16384, 64), "stream", 2), ((2, 20, 4096, 64), "stream", 2), ((2, 20, 2304, 64), "stream", 2),
    ((2, 10, 9216, 64), "stream", 2), ((1, 10, 2304, 64), "split", 3), ((2, 20, 144, 64), "cluster", 1),
    ((2, 20, 576, 64), "fused", 1), ((2, 2, 144, 64), "cluster", 1),
    ((2, 8, 4096, 40), "fused", 1), ((2, 8, 1024, 80), "fused", 1), ((2, 8, 256, 160), "fused", 1),
    ((2, 8, 64, 160), "fused", 1), ((2, 100, 256, 160), "fused", 1), ((2, 100, 8192, 160), "fused", 1),
    ((2, 100, 131072, 160), "split", 3), ((2, 8, 1000, 160), "fused", 1), ((1, 1, 100000, 160), "fused", 1),
    ((2, 8, 16384, 160), "fused", 1), ((32, 8, 4096, 40), "fused", 1), ((2, 8, 4096, 128), "split", 3),
    ((2, 8, 64, 128), "cluster", 1), ((300, 1, 4096, 64), "stream", 3),
]


def test_auto_policy_without_a_device():
    for dims, want, launches in AUTO_POLICY:
        variant, n, ctas = attn.linfusion_attn_plan(attn.make_desc(*dims), 148)
        assert (variant, n) == (want, launches), (dims, variant, n)
        assert 0 <= ctas <= 148
    # the grids of the one-dimensional kernels: equal CTA counts per slab for short runs, every SM for long ones
    assert attn.linfusion_attn_plan(attn.make_desc(2, 20, 4096, 64), 148)[2] == 120
    assert attn.linfusion_attn_plan(attn.make_desc(2, 10, 16384, 64), 148)[2] == 140
    assert attn.linfusion_attn_plan(attn.make_desc(2, 10, 524288, 64), 148)[2] == 148
    assert attn.linfusion_attn_plan(attn.make_desc(2, 8, 4096, 40), 148)[2] == 128        # 8 CTAs per slab
    assert attn.linfusion_attn_plan(attn.make_desc(2, 8, 1024, 80), 148)[2] == 64         # 4 per slab
    assert attn.linfusion_attn_plan(attn.make_desc(2, 8, 256, 160), 148)[2] == 16         # one per slab
    assert attn.linfusion_attn_plan(attn.make_desc(32, 8, 4096, 40), 148)[2] == 148       # whole slabs in turn
    assert attn.linfusion_attn_plan(attn.make_desc(2, 8, 1024, 160), 148)[2] == 128       # 8 per slab, sharing the summing
    assert attn.linfusion_attn_plan(attn.make_desc(1, 1, 100000, 160), 148)[2] == 131
    # a requested variant is kept; a smaller device changes the split
    assert attn.linfusion_attn_plan(attn.make_desc(2, 8, 4096, 40, variant="split"), 148)[0] == "split"
    assert attn.linfusion_attn_plan(attn.make_desc(2, 20, 4096, 64), 74)[2] == 74         # 40 of 74 SMs would be too few
    lib = attn.load_library()
    assert lib.linfusion_attn_plan(None, 0, None, None, None) == attn.ERR_INVALID_ARG
    with pytest.raises(attn.LinFusionError) as e:
        attn.linfusion_attn_plan(attn.make_desc(2, 8, 4096, 48), 148)
    assert e.value.code == attn.ERR_UNSUPPORTED
