"""Host-only checks of the C-ABI library: it loads without a GPU, exports every
symbol include/gf.h declares, and rejects bad arguments with the documented
status codes before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    """Every function declared in include/*.h (gf.h: the method; gf_bench.h: instrumentation)."""
    names = set()
    inc = os.path.join(ROOT, "include")
    for header in sorted(os.listdir(inc)):
        if not header.endswith(".h"):
            continue
        text = open(os.path.join(inc, header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names.update(re.findall(r"\b(gf_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol(gf):
    L = gf.lib()
    names = declared_symbols()
    assert "gf_backward" in names and "gf_stash_forward" in names
    for n in names:
        assert hasattr(L, n), n
    assert set(gf.binding.EXPORTS) == set(names)


def test_status_strings(gf):
    for code in range(8):
        assert gf.status_string(code).startswith("GF_")
    assert "unknown" in gf.status_string(99)


def test_stash_dims_are_ceil_mode(gf):
    d = gf.make_desc(3, 10, 20, 14, 15, 3, r=4)
    assert gf.gf_stash_dims(d) == (3, 10, 4, 4)
    assert gf.gf_stash_bytes(d) == 3 * 10 * 16 * 4
    d = gf.make_desc(3, 10, 20, 14, 15, 3, r=4, dtype=gf.GF_BF16)
    assert gf.gf_stash_bytes(d) == 3 * 10 * 16 * 2
    d = gf.make_desc(3, 10, 20, 14, 15, 3, r=1)
    assert gf.gf_stash_dims(d) == (3, 10, 14, 15)
    d = gf.make_desc(1, 4, 4, 5, 6, 3, r=9)
    assert gf.gf_stash_dims(d) == (1, 4, 1, 1)


def _golden_rows():
    path = os.path.join(os.path.dirname(__file__), "golden", "table_imagenet_mem.txt")
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, layers = line.split("|")
        model, k, vanilla, ours = head.split()
        yield model, int(k), float(ours), [tuple(int(t) for t in lay.split(",")) for lay in layers.split(";")]


@pytest.mark.parametrize("model,k,ours_kb,shapes", list(_golden_rows()))
def test_stash_bytes_match_the_papers_mem_column(gf, model, k, ours_kb, shapes):
    """Table "ImageNet classification", column Mem, rows "Ours" (fp32, batch 1, r = 2).
    The stash lives on the grid of g_y, so a layer is described by its g_y map."""
    total = 0
    for c_in, hx, wx, hy, wy in shapes:
        stride = hx // hy
        assert hx == hy * stride and wx == wy * stride
        total += gf.gf_stash_bytes(gf.make_desc(1, c_in, c_in, hx, wx, 3, r=2, stride=stride))
    assert abs(total / 1024 - ours_kb) < 0.005


def _status(gf, fn, *args):
    try:
        fn(*args)
    except gf.GfError as e:
        return e.status
    return gf.GF_OK


def test_descriptor_validation(gf):
    ok = dict(N=2, C_in=8, C_out=8, H=8, W=8, KH=3, r=2)

    def st(**kw):
        a = dict(ok)
        a.update(kw)
        pos = [a.pop(k) for k in ("N", "C_in", "C_out", "H", "W", "KH")]
        return _status(gf, gf.gf_backward_workspace_bytes, gf.make_desc(*pos, **a))

    assert st() == gf.GF_OK
    assert st(N=0) == gf.GF_ERR_BAD_DESC
    assert st(r=0) == gf.GF_ERR_BAD_DESC
    assert st(groups=3) == gf.GF_ERR_BAD_DESC
    assert st(dtype=7) == gf.GF_ERR_BAD_DESC
    assert st(layout=5) == gf.GF_ERR_BAD_DESC
    # channels-last with r >= 2: stride 1, channel counts in multiples of 8, dense or depthwise
    assert st(layout=gf.GF_NHWC) == gf.GF_OK
    assert st(layout=gf.GF_NHWC, groups=8) == gf.GF_OK
    assert st(layout=gf.GF_NHWC, C_in=12, C_out=12) == gf.GF_ERR_UNSUPPORTED
    assert st(layout=gf.GF_NHWC, groups=2) == gf.GF_ERR_UNSUPPORTED
    assert st(layout=gf.GF_NHWC, stride=2) == gf.GF_ERR_UNSUPPORTED
    assert st(layout=gf.GF_NHWC, r=1) == gf.GF_OK                  # exact backward: as for NCHW
    assert st(layout=gf.GF_NHWC, r=1, C_in=12, C_out=12, groups=2) == gf.GF_OK
    assert st(stride=2) == gf.GF_OK                          # s | H and s | W: g_y is [H/s, W/s]
    assert st(stride=3) == gf.GF_ERR_UNSUPPORTED             # 3 does not divide 8
    assert st(stride=0) == gf.GF_ERR_BAD_DESC
    assert st(KH=2) == gf.GF_ERR_UNSUPPORTED
    assert st(pad_h=0) == gf.GF_ERR_UNSUPPORTED
    assert st(KH=3, KW=5, pad_w=1) == gf.GF_ERR_UNSUPPORTED
    assert st(KH=3, KW=5) == gf.GF_OK
    assert st(groups=8) == gf.GF_OK and st(groups=4) == gf.GF_OK


def test_pointer_validation_happens_before_any_launch(gf):
    L = gf.lib()
    d = gf.make_desc(2, 8, 8, 8, 8, 3, r=2)
    vp = ctypes.c_void_p
    a, b = vp(0x1000), vp(0x2000)   # never dereferenced: all calls fail on the host
    assert L.gf_stash_forward(None, a, b, None) == gf.GF_ERR_NULL
    assert L.gf_stash_forward(ctypes.byref(d), None, b, None) == gf.GF_ERR_NULL
    assert L.gf_stash_forward(ctypes.byref(d), vp(0x1004), b, None) == gf.GF_ERR_ALIGN
    assert L.gf_backward(ctypes.byref(d), None, a, a, a, a, a, 1 << 30, None) == gf.GF_ERR_NULL
    assert L.gf_backward(ctypes.byref(d), a, a, a, a, a, None, 1 << 30, None) == gf.GF_ERR_NULL
    assert L.gf_backward(ctypes.byref(d), a, None, a, a, a, a, 1 << 30, None) == gf.GF_ERR_NULL
    assert L.gf_backward(ctypes.byref(d), a, a, a, a, vp(0x1008), a, 1 << 30, None) == gf.GF_ERR_ALIGN
    assert L.gf_backward(ctypes.byref(d), a, a, a, a, a, a, 16, None) == gf.GF_ERR_WORKSPACE
    need = gf.gf_backward_workspace_bytes(d)
    assert L.gf_backward(ctypes.byref(d), a, a, a, a, a, a, need - 1, None) == gf.GF_ERR_WORKSPACE
    assert L.gf_layer_step_host(ctypes.byref(d), a, a, a, a, a, a, 16, None) == gf.GF_ERR_WORKSPACE
    assert L.gf_last_async_status(None, None) == gf.GF_ERR_NULL
    assert gf.gf_host_step_arena_bytes(d) > need


def test_missing_library_fails_loudly(gf, monkeypatch):
    from paper_2301_00330_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "library_path", lambda: "/nonexistent/libgf_b200.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.gf_kernel_launch_count()


def test_product_never_imports_the_checker():
    pkg = os.path.join(ROOT, "paper_2301_00330_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), os.path.join(dirpath, f)


def test_diagnostics_reject_bad_arguments(gf):
    """Section 4.1 diagnostics: argument checks come before anything touches the device."""
    L = gf.lib()
    a = ctypes.c_void_p(0x1000)
    assert L.gf_snr_terms(None, a, 4, 0, a, None) == gf.GF_ERR_NULL
    assert L.gf_snr_terms(a, a, -1, 0, a, None) == gf.GF_ERR_BAD_DESC
    assert L.gf_snr_terms(a, a, 4, 0, ctypes.c_void_p(0x1004), None) == gf.GF_ERR_ALIGN
    assert L.gf_filter_snr_terms(a, 1, 0, 4, 2, 0, a, None) == gf.GF_ERR_BAD_DESC
    assert L.gf_dcac_ratio(a, 1, 1, 3, 3, 2, 3, 0, a, None) == gf.GF_ERR_BAD_DESC          # DFT smaller than the kernel
    assert L.gf_dcac_ratio(a, 1, 1, 3, 3, 128, 3, 0, a, None) == gf.GF_ERR_UNSUPPORTED


def test_int8_entry_point_validates_on_the_host(gf):
    """gf_backward_int8: dense stride-1 layers with r >= 2 whose integer sums fit 32 bits."""
    L = gf.lib()
    size = ctypes.c_size_t(0)
    ok = gf.make_desc(2, 8, 8, 8, 8, 3, r=2)
    assert L.gf_backward_int8_workspace_bytes(ctypes.byref(ok), ctypes.byref(size)) == gf.GF_OK and size.value > 0
    for bad in (gf.make_desc(2, 8, 8, 8, 8, 3, r=1), gf.make_desc(2, 8, 8, 8, 8, 3, r=2, groups=2),
                gf.make_desc(2, 8, 8, 8, 8, 3, r=2, stride=2), gf.make_desc(4096, 8, 8, 64, 64, 3, r=2)):
        assert L.gf_backward_int8_workspace_bytes(ctypes.byref(bad), ctypes.byref(size)) == gf.GF_ERR_UNSUPPORTED
    a = ctypes.c_void_p(0x1000)
    assert L.gf_backward_int8(ctypes.byref(ok), a, a, a, a, a, a, 16, None) == gf.GF_ERR_WORKSPACE
    assert L.gf_backward_int8(ctypes.byref(ok), None, a, a, a, a, a, 1 << 30, None) == gf.GF_ERR_NULL
