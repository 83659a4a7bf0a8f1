"""ctypes binding over the C ABI declared in include/gf.h.

Argument marshalling only: every step of the method runs in the CUDA kernels
of libgf_b200.so.  torch is used for device memory and streams.  There is no
CPU fallback: if the library is missing or cannot be loaded, every entry point
raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

from . import build as _build

GF_OK, GF_ERR_NULL, GF_ERR_BAD_DESC, GF_ERR_UNSUPPORTED = 0, 1, 2, 3
GF_ERR_WORKSPACE, GF_ERR_ALIGN, GF_ERR_CUDA, GF_ERR_TIMEOUT = 4, 5, 6, 7
GF_F32, GF_BF16 = 0, 1
GF_NCHW, GF_NHWC = 0, 1
GF_PATH_AUTO, GF_PATH_FUSED, GF_PATH_SPLIT = 0, 1, 2
GF_ACT_NONE, GF_ACT_RELU, GF_ACT_RELU6 = 0, 1, 2

EXPORTS = (
    "gf_stash_dims", "gf_stash_bytes", "gf_backward_workspace_bytes", "gf_stash_forward",
    "gf_backward", "gf_last_async_status", "gf_host_step_arena_bytes", "gf_layer_step_host",
    "gf_kernel_launch_count", "gf_status_string", "gf_profile_configure", "gf_profile_read",
    "gf_kernel_name", "gf_kernel_id_count", "gf_backward_static_scratch", "gf_set_dense_path",
    "gf_snr_terms", "gf_filter_snr_terms", "gf_dcac_ratio", "gf_act_stash_forward",
    "gf_backward_int8", "gf_backward_int8_workspace_bytes", "gf_selftest_bounded_wait",
)


class gf_conv_desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("N", "C_in", "C_out", "H", "W", "KH", "KW", "stride", "pad_h", "pad_w",
                 "groups", "r", "dtype", "layout")]


class gf_kernel_time(ctypes.Structure):
    _fields_ = [("kernel_id", ctypes.c_int32), ("launches", ctypes.c_int32), ("total_ms", ctypes.c_double)]


class GfError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)}")


_lib = None


def library_path() -> str:
    return _build.LIB


def build_library(force: bool = False) -> str:
    """Compile libgf_b200.so for sm_100a if it is missing or stale."""
    return _build.build(force=force)


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise RuntimeError(
                f"{path} is missing: build it with `python -m paper_2301_00330_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(path)
        vp, sz = ctypes.c_void_p, ctypes.c_size_t
        dp = ctypes.POINTER(gf_conv_desc)
        L.gf_stash_dims.argtypes = [dp, ctypes.POINTER(ctypes.c_int64 * 4)]
        L.gf_stash_bytes.argtypes = [dp, ctypes.POINTER(sz)]
        L.gf_backward_workspace_bytes.argtypes = [dp, ctypes.POINTER(sz)]
        L.gf_stash_forward.argtypes = [dp, vp, vp, vp]
        L.gf_act_stash_forward.argtypes = [dp, ctypes.c_int32, vp, vp, vp, vp]
        L.gf_act_stash_forward.restype = ctypes.c_int
        L.gf_backward.argtypes = [dp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.gf_backward_int8.argtypes = [dp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.gf_backward_int8.restype = ctypes.c_int
        L.gf_backward_int8_workspace_bytes.argtypes = [dp, ctypes.POINTER(sz)]
        L.gf_backward_int8_workspace_bytes.restype = ctypes.c_int
        L.gf_backward_static_scratch.argtypes = [dp, vp, vp, vp, vp, vp, vp]
        L.gf_backward_static_scratch.restype = ctypes.c_int
        L.gf_last_async_status.argtypes = [vp, vp]
        L.gf_host_step_arena_bytes.argtypes = [dp, ctypes.POINTER(sz)]
        L.gf_layer_step_host.argtypes = [dp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.gf_kernel_launch_count.argtypes = []
        L.gf_kernel_launch_count.restype = ctypes.c_uint64
        L.gf_profile_configure.argtypes = [ctypes.c_int32, ctypes.c_int32]
        L.gf_profile_configure.restype = ctypes.c_int
        L.gf_profile_read.argtypes = [ctypes.POINTER(gf_kernel_time), ctypes.c_int32]
        L.gf_profile_read.restype = ctypes.c_int32
        L.gf_kernel_name.argtypes = [ctypes.c_int32]
        L.gf_kernel_name.restype = ctypes.c_char_p
        L.gf_kernel_id_count.argtypes = []
        L.gf_kernel_id_count.restype = ctypes.c_int32
        L.gf_set_dense_path.argtypes = [ctypes.c_int32]
        L.gf_set_dense_path.restype = ctypes.c_int
        i32, i64 = ctypes.c_int32, ctypes.c_int64
        L.gf_snr_terms.argtypes = [vp, vp, i64, i32, vp, vp]
        L.gf_filter_snr_terms.argtypes = [vp, i64, i32, i32, i32, i32, vp, vp]
        L.gf_dcac_ratio.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32, vp, vp]
        for name in ("gf_snr_terms", "gf_filter_snr_terms", "gf_dcac_ratio"):
            getattr(L, name).restype = ctypes.c_int
        L.gf_selftest_bounded_wait.argtypes = [vp, ctypes.c_int64, vp]
        L.gf_selftest_bounded_wait.restype = ctypes.c_int
        L.gf_status_string.argtypes = [ctypes.c_int]
        L.gf_status_string.restype = ctypes.c_char_p
        for name in ("gf_stash_dims", "gf_stash_bytes", "gf_backward_workspace_bytes", "gf_stash_forward",
                     "gf_backward", "gf_last_async_status", "gf_host_step_arena_bytes", "gf_layer_step_host"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().gf_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != GF_OK:
        raise GfError(status, where)


def make_desc(N, C_in, C_out, H, W, KH, KW=None, *, r, groups=1, stride=1, pad_h=None, pad_w=None,
              dtype=GF_F32, layout=GF_NCHW) -> gf_conv_desc:
    KW = KH if KW is None else KW
    pad_h = (KH - 1) // 2 if pad_h is None else pad_h
    pad_w = (KW - 1) // 2 if pad_w is None else pad_w
    if isinstance(dtype, torch.dtype):
        dtype = {torch.float32: GF_F32, torch.bfloat16: GF_BF16}[dtype]
    return gf_conv_desc(N, C_in, C_out, H, W, KH, KW, stride, pad_h, pad_w, groups, r, dtype, layout)


def desc_for(layer) -> gf_conv_desc:
    """Descriptor of a workloads.Layer."""
    return make_desc(layer.N, layer.C_in, layer.C_out, layer.H, layer.W, layer.K, r=layer.r,
                     groups=layer.groups, dtype=GF_F32 if layer.dtype == "f32" else GF_BF16)


def _ptr(t) -> ctypes.c_void_p:
    if t is None:
        return ctypes.c_void_p(0)
    if isinstance(t, torch.Tensor):
        # dense in either order; which one the bytes are in is the descriptor's `layout`
        if not (t.is_contiguous() or (t.dim() == 4 and t.is_contiguous(memory_format=torch.channels_last))):
            raise ValueError("tensors passed to the gf_* calls must be dense (contiguous, or channels_last for GF_NHWC)")
        return ctypes.c_void_p(t.data_ptr())
    return ctypes.c_void_p(int(t))


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    if isinstance(stream, torch.cuda.Stream):
        return ctypes.c_void_p(stream.cuda_stream)
    return ctypes.c_void_p(int(stream))


# ---- the C calls, same names ----------------------------------------------------

def gf_stash_dims(desc: gf_conv_desc) -> tuple[int, int, int, int]:
    dims = (ctypes.c_int64 * 4)()
    _check(lib().gf_stash_dims(ctypes.byref(desc), ctypes.byref(dims)), "gf_stash_dims")
    return tuple(int(v) for v in dims)


def gf_stash_bytes(desc: gf_conv_desc) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().gf_stash_bytes(ctypes.byref(desc), ctypes.byref(out)), "gf_stash_bytes")
    return int(out.value)


def gf_backward_workspace_bytes(desc: gf_conv_desc) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().gf_backward_workspace_bytes(ctypes.byref(desc), ctypes.byref(out)),
           "gf_backward_workspace_bytes")
    return int(out.value)


def gf_stash_forward(desc: gf_conv_desc, x, stash, stream=None) -> None:
    _check(lib().gf_stash_forward(ctypes.byref(desc), _ptr(x), _ptr(stash), _stream(stream)),
           "gf_stash_forward")


def gf_act_stash_forward(desc: gf_conv_desc, act: int, z, x, stash, stream=None) -> None:
    """x <- act(z) and stash <- patch sums of x, in one pass over z (x may be z)."""
    _check(lib().gf_act_stash_forward(ctypes.byref(desc), int(act), _ptr(z), _ptr(x), _ptr(stash), _stream(stream)),
           "gf_act_stash_forward")


def gf_backward(desc: gf_conv_desc, g_y, stash, W, g_W, g_X, workspace, workspace_bytes=None,
                stream=None) -> None:
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(lib().gf_backward(ctypes.byref(desc), _ptr(g_y), _ptr(stash), _ptr(W), _ptr(g_W), _ptr(g_X),
                             _ptr(workspace), ctypes.c_size_t(workspace_bytes), _stream(stream)),
           "gf_backward")


def gf_backward_int8_workspace_bytes(desc: gf_conv_desc) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().gf_backward_int8_workspace_bytes(ctypes.byref(desc), ctypes.byref(out)), "gf_backward_int8_workspace_bytes")
    return int(out.value)


def gf_backward_int8(desc: gf_conv_desc, g_y, stash, W, g_W, g_X, workspace, workspace_bytes=None, stream=None) -> None:
    """gf_backward with the operands of the two reduced contractions quantised to INT8."""
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(lib().gf_backward_int8(ctypes.byref(desc), _ptr(g_y), _ptr(stash), _ptr(W), _ptr(g_W), _ptr(g_X), _ptr(workspace),
                                  ctypes.c_size_t(workspace_bytes), _stream(stream)), "gf_backward_int8")


GF_STATIC_SCRATCH_BYTES = 8 << 20


def gf_backward_static_scratch(desc: gf_conv_desc, g_y, stash, W, g_W, g_X, stream=None) -> None:
    """gf_backward without a workspace argument: the scratch is an array built into the
    library (GF_STATIC_SCRATCH_BYTES), for callers that may not allocate device memory.
    Calls must not overlap on the GPU; larger layers raise GfError(GF_ERR_WORKSPACE)."""
    _check(lib().gf_backward_static_scratch(ctypes.byref(desc), _ptr(g_y), _ptr(stash), _ptr(W), _ptr(g_W),
                                            _ptr(g_X), _stream(stream)), "gf_backward_static_scratch")


def gf_last_async_status(workspace, stream=None) -> int:
    return int(lib().gf_last_async_status(_ptr(workspace), _stream(stream)))


def gf_host_step_arena_bytes(desc: gf_conv_desc) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().gf_host_step_arena_bytes(ctypes.byref(desc), ctypes.byref(out)), "gf_host_step_arena_bytes")
    return int(out.value)


def gf_layer_step_host(desc: gf_conv_desc, h_x, h_gy, h_W, h_gW, h_gX, arena, arena_bytes=None,
                       stream=None) -> None:
    if arena_bytes is None:
        arena_bytes = arena.numel() * arena.element_size()
    _check(lib().gf_layer_step_host(ctypes.byref(desc), _ptr(h_x), _ptr(h_gy), _ptr(h_W), _ptr(h_gW),
                                    _ptr(h_gX), _ptr(arena), ctypes.c_size_t(arena_bytes), _stream(stream)),
           "gf_layer_step_host")


def gf_set_dense_path(path: int) -> None:
    """GF_PATH_AUTO (the library's choice per layer), GF_PATH_FUSED or GF_PATH_SPLIT, process-wide."""
    _check(lib().gf_set_dense_path(int(path)), "gf_set_dense_path")


def _gf_dtype(t: torch.Tensor) -> int:
    return {torch.float32: GF_F32, torch.bfloat16: GF_BF16}[t.dtype]


def gf_snr_terms(ref: torch.Tensor, approx: torch.Tensor, energies: torch.Tensor, stream=None) -> None:
    """energies (2 doubles on the device) <- sum ref^2, sum (ref - approx)^2."""
    assert ref.dtype == approx.dtype and ref.numel() == approx.numel() and energies.dtype == torch.float64
    _check(lib().gf_snr_terms(_ptr(ref), _ptr(approx), ctypes.c_int64(ref.numel()), _gf_dtype(ref), _ptr(energies),
                              _stream(stream)), "gf_snr_terms")


def gf_filter_snr_terms(g: torch.Tensor, r: int, energies: torch.Tensor, stream=None) -> None:
    """The SNR terms of the gradient filter with patch size r on g [..., H, W]."""
    assert energies.dtype == torch.float64 and g.dim() >= 2
    H, W = int(g.shape[-2]), int(g.shape[-1])
    _check(lib().gf_filter_snr_terms(_ptr(g), ctypes.c_int64(g.numel() // (H * W)), H, W, int(r), _gf_dtype(g),
                                     _ptr(energies), _stream(stream)), "gf_filter_snr_terms")


def gf_dcac_ratio(W: torch.Tensor, ratio: torch.Tensor, dft: tuple[int, int] = (0, 0), stream=None) -> None:
    """ratio [C_out, C_ig] (fp32, device) <- DC / largest AC energy of every kernel of W [C_out, C_ig, KH, KW]."""
    C_out, C_ig, KH, KW = (int(v) for v in W.shape)
    assert ratio.dtype == torch.float32 and ratio.numel() == C_out * C_ig
    _check(lib().gf_dcac_ratio(_ptr(W), C_out, C_ig, KH, KW, int(dft[0]), int(dft[1]), _gf_dtype(W), _ptr(ratio),
                               _stream(stream)), "gf_dcac_ratio")


def gf_selftest_bounded_wait(workspace, limit_cycles: int, stream=None) -> None:
    """Launches a block whose bounded wait must expire; it records that in the workspace's error word."""
    _check(lib().gf_selftest_bounded_wait(_ptr(workspace), ctypes.c_int64(int(limit_cycles)), _stream(stream)),
           "gf_selftest_bounded_wait")


def gf_kernel_launch_count() -> int:
    return int(lib().gf_kernel_launch_count())


def gf_kernel_id_count() -> int:
    return int(lib().gf_kernel_id_count())


def gf_kernel_name(kernel_id: int) -> str | None:
    n = lib().gf_kernel_name(int(kernel_id))
    return n.decode() if n else None


def kernel_id(name: str) -> int:
    for k in range(gf_kernel_id_count()):
        if gf_kernel_name(k) == name:
            return k
    raise KeyError(name)


def gf_profile_configure(mode: int, kernel_id: int = -1) -> None:
    _check(lib().gf_profile_configure(int(mode), int(kernel_id)), "gf_profile_configure")


def gf_profile_read() -> dict[str, tuple[int, float]]:
    """{kernel name: (timed launches, total ms)} since the last read."""
    n = gf_kernel_id_count()
    buf = (gf_kernel_time * n)()
    got = lib().gf_profile_read(buf, n)
    if got < 0:
        raise GfError(GF_ERR_CUDA, "gf_profile_read")
    return {gf_kernel_name(buf[i].kernel_id): (int(buf[i].launches), float(buf[i].total_ms)) for i in range(got)}


# ---- conveniences that only allocate ---------------------------------------------

@dataclass
class LayerBuffers:
    desc: gf_conv_desc
    stash: torch.Tensor
    g_W: torch.Tensor
    g_X: torch.Tensor
    workspace: torch.Tensor


def alloc_layer(desc: gf_conv_desc, device="cuda") -> LayerBuffers:
    dt = torch.float32 if desc.dtype == GF_F32 else torch.bfloat16
    stash = torch.empty(gf_stash_dims(desc), dtype=dt, device=device)
    g_W = torch.empty((desc.C_out, desc.C_in // desc.groups, desc.KH, desc.KW), dtype=torch.float32,
                      device=device)
    g_X = torch.empty((desc.N, desc.C_in, desc.H, desc.W), dtype=dt, device=device)
    ws = torch.empty(gf_backward_workspace_bytes(desc), dtype=torch.uint8, device=device)
    return LayerBuffers(desc, stash, g_W, g_X, ws)
