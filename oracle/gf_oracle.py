"""numpy front end of the fp64 CPU oracle (oracle/gf_oracle.c).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests, the smoke check and the
benchmark's CPU-baseline leg may import this module.  It never touches the CUDA
library.  Every array is converted to contiguous float64 before the C loops run.

The functions mirror the paper's steps one to one:

  patch_sum      x~  (Section 3.4, text after Eq. (grad_w))
  patch_mean     unique values of g~_y (Section 3.3)
  kernel_sum     theta~' (text under Eq. (grad_x))
  reduced_gw     Eq. (grad_w), once per patch, broadcast to every tap
  reduced_gx     Eq. (grad_x) + expansion
  exact_backward vanilla BP by brute force (Section 3.1); also the r == 1 case
  literal_backward  the supplement's derivations with padded patches, no pre-sums

``stash_forward`` / ``backward`` compose them in the order of the method.
Partial edge patches use the mean over existing elements: PARITY UNPINNED for
that divisor (see the header of gf_oracle.c).
"""
from __future__ import annotations

import ctypes

import numpy as np

from . import build as _build

_lib = None
_i64 = ctypes.c_int64
_dp = ctypes.POINTER(ctypes.c_double)


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        _lib.gfo_num_threads.restype = ctypes.c_int
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _p(a: np.ndarray | None):
    if a is None:
        return ctypes.cast(None, _dp)
    return a.ctypes.data_as(_dp)


def num_threads() -> int:
    return int(_load().gfo_num_threads())


def grid(H: int, W: int, r: int) -> tuple[int, int]:
    """ceil(H/r) x ceil(W/r) patches per channel (Section 3.3)."""
    return -(-H // r), -(-W // r)


def patch_sum(x, r: int) -> np.ndarray:
    x = _f64(x)
    N, C, H, W = x.shape
    Hp, Wp = grid(H, W, r)
    out = np.empty((N, C, Hp, Wp), dtype=np.float64)
    _load().gfo_patch_sum(_p(x), _i64(N), _i64(C), _i64(H), _i64(W), _i64(r), _p(out))
    return out


def patch_mean(g, r: int) -> np.ndarray:
    g = _f64(g)
    N, C, H, W = g.shape
    Hp, Wp = grid(H, W, r)
    out = np.empty((N, C, Hp, Wp), dtype=np.float64)
    _load().gfo_patch_mean(_p(g), _i64(N), _i64(C), _i64(H), _i64(W), _i64(r), _p(out))
    return out


def expand(u, H: int, W: int, r: int) -> np.ndarray:
    u = _f64(u)
    N, C, Hp, Wp = u.shape
    assert (Hp, Wp) == grid(H, W, r)
    out = np.empty((N, C, H, W), dtype=np.float64)
    _load().gfo_expand(_p(u), _i64(N), _i64(C), _i64(H), _i64(W), _i64(r), _p(out))
    return out


def kernel_sum(theta) -> np.ndarray:
    theta = _f64(theta)
    Cout, Cig, KH, KW = theta.shape
    out = np.empty((Cout, Cig), dtype=np.float64)
    _load().gfo_kernel_sum(_p(theta), _i64(Cout), _i64(Cig), _i64(KH), _i64(KW), _p(out))
    return out


def reduced_gw(xs, gm, groups: int, KH: int, KW: int) -> np.ndarray:
    xs, gm = _f64(xs), _f64(gm)
    N, Cin, Hp, Wp = xs.shape
    N2, Cout, Hp2, Wp2 = gm.shape
    assert (N, Hp, Wp) == (N2, Hp2, Wp2)
    assert Cin % groups == 0 and Cout % groups == 0
    out = np.empty((Cout, Cin // groups, KH, KW), dtype=np.float64)
    _load().gfo_reduced_gw(_p(xs), _p(gm), _i64(N), _i64(Cin), _i64(Cout), _i64(groups),
                           _i64(Hp), _i64(Wp), _i64(KH), _i64(KW), _p(out))
    return out


def reduced_gx(gm, ts, groups: int, H: int, W: int, r: int) -> np.ndarray:
    gm, ts = _f64(gm), _f64(ts)
    N, Cout, Hp, Wp = gm.shape
    Cout2, Cig = ts.shape
    assert Cout == Cout2 and (Hp, Wp) == grid(H, W, r)
    Cin = Cig * groups
    out = np.empty((N, Cin, H, W), dtype=np.float64)
    _load().gfo_reduced_gx(_p(gm), _p(ts), _i64(N), _i64(Cin), _i64(Cout), _i64(groups),
                           _i64(H), _i64(W), _i64(r), _p(out))
    return out


def exact_backward(x, gy, theta, groups: int = 1, pad: tuple[int, int] | int = 0,
                   need_gw: bool = True, need_gx: bool = True):
    """Vanilla BP of a stride-1 convolution by brute force (Section 3.1)."""
    x, gy, theta = _f64(x), _f64(gy), _f64(theta)
    ph, pw = (pad, pad) if isinstance(pad, int) else pad
    N, Cin, H, W = x.shape
    Cout, Cig, KH, KW = theta.shape
    assert Cig * groups == Cin and Cout % groups == 0
    assert gy.shape == (N, Cout, H + 2 * ph - KH + 1, W + 2 * pw - KW + 1)
    gw = np.empty_like(theta) if need_gw else None
    gx = np.empty_like(x) if need_gx else None
    _load().gfo_exact_backward(_p(x), _p(gy), _p(theta), _i64(N), _i64(Cin), _i64(Cout),
                               _i64(groups), _i64(H), _i64(W), _i64(KH), _i64(KW),
                               _i64(ph), _i64(pw), _p(gw), _p(gx))
    return gw, gx


def literal_backward(x, gy, theta, r: int, groups: int = 1,
                     need_gw: bool = True, need_gx: bool = True):
    """The supplement's derivations taken literally (padded patches, theta not
    pre-summed, loops over full-resolution pixels and taps)."""
    x, gy, theta = _f64(x), _f64(gy), _f64(theta)
    N, Cin, H, W = x.shape
    Cout, Cig, KH, KW = theta.shape
    gm = patch_mean(gy, r)
    # x replaced by its patch-constant field: unique value = patch sum / |patch|
    xmean = patch_mean(x, r)
    gw = np.empty_like(theta) if need_gw else None
    gx = np.empty_like(x) if need_gx else None
    _load().gfo_literal_backward(_p(xmean), _p(gm), _p(theta), _i64(N), _i64(Cin),
                                 _i64(Cout), _i64(groups), _i64(H), _i64(W), _i64(r),
                                 _i64(KH), _i64(KW), _p(gw), _p(gx))
    return gw, gx


# ---------------------------------------------------------------------------
# The method, in its own order
# ---------------------------------------------------------------------------

def activation(z, kind: str) -> np.ndarray:
    """The producers of x in the paper's networks: "none", "relu" = max(z, 0) (ResNet),
    "relu6" = min(max(z, 0), 6) (MobileNetV2, MCUNet).  Plain element-wise definitions."""
    z = _f64(z)
    out = np.empty_like(z)
    flat_in, flat_out = z.reshape(-1), out.reshape(-1)
    for i in range(flat_in.size):
        v = flat_in[i]
        if kind == "relu":
            v = v if v > 0.0 else 0.0
        elif kind == "relu6":
            v = 0.0 if v < 0.0 else (6.0 if v > 6.0 else v)
        elif kind != "none":
            raise ValueError(kind)
        flat_out[i] = v
    return out


def activation_fast(z, kind: str) -> np.ndarray:
    """activation() through numpy's clip, for tensors too large for a Python loop."""
    z = _f64(z)
    if kind == "none":
        return z.copy()
    return np.clip(z, 0.0, 6.0 if kind == "relu6" else None)


def act_stash_forward(z, kind: str, r: int):
    """Forward-side step fused into the producer of x (Section 4.2): x = act(z) and the stash of
    that x.  Returns (x, stash)."""
    x = activation_fast(z, kind)
    return x, stash_forward(x, r)


def stash_forward(x, r: int) -> np.ndarray:
    """What the forward pass keeps instead of x.  r == 1: x itself."""
    if r == 1:
        return _f64(x).copy()
    return patch_sum(x, r)


def backward(gy, stash, theta, r: int, groups: int = 1, pad: tuple[int, int] | int | None = None,
             need_gw: bool = True, need_gx: bool = True):
    """Filtered convolution backward: (g_W, g_X) from g_y, the stash and theta.

    r >= 2: gradient filter, kernel sum, Eq. (grad_w), Eq. (grad_x) + expansion.
    r == 1: exact convolution backward, the stash being x.
    """
    gy, stash, theta = _f64(gy), _f64(stash), _f64(theta)
    Cout, Cig, KH, KW = theta.shape
    if pad is None:
        pad = ((KH - 1) // 2, (KW - 1) // 2)
    if r == 1:
        return exact_backward(stash, gy, theta, groups, pad, need_gw, need_gx)
    N, _, H, W = gy.shape
    gm = patch_mean(gy, r)
    gw = reduced_gw(stash, gm, groups, KH, KW) if need_gw else None
    gx = reduced_gx(gm, kernel_sum(theta), groups, H, W, r) if need_gx else None
    return gw, gx


def stash_num_values(C_in: int, H_y: int, W_y: int, r: int) -> int:
    """Values kept per image for one layer: one per channel and per patch of the
    g_y grid (Section 4.3: ceil(H/r) ceil(W/r) unique elements per channel)."""
    Hp, Wp = grid(H_y, W_y, r)
    return C_in * Hp * Wp
