"""fp64 CPU oracle of the filtered backward pass of a STRIDED convolution.

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests, the smoke check and the benchmark's
CPU-baseline leg may import this module.  It never touches the CUDA library.

The paper writes its method for stride 1 (Eq. (grad_x) indexes g_x and g_y with the same (h, w)),
yet the networks it fine-tunes have stride-2 convolutions inside the trained range, and its ImageNet
table books the stride-2 layer's stash on the patch grid of that layer's g_y (a 14 x 14 input kept as
4 x 4 values per channel at r = 2).  PARITY UNPINNED BY THE PAPER: the formulas below are this
library's reading, obtained by carrying the paper's own two approximations over to stride s --

  * the gradient filter (Section 3.3) acts on g_y [N, C_out, H/s, W/s] with patch size r;
  * inside a patch g~_y is treated as constant at every offset the kernel reaches ("padded
    patches" of the supplement), and x is replaced by its average over the window of x that the
    patch sees: the (r s) x (r s) block of pixels [a r s, (a+1) r s) x [b r s, (b+1) r s);

and they are pinned by what exact backpropagation fixes (tests/test_oracle_strided_pins.py): the
exact strided backward against fp64 autograd; equality with the exact input gradient of the
expanded g~_y at every pixel whose kernel footprint stays inside one patch, and everywhere for
1 x 1 kernels; equality of g~_W with the exact centre tap when x is window-constant; reduction to
the stride-1 oracle at s = 1; and the stash grid of the paper's table.

Geometry: odd K, pad (K-1)/2, s | H and s | W, so g_y is [N, C_out, H/s, W/s].
  stash   X~[n,c,a,b]      = sum of x over window (a, b)                      (window r s)
  phases  Th[p,q][co,cl]   = sum of theta[co,cl,u,v] over taps with (p + pad_h - u) % s == 0 and
                             (q + pad_w - v) % s == 0: the taps through which pixel phase (p, q) =
                             (h % s, w % s) of x reaches any output at all
  g~_X[n,ci,h,w]           = sum_co G-[n,co,h // (r s), w // (r s)] Th[h % s, w % s][co,cl]
  g~_W[co,cl,u,v]          = (1 / s^2) sum_{n,a,b} X~[n,ci,a,b] G-[n,co,a,b]     for every tap
(the factor 1/s^2: a patch holds r^2 outputs, each of which meets ONE pixel of x per tap, and
the window average stands for that pixel: r^2 X~ / (r s)^2).
"""
from __future__ import annotations

import numpy as np

from . import gf_oracle as _o


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def exact_backward_strided(x, gy, theta, stride: int, groups: int = 1, pad: tuple[int, int] | int = 0,
                           need_gw: bool = True, need_gx: bool = True):
    """Vanilla BP of a strided convolution by brute force over the taps (Section 3.1 with the output
    sampled every `stride` pixels): y[n,co,i,j] = sum theta[co,cl,u,v] x[n,ci,s i + u - ph, s j + v - pw]."""
    x, gy, theta = _f64(x), _f64(gy), _f64(theta)
    ph, pw = (pad, pad) if isinstance(pad, int) else pad
    N, Cin, H, W = x.shape
    Cout, Cig, KH, KW = theta.shape
    s = stride
    Hy, Wy = (H + 2 * ph - KH) // s + 1, (W + 2 * pw - KW) // s + 1
    assert gy.shape == (N, Cout, Hy, Wy) and Cig * groups == Cin
    Cog = Cout // groups
    gw = np.zeros_like(theta) if need_gw else None
    gx = np.zeros_like(x) if need_gx else None
    for i in range(Hy):
        for j in range(Wy):
            for u in range(KH):
                for v in range(KW):
                    h, w = s * i + u - ph, s * j + v - pw
                    if h < 0 or h >= H or w < 0 or w >= W:
                        continue
                    for q in range(groups):
                        co = slice(q * Cog, (q + 1) * Cog)
                        ci = slice(q * Cig, (q + 1) * Cig)
                        if need_gw:      # [Cog, Cig] += sum_n gy[n, co] x[n, ci]
                            gw[co, :, u, v] += gy[:, co, i, j].T @ x[:, ci, h, w]
                        if need_gx:      # [N, Cig] += gy[n, co] theta[co, cl]
                            gx[:, ci, h, w] += gy[:, co, i, j] @ theta[co, :, u, v]
    return gw, gx


def kernel_phase_sums(theta, stride: int, pad: tuple[int, int] | None = None) -> np.ndarray:
    """[s, s, C_out, C_ig]: per pixel phase of x, the sum of the taps that connect it to an output."""
    theta = _f64(theta)
    Cout, Cig, KH, KW = theta.shape
    ph, pw = ((KH - 1) // 2, (KW - 1) // 2) if pad is None else pad
    s = stride
    out = np.zeros((s, s, Cout, Cig), dtype=np.float64)
    for p in range(s):
        for q in range(s):
            for u in range(KH):
                for v in range(KW):
                    if (p + ph - u) % s == 0 and (q + pw - v) % s == 0:
                        out[p, q] += theta[:, :, u, v]
    return out


def strided_stash_forward(x, r: int, stride: int) -> np.ndarray:
    """What the forward pass keeps: x summed over the windows that the patches of g_y see."""
    if r == 1:
        return _f64(x).copy()
    return _o.patch_sum(x, r * stride)


def strided_backward(gy, stash, theta, r: int, stride: int, groups: int = 1, need_gw: bool = True, need_gx: bool = True):
    """(g~_W, g~_X) of a strided layer from g_y [N,C_out,H/s,W/s], the stash and theta; r >= 2."""
    gy, stash, theta = _f64(gy), _f64(stash), _f64(theta)
    assert r >= 2
    s = stride
    N, Cout, Hy, Wy = gy.shape
    Cout2, Cig, KH, KW = theta.shape
    assert Cout == Cout2
    Cin, Cog = Cig * groups, Cout // groups
    H, W = Hy * s, Wy * s
    gm = _o.patch_mean(gy, r)
    Hp, Wp = gm.shape[2], gm.shape[3]
    assert stash.shape == (N, Cin, Hp, Wp)
    gw = gx = None
    if need_gw:
        gw = _o.reduced_gw(stash, gm, groups, KH, KW) / float(s * s)
    if need_gx:
        th = kernel_phase_sums(theta, s)
        gx = np.empty((N, Cin, H, W), dtype=np.float64)
        for h in range(H):
            for w in range(W):
                a, b = h // (r * s), w // (r * s)
                for q in range(groups):
                    co = slice(q * Cog, (q + 1) * Cog)
                    ci = slice(q * Cig, (q + 1) * Cig)
                    gx[:, ci, h, w] = gm[:, co, a, b] @ th[h % s, w % s][co, :]
    return gw, gx
