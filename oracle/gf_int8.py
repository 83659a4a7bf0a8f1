"""CPU oracle of the INT8 variant of the two reduced contractions (the supplement's section on
combining gradient filtering with gradient quantization: feature maps, weights and gradients as
INT8; Table "cifar_gq").

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests, the smoke check and the benchmark's
CPU-baseline leg may import this module.  It never touches the CUDA library.

The paper names the quantization schemes it combines with (per-tensor PTQ and per-sample PSQ, both
INT8) and gives no formulas; this oracle fixes the plainest of them, PER-TENSOR SYMMETRIC INT8 WITH
ROUND-TO-NEAREST-EVEN, applied to the three operands of the reduced contractions:

    scale(t) = max|t| / 127                    (1 when the tensor is all zeros)
    code(v)  = clamp(rint(v / scale), -127, 127)
    g~_W[co,ci,u,v] = (sum_{n,a,b} code_X[n,ci,a,b] code_G[n,co,a,b])    * (scale_X * scale_G)   (Eq. (grad_w))
    g~_X[n,ci,h,w]  = (sum_co code_G[n,co,h/r,w/r] code_Th[co,ci])        * (scale_G * scale_Th)  (Eq. (grad_x))

with X~ the stash, G- the patch means of g_y and Th the kernel sums.  The integer sums are exact
(int32 on the GPU, int64 here; the caller keeps K * 127^2 below 2^31).

A quantised code is an integer decided by floating-point arithmetic, so both sides must take that
decision in the same precision and order.  The precision is the kernel's, fp32, and the order is
fixed here: G- is the sum of the patch's elements taken row by row, left to right, in fp32, times
the fp32 reciprocal of their count; Th is the sum of the taps in memory order in fp32; scale and
code use fp32 division; the integer sum is converted to fp32, the two scales are multiplied in
fp32, and the two are multiplied in fp32.  Every step is an IEEE single-precision operation, which
numpy's float32 type reproduces bit for bit.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def patch_mean_f32(g, r: int) -> np.ndarray:
    """Patch means of g [N,C,H,W] in fp32, elements added row by row, left to right, from zero."""
    g = _f32(g)
    N, C, H, W = g.shape
    Hp, Wp = -(-H // r), -(-W // r)
    acc = np.zeros((N, C, Hp, Wp), dtype=F32)
    cnt = np.zeros((Hp, Wp), dtype=np.int64)
    for i in range(r):
        for j in range(r):
            sub = g[:, :, i::r, j::r]                    # element (i, j) of every patch that has one
            hp, wp = sub.shape[2], sub.shape[3]
            acc[:, :, :hp, :wp] = acc[:, :, :hp, :wp] + sub
            cnt[:hp, :wp] += 1
    inv = (F32(1.0) / cnt.astype(F32)).astype(F32)
    return (acc * inv).astype(F32)


def kernel_sum_f32(theta) -> np.ndarray:
    theta = _f32(theta)
    Cout, Cig, KH, KW = theta.shape
    acc = np.zeros((Cout, Cig), dtype=F32)
    for u in range(KH):
        for v in range(KW):
            acc = (acc + theta[:, :, u, v]).astype(F32)
    return acc


def quantize(t) -> tuple[np.ndarray, np.float32]:
    """(codes int8, scale fp32) of a tensor: per-tensor symmetric, round to nearest even."""
    t = _f32(t)
    amax = F32(np.max(np.abs(t))) if t.size else F32(0.0)
    scale = F32(amax / F32(127.0)) if amax > 0 else F32(1.0)
    codes = np.rint((t / scale).astype(F32))
    codes = np.clip(codes, -127.0, 127.0)
    return codes.astype(np.int8), scale


def dequantize(codes, scale) -> np.ndarray:
    return codes.astype(np.float64) * float(scale)


def int8_backward(gy, stash, theta, r: int, out_dtype=np.float32):
    """(g~_W [C_out,C_in,KH,KW] fp32, g~_X [N,C_in,H,W] fp32 values already rounded to out_dtype's
    grid by the caller if it is narrower) of a dense stride-1 layer with INT8 operands."""
    gm = patch_mean_f32(gy, r)
    N, Cout, Hp, Wp = gm.shape
    H, W = np.asarray(gy).shape[2:]
    theta = _f32(theta)
    KH, KW = theta.shape[2:]
    qg, sg = quantize(gm)
    qx, sx = quantize(stash)
    qt, st = quantize(kernel_sum_f32(theta))
    Cin = qx.shape[1]
    g64, x64, t64 = qg.astype(np.int64), qx.astype(np.int64), qt.astype(np.int64)
    acc_w = np.einsum("nopq,nipq->oi", g64, x64)                       # exact integers
    acc_x = np.einsum("nopq,oi->nipq", g64, t64)
    assert np.abs(acc_w).max(initial=0) < 2 ** 31 and np.abs(acc_x).max(initial=0) < 2 ** 31
    gw_u = (acc_w.astype(F32) * F32(sg * sx)).astype(F32)
    gx_u = (acc_x.astype(F32) * F32(sg * st)).astype(F32)
    gw = np.broadcast_to(gw_u[:, :, None, None], (Cout, Cin, KH, KW)).copy()
    gx = np.repeat(np.repeat(gx_u, r, axis=2), r, axis=3)[:, :, :H, :W].copy()
    return gw, gx
