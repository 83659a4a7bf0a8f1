"""Pins of the INT8 oracle (oracle/gf_int8.py; the supplement's section on combining gradient
filtering with gradient quantization).  The paper gives no formulas for the quantizer; these tests
pin the chosen one (per-tensor symmetric, round to nearest even) to its definition and tie the
integer contractions to the pinned fp64 oracle of the method."""
import struct

import numpy as np
import pytest

import oracle
from oracle import int8


def rng(seed):
    return np.random.default_rng(seed)


def test_quantizer_against_scalar_definition():
    t = rng(0).normal(size=(3, 5, 7)).astype(np.float32)
    codes, scale = int8.quantize(t)
    amax = max(abs(float(v)) for v in t.ravel())
    f32 = lambda v: struct.unpack("f", struct.pack("f", v))[0]          # round a Python float to fp32
    s = f32(f32(amax) / 127.0)
    assert float(scale) == s
    for v, c in zip(t.ravel(), codes.ravel()):
        q = f32(float(v) / s)                                           # fp32 quotient
        lo = np.floor(q)
        ref = lo if q - lo < 0.5 else lo + 1 if q - lo > 0.5 else (lo if lo % 2 == 0 else lo + 1)
        assert int(c) == int(max(-127, min(127, ref)))
    assert codes.dtype == np.int8 and codes.min() >= -127 and codes.max() <= 127
    assert abs(int(codes.ravel()[np.argmax(np.abs(t))])) == 127        # the extreme value maps to the extreme code
    assert np.abs(int8.dequantize(codes, scale) - t).max() <= 0.5 * float(scale) * (1 + 1e-6)


def test_quantizer_special_cases():
    z, s = int8.quantize(np.zeros((2, 3)))
    assert float(s) == 1.0 and not z.any()
    grid = np.arange(-127, 128, dtype=np.float32).reshape(5, 51)       # already on the grid: scale 1, codes = values
    c, s = int8.quantize(grid)
    assert float(s) == 1.0 and np.array_equal(c.astype(np.float32), grid)
    c2, s2 = int8.quantize(grid * np.float32(0.25))                    # power-of-two rescaling moves only the scale
    assert float(s2) == 0.25 and np.array_equal(c2, c)
    half = np.array([127.0, 0.5, 1.5, 2.5, -0.5, -1.5], dtype=np.float32)
    assert list(int8.quantize(half)[0]) == [127, 0, 2, 2, 0, -2]       # ties go to the even code


def test_fp32_patch_mean_and_kernel_sum_follow_the_fp64_oracle():
    g = rng(1).normal(size=(2, 3, 7, 10)).astype(np.float32)
    for r in (2, 3, 4):
        got = int8.patch_mean_f32(g, r)
        assert got.dtype == np.float32
        assert np.allclose(got, oracle.patch_mean(g, r), rtol=1e-6, atol=1e-7)
    # the stated order, element by element, on one partial patch
    r = 4
    blk = g[1, 2, 4:7, 8:10]
    acc = np.float32(0)
    for i in range(blk.shape[0]):
        for j in range(blk.shape[1]):
            acc = np.float32(acc + blk[i, j])
    assert int8.patch_mean_f32(g, r)[1, 2, 1, 2] == np.float32(acc * np.float32(np.float32(1.0) / np.float32(6.0)))
    th = rng(2).normal(size=(4, 3, 3, 3)).astype(np.float32)
    assert np.allclose(int8.kernel_sum_f32(th), oracle.kernel_sum(th), rtol=1e-6, atol=1e-7)


@pytest.mark.parametrize("shape", [(2, 6, 4, 8, 8, 3, 2), (3, 5, 7, 7, 9, 3, 2), (2, 8, 8, 12, 12, 1, 4)])
def test_int8_backward_is_the_method_on_the_dequantised_operands(shape):
    """The integer contractions times the scales are Eq. (grad_w) and Eq. (grad_x) of the pinned
    fp64 oracle applied to the dequantised stash, patch means and kernel sums."""
    N, Cin, Cout, H, W, K, r = shape
    x = np.maximum(rng(3).normal(size=(N, Cin, H, W)), 0).astype(np.float32)
    gy = (rng(4).normal(size=(N, Cout, H, W)) * 1e-2).astype(np.float32)
    theta = (rng(5).normal(size=(Cout, Cin, K, K)) * 0.2).astype(np.float32)
    stash = oracle.stash_forward(x, r).astype(np.float32)
    gw, gx = int8.int8_backward(gy, stash, theta, r)
    qg, sg = int8.quantize(int8.patch_mean_f32(gy, r))
    qx, sx = int8.quantize(stash)
    qt, st = int8.quantize(int8.kernel_sum_f32(theta))
    gw_ref = oracle.reduced_gw(int8.dequantize(qx, sx), int8.dequantize(qg, sg), 1, K, K)
    gx_ref = oracle.reduced_gx(int8.dequantize(qg, sg), int8.dequantize(qt, st), 1, H, W, r)
    assert np.allclose(gw, gw_ref, rtol=3e-7, atol=1e-12)              # three fp32 roundings of the scaling
    assert np.allclose(gx, gx_ref, rtol=3e-7, atol=1e-12)
    assert np.array_equal(gw, np.broadcast_to(gw[:, :, :1, :1], gw.shape))
    # and close to the unquantised method: error of a few codes' worth
    gw_fp, gx_fp = oracle.backward(gy, stash, theta, r)
    assert np.abs(gw - gw_fp).max() <= 0.05 * np.abs(gw_fp).max()
    assert np.abs(gx - gx_fp).max() <= 0.05 * np.abs(gx_fp).max()


def test_int8_backward_is_exact_on_integer_grids():
    """Operands already on the INT8 grid with extreme value 127 (scales exactly 1): nothing is lost,
    the INT8 path gives the unquantised method's result exactly."""
    r, K = 2, 3
    x = rng(6).integers(0, 32, size=(2, 4, 8, 8)).astype(np.float32)
    x[0, 0, :2, :2] = [[32, 32], [32, 31]]                             # one patch sums to 127
    gbar = rng(7).integers(-127, 128, size=(2, 6, 4, 4)).astype(np.float32)
    gbar[0, 0, 0, 0] = 127.0
    gy = np.repeat(np.repeat(gbar, r, 2), r, 3)
    theta = rng(8).integers(-14, 15, size=(6, 4, K, K)).astype(np.float32)
    theta[0, 0] = 14.0
    theta[0, 0, 0, 0] = 15.0                                           # kernel sum of pair (0, 0): 127
    stash = oracle.stash_forward(x, r).astype(np.float32)
    assert np.abs(stash).max() == 127.0 and np.abs(int8.kernel_sum_f32(theta)).max() == 127.0
    gw, gx = int8.int8_backward(gy, stash, theta, r)
    gw_fp, gx_fp = oracle.backward(gy, stash, theta, r)
    assert np.abs(gw_fp).max() < 2 ** 24 and np.abs(gx_fp).max() < 2 ** 24
    assert np.array_equal(gw, gw_fp.astype(np.float32)) and np.array_equal(gx, gx_fp.astype(np.float32))
