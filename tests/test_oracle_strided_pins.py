"""Pins of the strided-convolution oracle (oracle/gf_strided.py).  The paper gives no formulas for
stride > 1 (parity unpinned by the paper); these tests pin the reading to what exact backpropagation
and the paper's table fix."""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle


def rng(seed):
    return np.random.default_rng(seed)


def autograd_backward(x, gy, theta, stride, groups, pad):
    xt = torch.from_numpy(x).requires_grad_(True)
    tt = torch.from_numpy(theta).requires_grad_(True)
    y = F.conv2d(xt, tt, None, stride, pad, 1, groups)
    assert tuple(y.shape) == gy.shape
    y.backward(torch.from_numpy(gy))
    return tt.grad.numpy(), xt.grad.numpy()


@pytest.mark.parametrize("N,Cin,Cout,H,W,K,s,G", [(2, 4, 6, 8, 8, 3, 2, 1), (1, 4, 4, 12, 8, 5, 2, 2), (2, 3, 5, 9, 9, 3, 3, 1),
                                                   (2, 6, 6, 8, 6, 3, 2, 6), (1, 2, 3, 8, 8, 1, 2, 1), (2, 4, 4, 7, 10, 3, 2, 1)])
def test_exact_strided_backward_equals_fp64_autograd(N, Cin, Cout, H, W, K, s, G):
    p = (K - 1) // 2
    x = rng(1).normal(size=(N, Cin, H, W))
    theta = rng(2).normal(size=(Cout, Cin // G, K, K))
    Hy, Wy = (H + 2 * p - K) // s + 1, (W + 2 * p - K) // s + 1
    gy = rng(3).normal(size=(N, Cout, Hy, Wy))
    gw, gx = oracle.exact_backward_strided(x, gy, theta, s, G, p)
    gw_ref, gx_ref = autograd_backward(x, gy, theta, s, G, p)
    assert np.allclose(gw, gw_ref, rtol=1e-11, atol=1e-11) and np.allclose(gx, gx_ref, rtol=1e-11, atol=1e-11)


def test_stride_one_reduces_to_the_paper_formulas():
    x, theta = rng(4).normal(size=(2, 6, 9, 10)), rng(5).normal(size=(4, 3, 3, 3))
    gy = rng(6).normal(size=(2, 4, 9, 10))
    for r in (2, 3):
        st = oracle.strided_stash_forward(x, r, 1)
        assert np.array_equal(st, oracle.stash_forward(x, r))
        gw, gx = oracle.strided_backward(gy, st, theta, r, 1, groups=2)
        gw_ref, gx_ref = oracle.backward(gy, st, theta, r, groups=2)
        assert np.allclose(gw, gw_ref, rtol=1e-13) and np.allclose(gx, gx_ref, rtol=1e-12, atol=1e-13)
    assert np.allclose(oracle.kernel_phase_sums(theta, 1)[0, 0], oracle.kernel_sum(theta), rtol=1e-13)


def test_phase_sums_partition_the_kernel():
    theta = rng(7).normal(size=(3, 2, 5, 5))
    for s in (2, 3):
        th = oracle.kernel_phase_sums(theta, s)
        assert np.allclose(th.sum(axis=(0, 1)), oracle.kernel_sum(theta), rtol=1e-12)   # every tap in exactly one phase
    th = oracle.kernel_phase_sums(rng(8).normal(size=(2, 2, 1, 1)), 2)                   # 1x1: only phase (0,0) is reached
    assert np.count_nonzero(th[0, 1]) == 0 and np.count_nonzero(th[1, 0]) == 0 and np.count_nonzero(th[1, 1]) == 0


@pytest.mark.parametrize("K,s,r,G", [(3, 2, 2, 1), (3, 2, 4, 1), (5, 2, 4, 2), (3, 3, 2, 1)])
def test_interior_pixels_equal_exact_input_gradient_of_the_expanded_map(K, s, r, G):
    """Wherever every output that a pixel of x reaches lies inside ONE patch of g_y (and inside the
    map, through every tap of the pixel's phase), the reduced g~_X is the exact input gradient of
    the piecewise-constant g~_y: the stride-s form of the paper's interior-pixel statement."""
    p = (K - 1) // 2
    N, Cin, Cout, Hy, Wy = 2, 4, 6, 3 * r + 1, 2 * r
    H, W = Hy * s, Wy * s
    theta = rng(10).normal(size=(Cout, Cin // G, K, K))
    gy = rng(11).normal(size=(N, Cout, Hy, Wy))
    gm = oracle.patch_mean(gy, r)
    g_tilde = oracle.expand(gm, Hy, Wy, r)
    _, gx_exact = oracle.exact_backward_strided(np.zeros((N, Cin, H, W)), g_tilde, theta, s, G, p, need_gw=False)
    stash = np.zeros((N, Cin, gm.shape[2], gm.shape[3]))
    _, gx = oracle.strided_backward(gy, stash, theta, r, s, G, need_gw=False)

    def interior(h, size_y):
        outs = [(h + p - u) // s for u in range(K) if (h + p - u) % s == 0]
        return all(0 <= i < size_y and i // r == h // (r * s) for i in outs)

    mask = np.array([[interior(h, Hy) and interior(w, Wy) for w in range(W)] for h in range(H)])
    assert mask.sum() >= 4 and (~mask).sum() >= 4
    assert np.allclose(gx[:, :, mask], gx_exact[:, :, mask], rtol=1e-11, atol=1e-12)
    assert not np.allclose(gx[:, :, ~mask], gx_exact[:, :, ~mask], rtol=1e-6, atol=1e-9)    # an approximation elsewhere


def test_one_by_one_kernels_are_exact_everywhere_for_gx():
    s, r = 2, 2
    theta = rng(12).normal(size=(5, 3, 1, 1))
    gy = rng(13).normal(size=(2, 5, 5, 6))
    g_tilde = oracle.expand(oracle.patch_mean(gy, r), 5, 6, r)
    _, gx_exact = oracle.exact_backward_strided(np.zeros((2, 3, 10, 12)), g_tilde, theta, s, 1, 0, need_gw=False)
    _, gx = oracle.strided_backward(gy, np.zeros((2, 3, 3, 3)), theta, r, s, need_gw=False)
    assert np.allclose(gx, gx_exact, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("K", [1, 3])
def test_gw_equals_exact_centre_tap_for_window_constant_x(K):
    """With x constant over every (r s) x (r s) window, replacing x by its window average loses
    nothing, and the tap that reads x at zero offset meets no boundary: g~_W equals the exact
    weight gradient of (x, expanded g~_y) at the centre tap.  Partial edge patches included."""
    s, r, p = 2, 2, (K - 1) // 2
    N, Cin, Cout, Hy, Wy = 2, 4, 6, 5, 7                     # partial patches on both axes
    H, W = Hy * s, Wy * s
    Hp, Wp = -(-Hy // r), -(-Wy // r)
    xc = rng(14).normal(size=(N, Cin, Hp, Wp))
    x = oracle.expand(xc, H, W, r * s)
    gy = rng(15).normal(size=(N, Cout, Hy, Wy))
    theta = rng(16).normal(size=(Cout, Cin // 2, K, K))
    g_tilde = oracle.expand(oracle.patch_mean(gy, r), Hy, Wy, r)
    gw_exact, _ = oracle.exact_backward_strided(x, g_tilde, theta, s, 2, p, need_gx=False)
    gw, _ = oracle.strided_backward(gy, oracle.strided_stash_forward(x, r, s), theta, r, s, 2, need_gx=False)
    assert np.allclose(gw[:, :, p, p], gw_exact[:, :, p, p], rtol=1e-11, atol=1e-12)
    assert np.allclose(gw, gw[:, :, :1, :1])                 # every tap carries the same value


def test_structure_of_the_strided_results():
    s, r = 2, 2
    theta = rng(17).normal(size=(4, 4, 3, 3))
    gy = rng(18).normal(size=(1, 4, 4, 4))
    _, gx = oracle.strided_backward(gy, np.zeros((1, 4, 2, 2)), theta, r, s, need_gw=False)
    win = gx.reshape(1, 4, 2, r * s, 2, r * s)
    assert np.allclose(win[:, :, :, :-s], win[:, :, :, s:], rtol=1e-13)         # period s inside every window
    assert np.allclose(win[:, :, :, :, :, :-s], win[:, :, :, :, :, s:], rtol=1e-13)
    # linear in g_y and in theta
    gy2 = rng(19).normal(size=gy.shape)
    _, a = oracle.strided_backward(gy + 2 * gy2, np.zeros((1, 4, 2, 2)), theta, r, s, need_gw=False)
    _, b = oracle.strided_backward(gy2, np.zeros((1, 4, 2, 2)), theta, r, s, need_gw=False)
    assert np.allclose(a, gx + 2 * b, rtol=1e-12, atol=1e-13)


def test_literal_loops_on_a_tiny_layer():
    """The definitions as pure-Python loops over pixels, output channels and taps."""
    s, r, K, p = 2, 2, 3, 1
    N, Cin, Cout, Hy, Wy = 1, 2, 3, 3, 2
    H, W = Hy * s, Wy * s
    x, gy = rng(20).normal(size=(N, Cin, H, W)), rng(21).normal(size=(N, Cout, Hy, Wy))
    theta = rng(22).normal(size=(Cout, Cin, K, K))
    gm = oracle.patch_mean(gy, r)
    stash = oracle.strided_stash_forward(x, r, s)
    gw, gx = oracle.strided_backward(gy, stash, theta, r, s)
    for n in range(N):
        for ci in range(Cin):
            for h in range(H):
                for w in range(W):
                    acc = 0.0
                    for co in range(Cout):
                        for u in range(K):
                            for v in range(K):
                                if (h + p - u) % s == 0 and (w + p - v) % s == 0:
                                    acc += theta[co, ci, u, v] * gm[n, co, h // (r * s), w // (r * s)]
                    assert gx[n, ci, h, w] == pytest.approx(acc, rel=1e-12, abs=1e-14)
    for co in range(Cout):
        for ci in range(Cin):
            acc = 0.0
            for n in range(N):
                for i in range(Hy):
                    for j in range(Wy):
                        a, b = i // r, j // r
                        h0, h1 = a * r * s, min((a + 1) * r * s, H)
                        w0, w1 = b * r * s, min((b + 1) * r * s, W)
                        acc += x[n, ci, h0:h1, w0:w1].mean() * gm[n, co, a, b]     # window average for the pixel the tap meets
            assert np.allclose(gw[co, ci], acc, rtol=1e-12)


def test_stash_grid_is_the_papers_table_row():
    """ImageNet table, ResNet-18 "4 layers": the stride-2 layer keeps its 14 x 14 x 256 input on the
    4 x 4 grid of its 7 x 7 g_y at r = 2: 256 * 16 values * 4 B = 16 KB of the row's 112 KB."""
    x = np.zeros((1, 256, 14, 14))
    stash = oracle.strided_stash_forward(x, 2, 2)
    assert stash.shape == (1, 256, 4, 4)
    path = os.path.join(os.path.dirname(__file__), "golden", "table_imagenet_mem.txt")
    row = [l for l in open(path) if l.split()[:2] == ["resnet18", "4"]]
    assert len(row) == 1 and row[0].split()[3] == "112.00"
    assert 3 * 32.0 + stash.size * 4 / 1024.0 == 112.0
