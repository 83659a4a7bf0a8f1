"""Pins for the fp64 CPU oracle: it is checked against what the paper and the
mathematics fix, never against itself.

  P1  exact backward == autograd of a library fp64 convolution; r == 1 is that
  P2  centre-tap identity for g_W (exact weight gradient of the expanded g~_y)
  P3  interior-pixel identity for g_X (kernel footprint inside one patch)
  P4  1x1 kernels: both reduced formulas equal exact BP on the expanded g~_y
  P5  the supplement's literal padded-patch loops == the reduced formulas
  P6  stash size == "Mem" column of the paper's ImageNet table
  P7  structural invariants
  P8  an independent tensor-op restatement + brute force on tiny inputs
"""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle

RTOL = 1e-11


def rel(a, b):
    a, b = np.asarray(a), np.asarray(b)
    den = np.abs(b).max()
    return np.abs(a - b).max() / (den if den > 0 else 1.0)


def rnd(rng, *shape):
    return rng.standard_normal(shape)


def torch_exact(x, gy, w, groups, pad):
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    wt = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    y = F.conv2d(xt, wt, None, stride=1, padding=pad, groups=groups)
    y.backward(torch.tensor(gy, dtype=torch.float64))
    return wt.grad.numpy(), xt.grad.numpy()


# ------------------------------------------------------------------ P1
@pytest.mark.parametrize("N,Cin,Cout,G,H,W,K,pad", [
    (2, 4, 6, 1, 7, 5, 3, 1),
    (1, 6, 4, 2, 6, 8, 3, 1),
    (2, 4, 4, 4, 5, 5, 3, 1),       # depthwise
    (2, 3, 5, 1, 6, 4, 1, 0),
    (1, 2, 3, 1, 9, 7, 5, 2),
    (1, 2, 2, 1, 6, 6, 3, 0),       # "valid" padding, H_y != H
    (1, 2, 2, 1, 5, 7, (3, 1), (1, 0)),
])
def test_p1_exact_backward_matches_library_autograd(N, Cin, Cout, G, H, W, K, pad):
    rng = np.random.default_rng(11)
    KH, KW = (K, K) if isinstance(K, int) else K
    ph, pw = (pad, pad) if isinstance(pad, int) else pad
    x = rnd(rng, N, Cin, H, W)
    w = rnd(rng, Cout, Cin // G, KH, KW)
    gy = rnd(rng, N, Cout, H + 2 * ph - KH + 1, W + 2 * pw - KW + 1)
    gw, gx = oracle.exact_backward(x, gy, w, G, (ph, pw))
    gw_t, gx_t = torch_exact(x, gy, w, G, (ph, pw))
    assert rel(gw, gw_t) < RTOL and rel(gx, gx_t) < RTOL


def test_p1_r1_is_exact_backprop():
    rng = np.random.default_rng(12)
    x, w, gy = rnd(rng, 2, 4, 6, 6), rnd(rng, 6, 2, 3, 3), rnd(rng, 2, 6, 6, 6)
    stash = oracle.stash_forward(x, 1)
    assert np.array_equal(stash, x)
    gw, gx = oracle.backward(gy, stash, w, 1, groups=2)
    gw_t, gx_t = torch_exact(x, gy, w, 2, 1)
    assert rel(gw, gw_t) < RTOL and rel(gx, gx_t) < RTOL


def test_p1_reduced_formulas_at_r1_equal_exact_for_1x1_kernels():
    rng = np.random.default_rng(13)
    x, w, gy = rnd(rng, 2, 6, 5, 4), rnd(rng, 4, 3, 1, 1), rnd(rng, 2, 4, 5, 4)
    gm = oracle.patch_mean(gy, 1)
    gw = oracle.reduced_gw(oracle.patch_sum(x, 1), gm, 2, 1, 1)
    gx = oracle.reduced_gx(gm, oracle.kernel_sum(w), 2, 5, 4, 1)
    gw_t, gx_t = torch_exact(x, gy, w, 2, 0)
    assert rel(gw, gw_t) < RTOL and rel(gx, gx_t) < RTOL


# ------------------------------------------------------------------ P2
@pytest.mark.parametrize("H,W,r,K,G", [
    (8, 8, 2, 3, 1), (7, 9, 2, 3, 1), (10, 6, 4, 3, 2), (9, 9, 7, 5, 1),
    (5, 5, 8, 3, 1), (6, 6, 3, 3, 4), (12, 8, 4, 1, 1),
])
def test_p2_centre_tap_of_gw_is_exact_on_expanded_gradient(H, W, r, K, G):
    rng = np.random.default_rng(21)
    N, Cin, Cout = 2, 4, 8
    x, w, gy = rnd(rng, N, Cin, H, W), rnd(rng, Cout, Cin // G, K, K), rnd(rng, N, Cout, H, W)
    gw, _ = oracle.backward(gy, oracle.stash_forward(x, r), w, r, groups=G, need_gx=False)
    gy_tilde = oracle.expand(oracle.patch_mean(gy, r), H, W, r)
    gw_exact, _ = torch_exact(x, gy_tilde, w, G, (K - 1) // 2)
    c = (K - 1) // 2
    assert rel(gw[:, :, c, c], gw_exact[:, :, c, c]) < RTOL
    # every tap carries that same value (Eq. (grad_w) has no u, v on the right)
    assert np.array_equal(gw, np.broadcast_to(gw[:, :, c:c + 1, c:c + 1], gw.shape))


# ------------------------------------------------------------------ P3
@pytest.mark.parametrize("H,W,r,K", [(12, 9, 3, 3), (8, 8, 4, 3), (14, 14, 7, 3), (14, 10, 7, 5),
                                     (10, 11, 4, 3)])
def test_p3_gx_is_exact_where_the_kernel_stays_inside_one_patch(H, W, r, K):
    rng = np.random.default_rng(31)
    N, Cin, Cout = 2, 3, 5
    x, w, gy = rnd(rng, N, Cin, H, W), rnd(rng, Cout, Cin, K, K), rnd(rng, N, Cout, H, W)
    _, gx = oracle.backward(gy, oracle.stash_forward(x, r), w, r, need_gw=False)
    gy_tilde = oracle.expand(oracle.patch_mean(gy, r), H, W, r)
    _, gx_exact = torch_exact(x, gy_tilde, w, 1, (K - 1) // 2)
    c = (K - 1) // 2
    checked = 0
    for h in range(H):
        for ww in range(W):
            # footprint [h-c, h+c] x [w-c, w+c] inside the patch AND inside the image
            inside_h = (h % r) - c >= 0 and (h % r) + c <= min(r, H - (h // r) * r) - 1
            inside_w = (ww % r) - c >= 0 and (ww % r) + c <= min(r, W - (ww // r) * r) - 1
            if inside_h and inside_w:
                assert rel(gx[:, :, h, ww], gx_exact[:, :, h, ww]) < RTOL
                checked += 1
    assert checked > 0
    # and it is NOT exact on patch borders (the approximation is real)
    assert rel(gx, gx_exact) > 1e-3


# ------------------------------------------------------------------ P4
@pytest.mark.parametrize("H,W,r,Cin,Cout,G", [
    (8, 8, 2, 6, 4, 1), (7, 5, 2, 4, 6, 2), (9, 10, 4, 3, 3, 3), (6, 6, 8, 5, 2, 1), (7, 7, 7, 2, 4, 1),
])
def test_p4_1x1_kernels_reduced_equals_exact_on_expanded_gradient(H, W, r, Cin, Cout, G):
    rng = np.random.default_rng(41)
    N = 3
    x, w, gy = rnd(rng, N, Cin, H, W), rnd(rng, Cout, Cin // G, 1, 1), rnd(rng, N, Cout, H, W)
    gw, gx = oracle.backward(gy, oracle.stash_forward(x, r), w, r, groups=G)
    gy_tilde = oracle.expand(oracle.patch_mean(gy, r), H, W, r)
    gw_exact, gx_exact = torch_exact(x, gy_tilde, w, G, 0)
    assert rel(gw, gw_exact) < RTOL and rel(gx, gx_exact) < RTOL


# ------------------------------------------------------------------ P5
@pytest.mark.parametrize("H,W,r,K,G", [(8, 8, 2, 3, 1), (7, 9, 4, 3, 2), (6, 5, 3, 5, 1), (5, 5, 2, 1, 4)])
def test_p5_literal_padded_patch_loops_equal_reduced_formulas(H, W, r, K, G):
    rng = np.random.default_rng(51)
    N, Cin, Cout = 2, 4, 8
    x, w, gy = rnd(rng, N, Cin, H, W), rnd(rng, Cout, Cin // G, K, K), rnd(rng, N, Cout, H, W)
    gw, gx = oracle.backward(gy, oracle.stash_forward(x, r), w, r, groups=G)
    gw_l, gx_l = oracle.literal_backward(x, gy, w, r, groups=G)
    assert rel(gw, gw_l) < RTOL and rel(gx, gx_l) < RTOL


# ------------------------------------------------------------------ P6
def _golden_rows():
    path = os.path.join(os.path.dirname(__file__), "golden", "table_imagenet_mem.txt")
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, layers = line.split("|")
        model, k, vanilla, ours = head.split()
        shapes = [tuple(int(t) for t in lay.split(",")) for lay in layers.split(";")]
        yield model, int(k), float(vanilla), float(ours), shapes


@pytest.mark.parametrize("model,k,vanilla_kb,ours_kb,shapes", list(_golden_rows()))
def test_p6_stash_size_matches_the_papers_mem_column(model, k, vanilla_kb, ours_kb, shapes):
    assert len(shapes) == k
    vanilla = sum(c * hx * wx for c, hx, wx, _, _ in shapes) * 4 / 1024
    ours = sum(oracle.stash_num_values(c, hy, wy, 2) for c, _, _, hy, wy in shapes) * 4 / 1024
    assert abs(vanilla - vanilla_kb) < 0.005
    assert abs(ours - ours_kb) < 0.005
    # the produced array has that many values
    c, hx, wx, hy, wy = shapes[-1]
    if (hx, wx) == (hy, wy):
        assert oracle.stash_forward(np.zeros((1, c, hx, wx)), 2).size == oracle.stash_num_values(c, hy, wy, 2)


# ------------------------------------------------------------------ P7
def test_p7_structural_invariants():
    rng = np.random.default_rng(71)
    N, Cin, Cout, H, W, r, K = 2, 4, 6, 10, 7, 4, 3
    x, w, gy = rnd(rng, N, Cin, H, W), rnd(rng, Cout, Cin, K, K), rnd(rng, N, Cout, H, W)
    gm = oracle.patch_mean(gy, r)
    gw, gx = oracle.backward(gy, oracle.stash_forward(x, r), w, r)
    # (ii) g_X is constant on every patch
    assert np.array_equal(gx, oracle.expand(gx[:, :, ::r, ::r], H, W, r))
    # (iii) the filter leaves a patch-constant map unchanged, partial patches included
    pc = oracle.expand(rnd(rng, N, Cout, *oracle.grid(H, W, r)), H, W, r)
    assert rel(oracle.expand(oracle.patch_mean(pc, r), H, W, r), pc) < 1e-15
    # (v) mass: the filtered map has the same sum as g_y, per channel
    assert rel(oracle.expand(gm, H, W, r).sum((2, 3)), gy.sum((2, 3))) < 1e-12
    # the stash is a sum: total mass of x is kept
    assert rel(oracle.patch_sum(x, r).sum((2, 3)), x.sum((2, 3))) < 1e-12
    # (iv) linearity in g_y, x and theta
    gy2, x2, w2 = rnd(rng, *gy.shape), rnd(rng, *x.shape), rnd(rng, *w.shape)
    gw_b, gx_b = oracle.backward(2 * gy - 3 * gy2, oracle.stash_forward(x, r), w, r)
    gw_2, gx_2 = oracle.backward(gy2, oracle.stash_forward(x, r), w, r)
    assert rel(gw_b, 2 * gw - 3 * gw_2) < 1e-12 and rel(gx_b, 2 * gx - 3 * gx_2) < 1e-12
    gw_x, _ = oracle.backward(gy, oracle.stash_forward(x + 5 * x2, r), w, r)
    gw_x2, _ = oracle.backward(gy, oracle.stash_forward(x2, r), w, r)
    assert rel(gw_x, gw + 5 * gw_x2) < 1e-12
    _, gx_w = oracle.backward(gy, oracle.stash_forward(x, r), w - w2, r)
    _, gx_w2 = oracle.backward(gy, oracle.stash_forward(x, r), w2, r)
    assert rel(gx_w, gx - gx_w2) < 1e-12


def test_p7_one_patch_per_map_is_the_minimum_computation_case():
    rng = np.random.default_rng(72)
    N, Cin, Cout, H, W, K = 2, 3, 4, 5, 6, 3
    x, w, gy = rnd(rng, N, Cin, H, W), rnd(rng, Cout, Cin, K, K), rnd(rng, N, Cout, H, W)
    for r in (6, 9):
        gw, gx = oracle.backward(gy, oracle.stash_forward(x, r), w, r)
        gbar = gy.mean((2, 3))                      # one value per channel
        want_gx = np.einsum("no,oi->ni", gbar, w.sum((2, 3)))[:, :, None, None]
        assert rel(gx, np.broadcast_to(want_gx, gx.shape)) < RTOL
        want_gw = np.einsum("no,ni->oi", gbar, x.sum((2, 3)))[:, :, None, None]
        assert rel(gw, np.broadcast_to(want_gw, gw.shape)) < RTOL


# ------------------------------------------------------------------ P8
def _pool_torch(t, r, mean):
    """Patch sum / mean with tensor ops: zero-pad to a multiple of r, view as
    [N,C,Hp,r,Wp,r], masked sum and count."""
    N, C, H, W = t.shape
    Hp, Wp = -(-H // r), -(-W // r)
    tp = F.pad(t, (0, Wp * r - W, 0, Hp * r - H))
    ones = F.pad(torch.ones(1, 1, H, W, dtype=t.dtype), (0, Wp * r - W, 0, Hp * r - H))
    s = tp.view(N, C, Hp, r, Wp, r).sum((3, 5))
    cnt = ones.view(1, 1, Hp, r, Wp, r).sum((3, 5))
    return s / cnt if mean else s


@pytest.mark.parametrize("H,W,r,K,G", [(8, 8, 2, 3, 1), (7, 9, 2, 3, 2), (10, 6, 4, 3, 1), (9, 9, 7, 5, 1),
                                       (5, 5, 8, 3, 4), (28, 28, 4, 1, 1)])
def test_p8_tensor_op_restatement(H, W, r, K, G):
    rng = np.random.default_rng(81)
    N, Cin, Cout = 2, 4, 8
    x, w, gy = rnd(rng, N, Cin, H, W), rnd(rng, Cout, Cin // G, K, K), rnd(rng, N, Cout, H, W)
    xt, wt, gt = (torch.tensor(a, dtype=torch.float64) for a in (x, w, gy))
    xs, gm = _pool_torch(xt, r, False), _pool_torch(gt, r, True)
    assert rel(oracle.patch_sum(x, r), xs.numpy()) < RTOL
    assert rel(oracle.patch_mean(gy, r), gm.numpy()) < RTOL
    if H % r == 0 and W % r == 0:   # library pooling on full patches
        assert rel(oracle.patch_mean(gy, r), F.avg_pool2d(gt, r).numpy()) < RTOL
        assert rel(oracle.patch_sum(x, r), (F.avg_pool2d(xt, r) * r * r).numpy()) < RTOL
    ts = wt.sum((2, 3))
    Hp, Wp = xs.shape[2:]
    gw_t = torch.einsum("ngiab,ngoab->goi", xs.view(N, G, Cin // G, Hp, Wp),
                        gm.view(N, G, Cout // G, Hp, Wp)).reshape(Cout, Cin // G)
    gx_u = torch.einsum("ngoab,goi->ngiab", gm.view(N, G, Cout // G, Hp, Wp),
                        ts.view(G, Cout // G, Cin // G)).reshape(N, Cin, Hp, Wp)
    gx_t = gx_u.repeat_interleave(r, 2).repeat_interleave(r, 3)[:, :, :H, :W]
    gw, gx = oracle.backward(gy, oracle.stash_forward(x, r), w, r, groups=G)
    assert rel(gw, gw_t[:, :, None, None].expand(-1, -1, K, K).numpy()) < RTOL
    assert rel(gx, gx_t.numpy()) < RTOL


def test_p8_brute_force_python_loops_on_a_tiny_case():
    rng = np.random.default_rng(82)
    N, Cin, Cout, H, W, r, K, G = 1, 2, 2, 5, 3, 2, 3, 1
    x, w, gy = rnd(rng, N, Cin, H, W), rnd(rng, Cout, Cin, K, K), rnd(rng, N, Cout, H, W)
    Hp, Wp = 3, 2
    xs = np.zeros((N, Cin, Hp, Wp))
    gs = np.zeros((N, Cout, Hp, Wp))
    cnt = np.zeros((Hp, Wp))
    for h in range(H):
        for ww in range(W):
            cnt[h // r, ww // r] += 1
            xs[:, :, h // r, ww // r] += x[:, :, h, ww]
            gs[:, :, h // r, ww // r] += gy[:, :, h, ww]
    gm = gs / cnt
    assert rel(oracle.patch_sum(x, r), xs) < RTOL and rel(oracle.patch_mean(gy, r), gm) < RTOL
    gw, gx = oracle.backward(gy, xs, w, r)
    for co in range(Cout):
        for ci in range(Cin):
            want = sum(xs[0, ci, a, b] * gm[0, co, a, b] for a in range(Hp) for b in range(Wp))
            for u in range(K):
                for v in range(K):
                    assert abs(gw[co, ci, u, v] - want) < 1e-12
    for ci in range(Cin):
        for h in range(H):
            for ww in range(W):
                want = sum(gm[0, co, h // r, ww // r] * w[co, ci].sum() for co in range(Cout))
                assert abs(gx[0, ci, h, ww] - want) < 1e-12


def test_kernel_sum_ignores_rotation():
    rng = np.random.default_rng(83)
    w = rnd(rng, 3, 2, 3, 3)
    assert rel(oracle.kernel_sum(w), oracle.kernel_sum(w[:, :, ::-1, ::-1])) < 1e-15
    assert rel(oracle.kernel_sum(w), w.sum((2, 3))) < 1e-15


# ---- activation + stash (forward-side step fused into the producer of x, Section 4.2) ----

def test_activation_definitions_and_library_clip():
    z = np.array([-7.5, -0.0, 0.0, 0.25, 5.999, 6.0, 6.5, 100.0]).reshape(1, 1, 2, 4)
    assert np.array_equal(oracle.activation(z, "none"), z)
    assert np.array_equal(oracle.activation(z, "relu").ravel(), [0, 0, 0, 0.25, 5.999, 6.0, 6.5, 100.0])
    assert np.array_equal(oracle.activation(z, "relu6").ravel(), [0, 0, 0, 0.25, 5.999, 6.0, 6.0, 6.0])
    big = np.random.default_rng(3).normal(scale=4.0, size=(2, 3, 5, 7))
    for kind in ("none", "relu", "relu6"):
        assert np.array_equal(oracle.activation(big, kind), oracle.activation_fast(big, kind))
    assert np.array_equal(oracle.activation_fast(big, "relu"), torch.relu(torch.from_numpy(big)).numpy())
    assert np.array_equal(oracle.activation_fast(big, "relu6"), torch.nn.functional.relu6(torch.from_numpy(big)).numpy())
    with pytest.raises(ValueError):
        oracle.activation(z, "gelu")


def test_act_stash_forward_is_the_stash_of_the_activated_map():
    z = np.random.default_rng(8).normal(scale=3.0, size=(2, 3, 7, 9))
    for r in (1, 2, 4):
        x, stash = oracle.act_stash_forward(z, "relu6", r)
        assert np.array_equal(x, np.clip(z, 0, 6))
        assert np.array_equal(stash, oracle.stash_forward(np.clip(z, 0, 6), r))
        if r > 1:   # mass: the stash keeps the sum of the activated map
            assert stash.sum() == pytest.approx(np.clip(z, 0, 6).sum(), rel=1e-12)
