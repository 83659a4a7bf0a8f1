"""The autograd wrapper: gradients that come out of loss.backward() are the filtered ones."""
import numpy as np
import pytest
import torch

import oracle
from paper_2301_00330_b200 import workloads
from parity_util import TOL, f64, relerr

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,r,groups", [("f32", 2, 1), ("bf16", 2, 1), ("f32", 4, 8), ("f32", 1, 1)])
def test_backward_through_autograd_matches_the_oracle(gf, dtype, r, groups):
    L = workloads.Layer("autograd", 0, 0, 3, 8, 16, 12, 12, 3, groups, r, dtype, "normal", 1.0)
    x, gy, w = workloads.make_inputs(L)
    xd = x.cuda().requires_grad_(True)
    wd = w.cuda().requires_grad_(True)
    y = gf.filtered_conv2d(xd, wd, r=r, groups=groups)
    assert y.shape == (L.N, L.C_out, L.H, L.W)
    y.backward(gy.cuda())
    torch.cuda.synchronize()
    stash_ref = oracle.stash_forward(f64(x), r)
    gw_ref, gx_ref = oracle.backward(f64(gy), stash_ref, f64(w), r, groups=groups)
    assert relerr(f64(xd.grad), gx_ref) <= TOL[dtype]
    # the wrapper hands g_W back in the weight's dtype: one more bf16 rounding for bf16 weights
    assert relerr(f64(wd.grad), gw_ref) <= (TOL[dtype] if dtype == "f32" else 2 * TOL[dtype])


def test_module_trains_one_step(gf):
    torch.manual_seed(0)
    m = gf.FilteredConv2d(8, 8, 3, r=2, device="cuda")
    x = torch.randn(2, 8, 16, 16, device="cuda")
    before = m.weight.detach().clone()
    opt = torch.optim.SGD(m.parameters(), lr=0.1)
    loss = m(x).square().mean()
    loss.backward()
    opt.step()
    assert torch.isfinite(m.weight).all() and not torch.equal(before, m.weight)
    assert m.bias.grad is not None


def test_strided_layer_through_autograd(gf):
    """A stride-2 layer: the output has half the resolution and the gradients are the strided
    filtered ones (oracle/gf_strided.py)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(3)
    x = torch.randn((2, 8, 16, 16), generator=g)
    w = torch.randn((16, 8, 3, 3), generator=g) * 0.2
    gy = torch.randn((2, 16, 8, 8), generator=g)
    xd, wd = x.cuda().requires_grad_(True), w.cuda().requires_grad_(True)
    y = gf.filtered_conv2d(xd, wd, r=2, stride=2)
    assert y.shape == (2, 16, 8, 8)
    assert torch.allclose(y.detach().cpu(), torch.nn.functional.conv2d(x, w, None, 2, 1), rtol=1e-3, atol=1e-3)
    y.backward(gy.cuda())
    torch.cuda.synchronize()
    gw_ref, gx_ref = oracle.strided_backward(f64(gy), oracle.strided_stash_forward(f64(x), 2, 2), f64(w), 2, 2)
    assert relerr(f64(xd.grad), gx_ref) <= TOL["f32"] and relerr(f64(wd.grad), gw_ref) <= TOL["f32"]
