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


@pytest.mark.parametrize("groups,c_in,c_out", [(1, 16, 24), (16, 16, 16), (1, 12, 8)])
def test_channels_last_input_through_autograd(gf, groups, c_in, c_out):
    """An input in torch's channels_last format: the channels-last kernels where the library has them
    (the first two cases), a contiguous copy otherwise (12 channels); the gradients are the same
    filtered ones, and g_X comes back in the input's format when the channels-last kernels ran."""
    L = workloads.Layer("cl", 0, 0, 2, c_in, c_out, 12, 12, 3, groups, 2, "f32", "normal", 1.0)
    x, gy, w = workloads.make_inputs(L)
    xd = x.cuda().contiguous(memory_format=torch.channels_last).requires_grad_(True)
    wd = w.cuda().requires_grad_(True)
    launches = gf.gf_kernel_launch_count()
    y = gf.filtered_conv2d(xd, wd, r=2, groups=groups)
    y.backward(gy.cuda())
    torch.cuda.synchronize()
    assert gf.gf_kernel_launch_count() > launches
    stash_ref = oracle.stash_forward(f64(x), 2)
    gw_ref, gx_ref = oracle.backward(f64(gy), stash_ref, f64(w), 2, groups=groups)
    assert relerr(f64(xd.grad), gx_ref) <= TOL["f32"] and relerr(f64(wd.grad), gw_ref) <= TOL["f32"]
    if c_in % 8 == 0:
        assert xd.grad.is_contiguous(memory_format=torch.channels_last)
