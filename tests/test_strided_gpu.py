"""GPU parity of strided layers (stride 2 and 3; the reading of oracle/gf_strided.py -- the paper
writes its formulas for stride 1 only) against the fp64 CPU oracle on the same seeded inputs, element
by element, through the C ABI.  Tolerances as for stride 1: 1e-4 (fp32), 2e-2 (bf16 inputs)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2301_00330_b200 import workloads

from parity_util import TOL, Guarded, f64, relerr

pytestmark = pytest.mark.gpu

# (name, N, C_in, C_out, H, W, K, groups, r, stride)
CASES = [
    ("resnet18_downsample_3x3", 4, 64, 128, 28, 28, 3, 1, 2, 2),     # 14x14 g_y, 7x7 patches
    ("resnet18_last_stage_3x3", 3, 32, 64, 14, 14, 3, 1, 2, 2),      # 7x7 g_y: partial patches, the paper's table row
    ("shortcut_1x1", 3, 40, 72, 16, 16, 1, 1, 2, 2),
    ("mobilenet_dw_3x3", 2, 48, 48, 28, 28, 3, 48, 2, 2),            # depthwise, stride 2
    ("k5_r4", 2, 12, 20, 32, 32, 5, 1, 4, 2),
    ("grouped", 2, 16, 24, 16, 24, 3, 4, 2, 2),
    ("stride3", 2, 8, 12, 18, 27, 3, 1, 2, 3),
    ("r_not_dividing", 2, 8, 8, 20, 12, 3, 1, 3, 2),                 # 10x6 g_y with r = 3
    ("ragged_channels", 1, 70, 37, 8, 8, 3, 1, 2, 2),
]


def _inputs(N, Cin, Cout, H, W, K, G, stride, dtype, seed):
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    dt = workloads.torch_dtype(dtype)
    x = torch.randn((N, Cin, H, W), generator=g).clamp_(min=0.0).to(dt).contiguous()
    gy = (torch.randn((N, Cout, H // stride, W // stride), generator=g) * 1e-2).to(dt).contiguous()
    w = (torch.randn((Cout, Cin // G, K, K), generator=g) * (2.0 / (Cin // G * K * K)) ** 0.5).to(dt).contiguous()
    return x, gy, w


def _run(gf, desc, x, gy, w, dt, need_gw=True, need_gx=True):
    stash = Guarded(gf.gf_stash_dims(desc), dt)
    gf.gf_stash_forward(desc, x.cuda(), stash.t)
    gW = Guarded(tuple(w.shape), torch.float32)
    gX = Guarded(tuple(x.shape), dt)
    ws_bytes = gf.gf_backward_workspace_bytes(desc)
    ws = Guarded((ws_bytes,), torch.uint8)
    gf.gf_backward(desc, gy.cuda(), stash.t, w.cuda(), gW.t if need_gw else None, gX.t if need_gx else None, ws.t, ws_bytes)
    assert gf.gf_last_async_status(ws.t) == gf.GF_OK
    torch.cuda.synchronize()
    for b in (stash, gW, gX, ws):
        b.check()
    return stash.t, gW.t, gX.t


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("case", CASES, ids=lambda c: c[0])
def test_strided_layers_element_by_element(gf, case, dtype):
    name, N, Cin, Cout, H, W, K, G, r, stride = case
    x, gy, w = _inputs(N, Cin, Cout, H, W, K, G, stride, dtype, seed=len(name) * 31 + r)
    desc = gf.make_desc(N, Cin, Cout, H, W, K, r=r, groups=G, stride=stride, dtype=gf.GF_F32 if dtype == "f32" else gf.GF_BF16)
    stash_ref = oracle.strided_stash_forward(f64(x), r, stride)
    assert gf.gf_stash_dims(desc) == stash_ref.shape
    gw_ref, gx_ref = oracle.strided_backward(f64(gy), stash_ref, f64(w), r, stride, G)
    stash, gW, gX = _run(gf, desc, x, gy, w, workloads.torch_dtype(dtype))
    tol = TOL[dtype]
    assert relerr(f64(stash), stash_ref) <= tol
    assert relerr(f64(gW), gw_ref) <= tol
    assert relerr(f64(gX), gx_ref) <= tol
    # nullable outputs give the same values
    _, gW2, _ = _run(gf, desc, x, gy, w, workloads.torch_dtype(dtype), need_gx=False)
    _, _, gX2 = _run(gf, desc, x, gy, w, workloads.torch_dtype(dtype), need_gw=False)
    assert torch.equal(gX2, gX) and relerr(f64(gW2), f64(gW)) <= 1e-6


@pytest.mark.parametrize("case", [("exact_s2", 2, 8, 12, 12, 10, 3, 1, 1, 2), ("exact_s2_groups_k5", 2, 8, 8, 12, 12, 5, 2, 1, 2),
                                  ("exact_s3_1x1", 1, 6, 4, 9, 9, 1, 1, 1, 3)], ids=lambda c: c[0])
def test_patch_size_one_is_exact_strided_backward(gf, case):
    name, N, Cin, Cout, H, W, K, G, r, stride = case
    x, gy, w = _inputs(N, Cin, Cout, H, W, K, G, stride, "f32", seed=77)
    desc = gf.make_desc(N, Cin, Cout, H, W, K, r=1, groups=G, stride=stride)
    gw_ref, gx_ref = oracle.exact_backward_strided(f64(x), f64(gy), f64(w), stride, G, (K - 1) // 2)
    stash, gW, gX = _run(gf, desc, x, gy, w, torch.float32)
    assert torch.equal(stash.cpu(), x)
    assert relerr(f64(gW), gw_ref) <= TOL["f32"] and relerr(f64(gX), gx_ref) <= TOL["f32"]


def test_strided_exact_arithmetic_bit_for_bit(gf):
    """Integer-valued inputs for which every intermediate is an exactly representable integer."""
    N, Cin, Cout, H, W, K, r, stride = 3, 24, 40, 16, 16, 3, 2, 2
    g = torch.Generator(device="cpu")
    g.manual_seed(11)
    x = torch.randint(0, 4, (N, Cin, H, W), generator=g).float()
    gbar = torch.randint(-3, 4, (N, Cout, H // stride // r, W // stride // r), generator=g).float() * 4.0   # g_W carries 1/4
    gy = gbar.repeat_interleave(r, 2).repeat_interleave(r, 3).contiguous()
    w = torch.randint(-1, 2, (Cout, Cin, K, K), generator=g).float()
    desc = gf.make_desc(N, Cin, Cout, H, W, K, r=r, stride=stride)
    stash_ref = oracle.strided_stash_forward(f64(x), r, stride)
    gw_ref, gx_ref = oracle.strided_backward(f64(gy), stash_ref, f64(w), r, stride)
    stash, gW, gX = _run(gf, desc, x, gy, w, torch.float32)
    assert np.array_equal(f64(stash), stash_ref) and np.array_equal(f64(gW), gw_ref) and np.array_equal(f64(gX), gx_ref)


def test_unsupported_strided_geometry_is_refused(gf):
    import ctypes
    size = ctypes.c_size_t(0)
    odd = gf.make_desc(1, 4, 4, 15, 16, 3, r=2, stride=2)             # stride does not divide H
    assert gf.lib().gf_backward_workspace_bytes(ctypes.byref(odd), ctypes.byref(size)) == gf.GF_ERR_UNSUPPORTED
