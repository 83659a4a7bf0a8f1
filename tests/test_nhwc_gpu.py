"""GPU parity of the channels-last (NHWC) layout: x, g_y, the stash and g_X with the channels
innermost, W and g_W as always.  The oracle knows one layout only; its NCHW results are permuted.
The method (Sections 3.3 and 3.4, Eq. (grad_x) and Eq. (grad_w)) does not depend on the layout, so
the same bounds hold as for NCHW."""
import numpy as np
import pytest
import torch

import oracle
from paper_2301_00330_b200 import workloads
from paper_2301_00330_b200.workloads import Layer

from parity_util import TOL, Guarded, check_layer_sampled, f64, relerr

pytestmark = pytest.mark.gpu


def L(name, N, Cin, Cout, H, W, K, G, r, dtype="f32"):
    return Layer(name, 0, 0, N, Cin, Cout, H, W, K, G, r, dtype, "relu", 1e-2)


def nhwc(t: torch.Tensor) -> torch.Tensor:
    return t.permute(0, 2, 3, 1).contiguous()


def nchw_of(t: torch.Tensor) -> torch.Tensor:
    return t.permute(0, 3, 1, 2).contiguous()


def run_nhwc(gf, layer, x, gy, w, need_gw=True, need_gx=True, stash_in=None):
    """stash, g_W, g_X of the layer through the channels-last path, returned in NCHW order."""
    desc = gf.make_desc(layer.N, layer.C_in, layer.C_out, layer.H, layer.W, layer.K, r=layer.r, groups=layer.groups,
                        dtype=gf.GF_F32 if layer.dtype == "f32" else gf.GF_BF16, layout=gf.GF_NHWC)
    dt = workloads.torch_dtype(layer.dtype)
    n, c, hp, wp = gf.gf_stash_dims(desc)
    assert (n, c, hp, wp) == (layer.N, layer.C_in, layer.Hp, layer.Wp)
    stash = Guarded((n, hp, wp, c), dt)
    if stash_in is None:
        gf.gf_stash_forward(desc, nhwc(x).cuda(), stash.t)
    else:
        stash.t.copy_(nhwc(stash_in))
    gW = Guarded((layer.C_out, layer.C_ig, layer.K, layer.K), torch.float32)
    gX = Guarded((layer.N, layer.H, layer.W, layer.C_in), dt)
    ws_bytes = gf.gf_backward_workspace_bytes(desc)
    ws = Guarded((ws_bytes,), torch.uint8)
    gf.gf_backward(desc, nhwc(gy).cuda(), stash.t, w.cuda(), gW.t if need_gw else None, gX.t if need_gx else None,
                   ws.t, ws_bytes)
    assert gf.gf_last_async_status(ws.t) == gf.GF_OK
    torch.cuda.synchronize()
    for g in (stash, gW, gX, ws):
        g.check()
    return nchw_of(stash.t), gW.t, nchw_of(gX.t)


CASES = [
    L("one_tile", 2, 16, 24, 12, 12, 3, 1, 2),
    L("partial_patches_r4", 3, 24, 40, 14, 14, 3, 1, 4),
    L("odd_map_7x7", 2, 8, 8, 7, 7, 3, 1, 2),
    L("ragged_channel_tiles", 2, 72, 136, 9, 11, 3, 1, 2),
    L("ragged_channels_1x1", 2, 136, 72, 12, 20, 1, 1, 4),
    L("many_row_tiles", 5, 40, 48, 30, 30, 1, 1, 2),            # 1125 patches: nine row tiles, the last ragged
    L("wide_c_in", 3, 520, 64, 16, 16, 1, 1, 2),                # several c_i tiles in both contractions
    L("wide_c_out", 3, 40, 1032, 16, 16, 1, 1, 2),              # a long g_X contraction, ragged last chunk
    L("r7", 2, 16, 24, 32, 32, 3, 1, 7),
    L("r_gt_H", 1, 8, 8, 5, 5, 1, 1, 8),
    L("long_contraction", 40, 24, 16, 28, 28, 3, 1, 2),         # 7840 patches: the g_W split over the patches
    L("dw_r2", 2, 16, 16, 28, 28, 3, 16, 2),
    L("dw_r4_partial", 3, 24, 24, 14, 14, 3, 24, 4),
    L("dw_odd_c8", 2, 72, 72, 9, 7, 3, 72, 2),                  # 9 channel groups: not a divisor of the block size
    L("dw_k5", 2, 8, 8, 16, 48, 5, 8, 4),
]


@pytest.mark.parametrize("layer", CASES, ids=lambda l: l.name)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_nhwc_element_by_element(gf, layer, dtype):
    layer = layer.with_(dtype=dtype)
    x, gy, w = workloads.make_inputs(layer)
    tol = TOL[dtype]
    stash_ref = oracle.stash_forward(f64(x), layer.r)
    gw_ref, gx_ref = oracle.backward(f64(gy), stash_ref, f64(w), layer.r, groups=layer.groups)
    stash, gW, gX = run_nhwc(gf, layer, x, gy, w)
    errs = {"stash": relerr(f64(stash), stash_ref), "gW": relerr(f64(gW), gw_ref), "gX": relerr(f64(gX), gx_ref)}
    # the backward alone, on the oracle's stash rounded to the dtype
    st_round = torch.from_numpy(stash_ref).to(workloads.torch_dtype(dtype))
    gw_ref2, _ = oracle.backward(f64(gy), f64(st_round), f64(w), layer.r, groups=layer.groups, need_gx=False)
    _, gW2, _ = run_nhwc(gf, layer, x, gy, w, stash_in=st_round, need_gx=False)
    errs["gW_isolated"] = relerr(f64(gW2), gw_ref2)
    for k, v in errs.items():
        assert v <= tol, (layer.name, k, v, tol)
    assert bool((gW == gW[:, :, :1, :1]).all())                  # every tap of a kernel gets the same gradient


@pytest.mark.parametrize("index", [0, 1, 2])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_nhwc_full_size_mobilenetv2_block(gf, index, dtype):
    """The three layers of the benchmark's block at full size, channels last: the stash in full, g_W and
    g_X on sampled channels and images, and the properties that hold at any size."""
    layer = workloads.config3(2)[index].with_(dtype=dtype)
    check_layer_sampled(gf, layer, runner=run_nhwc)


@pytest.mark.parametrize("groups", [1, 16])
def test_nhwc_small_integers_are_exact(gf, groups):
    """Small integers, power-of-two patches: every sum is exact in bf16 products with fp32
    accumulation, so both layouts and the oracle agree to the last bit."""
    layer = L("ints", 2, 16, 16, 8, 8, 3, groups, 2)
    rng = np.random.default_rng(5)
    x = torch.from_numpy(rng.integers(0, 4, (2, 16, 8, 8)).astype(np.float32))
    gy = torch.from_numpy(rng.integers(-2, 3, (2, 16, 8, 8)).astype(np.float32) * 4.0)
    w = torch.from_numpy(rng.integers(-1, 2, (16, 16 // groups, 3, 3)).astype(np.float32))
    stash_ref = oracle.stash_forward(f64(x), 2)
    gw_ref, gx_ref = oracle.backward(f64(gy), stash_ref, f64(w), 2, groups=groups)
    stash, gW, gX = run_nhwc(gf, layer, x, gy, w)
    assert np.array_equal(f64(stash), stash_ref)
    assert np.array_equal(f64(gW), gw_ref)
    assert np.array_equal(f64(gX), gx_ref)


def test_nhwc_matches_nchw_path(gf):
    """The two layouts of the library against each other on one layer, beyond the oracle's bound."""
    from parity_util import run_gpu
    layer = L("both", 4, 96, 64, 28, 28, 1, 1, 2)
    x, gy, w = workloads.make_inputs(layer)
    s_a, gw_a, gx_a = run_gpu(gf, layer, x, gy, w)
    s_b, gw_b, gx_b = run_nhwc(gf, layer, x, gy, w)
    assert relerr(f64(s_b), f64(s_a)) <= 1e-6
    assert relerr(f64(gw_b), f64(gw_a)) <= 2e-5
    assert relerr(f64(gx_b), f64(gx_a)) <= 2e-5


def test_nhwc_nullable_outputs(gf):
    layer = L("nullable", 2, 24, 40, 14, 14, 3, 1, 2)
    x, gy, w = workloads.make_inputs(layer)
    _, gw_a, gx_a = run_nhwc(gf, layer, x, gy, w)
    _, gw_b, _ = run_nhwc(gf, layer, x, gy, w, need_gx=False)
    _, _, gx_c = run_nhwc(gf, layer, x, gy, w, need_gw=False)
    assert relerr(f64(gw_b), f64(gw_a)) <= TOL["f32"]
    assert torch.equal(gx_a, gx_c)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [(2, 8, 12, 9, 7, 3, 2, 1), (1, 4, 4, 8, 8, 5, 1, 1), (2, 6, 6, 8, 8, 3, 6, 1),
                                   (2, 6, 10, 8, 12, 3, 1, 2)], ids=["groups2", "k5", "depthwise", "stride2"])
def test_nhwc_r1_is_the_exact_backward(gf, shape, dtype):
    """r = 1 switches the method off (Section 4.2): the exact backward, here on channels-last tensors,
    any channel count, groups and dividing stride."""
    N, Cin, Cout, H, W, K, G, stride = shape
    layer = Layer("nhwc_r1", 0, 0, N, Cin, Cout, H, W, K, G, 1, dtype, "normal", 1.0)
    x, gy, w = workloads.make_inputs(layer)
    gy = gy[:, :, ::stride, ::stride].contiguous()
    desc = gf.make_desc(N, Cin, Cout, H, W, K, r=1, groups=G, stride=stride,
                        dtype=gf.GF_F32 if dtype == "f32" else gf.GF_BF16, layout=gf.GF_NHWC)
    dt = workloads.torch_dtype(dtype)
    stash = Guarded((N, H, W, Cin), dt)
    gf.gf_stash_forward(desc, nhwc(x).cuda(), stash.t)
    assert torch.equal(stash.t.cpu(), nhwc(x))                     # the stash is x itself
    gW = Guarded((Cout, Cin // G, K, K), torch.float32)
    gX = Guarded((N, H, W, Cin), dt)
    ws_bytes = gf.gf_backward_workspace_bytes(desc)
    ws = Guarded((ws_bytes,), torch.uint8)
    gf.gf_backward(desc, nhwc(gy).cuda(), stash.t, w.cuda(), gW.t, gX.t, ws.t, ws_bytes)
    assert gf.gf_last_async_status(ws.t) == gf.GF_OK
    torch.cuda.synchronize()
    for g in (stash, gW, gX, ws):
        g.check()
    if stride == 1:
        gw_ref, gx_ref = oracle.exact_backward(f64(x), f64(gy), f64(w), groups=G, pad=(K - 1) // 2)
    else:
        gw_ref, gx_ref = oracle.exact_backward_strided(f64(x), f64(gy), f64(w), stride, groups=G, pad=(K - 1) // 2)
    assert relerr(f64(gW.t), gw_ref) <= TOL[dtype] and relerr(f64(nchw_of(gX.t)), gx_ref) <= TOL[dtype]


def test_nhwc_static_scratch_and_host_step(gf):
    """The two other entry points that take a channels-last descriptor give the results of gf_backward."""
    layer = L("other_calls", 2, 24, 40, 14, 14, 3, 1, 2)
    x, gy, w = workloads.make_inputs(layer)
    stash, gw_a, gx_a = run_nhwc(gf, layer, x, gy, w)
    desc = gf.make_desc(layer.N, layer.C_in, layer.C_out, layer.H, layer.W, layer.K, r=layer.r, layout=gf.GF_NHWC)
    gW = torch.empty_like(gw_a)
    gX = torch.empty((layer.N, layer.H, layer.W, layer.C_in), device="cuda")
    gf.gf_backward_static_scratch(desc, nhwc(gy).cuda(), nhwc(stash), w.cuda(), gW, gX)
    torch.cuda.synchronize()
    assert relerr(f64(gW), f64(gw_a)) <= 1e-6 and torch.equal(nchw_of(gX), gx_a)
    # host buffers in, host buffers out
    h_x, h_gy, h_w = nhwc(x).pin_memory(), nhwc(gy).pin_memory(), w.pin_memory()
    h_gW = torch.empty(gw_a.shape, dtype=torch.float32).pin_memory()
    h_gX = torch.empty((layer.N, layer.H, layer.W, layer.C_in)).pin_memory()
    arena = torch.empty(gf.gf_host_step_arena_bytes(desc), dtype=torch.uint8, device="cuda")
    gf.gf_layer_step_host(desc, h_x, h_gy, h_w, h_gW, h_gX, arena)
    torch.cuda.synchronize()
    assert relerr(f64(h_gW), f64(gw_a)) <= 1e-6 and torch.equal(nchw_of(h_gX), gx_a.cpu())


def test_nhwc_unsupported_shapes_are_refused(gf):
    ok = dict(N=2, C_in=16, C_out=16, H=8, W=8, KH=3, r=2, layout=gf.GF_NHWC)

    def status(**kw):
        d = gf.make_desc(**{**ok, **kw})
        try:
            gf.gf_backward_workspace_bytes(d)
        except gf.GfError as e:
            return e.status
        return gf.GF_OK

    assert status() == gf.GF_OK
    assert status(C_in=12) == gf.GF_ERR_UNSUPPORTED                 # channel counts in multiples of 8
    assert status(C_out=20) == gf.GF_ERR_UNSUPPORTED
    assert status(groups=2) == gf.GF_ERR_UNSUPPORTED                # dense or depthwise only
    assert status(stride=2) == gf.GF_ERR_UNSUPPORTED
    assert status(r=1) == gf.GF_OK                                  # exact backward: as for NCHW
    assert status(r=1, C_in=12, groups=2, stride=2) == gf.GF_OK
