"""GPU parity of gf_backward_int8 (the reduced contractions on INT8 codes; supplement, gradient
quantization) against the INT8 oracle on the same seeded inputs, through the C ABI.  Every
floating-point step that decides a code is fixed in fp32 on both sides and the integer sums are
exact, so g_W and g_X must agree BIT FOR BIT (g_X after one rounding to the layer's dtype)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import int8
from paper_2301_00330_b200 import workloads
from paper_2301_00330_b200.workloads import Layer

from parity_util import Guarded, f64

pytestmark = pytest.mark.gpu


def L(name, N, Cin, Cout, H, W, K, r, dtype="f32"):
    return Layer(name, 0, 0, N, Cin, Cout, H, W, K, 1, r, dtype, "relu", 1e-2)


CASES = [
    L("one_tile", 2, 24, 40, 14, 14, 3, 2),
    L("partial_patches", 3, 24, 40, 14, 14, 3, 4),
    L("ragged_everything", 2, 70, 130, 9, 11, 3, 2),
    L("several_tiles", 5, 136, 264, 28, 28, 1, 2),              # 3 x 2 output tiles, K = 980 in 8 chunks
    L("long_k_split", 40, 96, 64, 28, 28, 1, 2),                # K = 7840: many slices of K
    L("r8", 4, 32, 48, 32, 32, 3, 8),
    L("r3_odd_map", 2, 16, 16, 13, 10, 3, 3),
    L("wide_co", 2, 40, 600, 8, 8, 1, 2),                       # c_o contraction in 5 chunks
    L("r4_wide_rows", 2, 16, 24, 16, 32, 3, 4),                 # bf16: two patches per 16-byte row of the gradient filter
    L("r2_wide_rows", 3, 8, 16, 12, 48, 1, 2),                  # two (fp32) / four (bf16) patches per 16-byte row
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("layer", CASES, ids=lambda l: l.name)
def test_int8_backward_bit_for_bit(gf, layer, dtype):
    layer = layer.with_(dtype=dtype)
    dt = workloads.torch_dtype(dtype)
    x, gy, w = workloads.make_inputs(layer)
    desc = gf.desc_for(layer)
    stash = torch.from_numpy(oracle.stash_forward(f64(x), layer.r)).to(dt)          # the same stash bits on both sides
    gw_ref, gx_ref = int8.int8_backward(gy.float().numpy(), stash.float().numpy(), w.float().numpy(), layer.r)
    gW = Guarded((layer.C_out, layer.C_in, layer.K, layer.K), torch.float32)
    gX = Guarded((layer.N, layer.C_in, layer.H, layer.W), dt)
    ws_bytes = gf.gf_backward_int8_workspace_bytes(desc)
    ws = Guarded((ws_bytes,), torch.uint8)
    for _ in range(2):                                                                # second call: stale workspace contents
        gf.gf_backward_int8(desc, gy.cuda(), stash.cuda(), w.cuda(), gW.t, gX.t, ws.t, ws_bytes)
        assert gf.gf_last_async_status(ws.t) == gf.GF_OK
        torch.cuda.synchronize()
        for b in (gW, gX, ws):
            b.check()
        assert np.array_equal(gW.t.cpu().numpy(), gw_ref)
        assert torch.equal(gX.t.cpu(), torch.from_numpy(gx_ref).to(dt))
    # nullable outputs
    gW2 = torch.full_like(gW.t, float("nan"))
    gf.gf_backward_int8(desc, gy.cuda(), stash.cuda(), w.cuda(), gW2, None, ws.t, ws_bytes)
    gX2 = torch.full_like(gX.t, float("nan"))
    gf.gf_backward_int8(desc, gy.cuda(), None, w.cuda(), None, gX2, ws.t, ws_bytes)
    torch.cuda.synchronize()
    assert torch.equal(gW2, gW.t) and torch.equal(gX2, gX.t)


def test_int8_backward_on_a_bench_layer_is_close_to_the_unquantised_method(gf):
    """Configuration 2's layer at a quarter of its batch: bit-exact against the INT8 oracle, and
    within a few per cent of the unquantised filtered backward (what quantization costs)."""
    layer = workloads.config2()[0].with_(N=16)
    x, gy, w = workloads.make_inputs(layer)
    desc = gf.desc_for(layer)
    stash = torch.from_numpy(oracle.stash_forward(f64(x), layer.r)).to(torch.bfloat16)
    gw_ref, gx_ref = int8.int8_backward(gy.float().numpy(), stash.float().numpy(), w.float().numpy(), layer.r)
    buf = gf.alloc_layer(desc)
    ws = torch.empty(gf.gf_backward_int8_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
    gf.gf_backward_int8(desc, gy.cuda(), stash.cuda(), w.cuda(), buf.g_W, buf.g_X, ws)
    torch.cuda.synchronize()
    assert np.array_equal(buf.g_W.cpu().numpy(), gw_ref)
    assert torch.equal(buf.g_X.cpu(), torch.from_numpy(gx_ref).to(torch.bfloat16))
    gw_fp, gx_fp = oracle.backward(f64(gy), f64(stash), f64(w), layer.r)
    assert np.abs(gw_ref - gw_fp).max() <= 0.05 * np.abs(gw_fp).max()
    assert np.abs(gx_ref - gx_fp).max() <= 0.05 * np.abs(gx_fp).max()
