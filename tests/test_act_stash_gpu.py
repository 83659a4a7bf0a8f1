"""GPU parity of gf_act_stash_forward (the forward-side step fused into the producer of x, Section
4.2): x = act(z) bit for bit, and the stash of that x within the tolerance of gf_stash_forward,
against the fp64 CPU oracle on the same seeded pre-activations, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2301_00330_b200 import workloads
from paper_2301_00330_b200.workloads import Layer

from parity_util import TOL, Guarded, f64, relerr

pytestmark = pytest.mark.gpu

ACTS = {"none": 0, "relu": 1, "relu6": 2}

SHAPES = [
    # (N, C, H, W, r)
    (3, 24, 14, 14, 2),       # streamed kernel, item mode
    (2, 16, 28, 28, 4),
    (4, 8, 16, 16, 4),        # streamed kernel, linear (shuffle) mode
    (2, 8, 32, 32, 8),
    (37, 40, 28, 28, 2),      # more tiles than ring slots per CTA
    (1, 3, 30, 30, 2),        # last tile not a multiple of 16 bytes in bf16
    (2, 5, 7, 9, 2),          # partial patches: activation and pooling as two passes
    (2, 6, 12, 9, 3),
    (1, 2, 16, 600, 8),       # patch rows wider than a tile
    (2, 4, 9, 9, 1),          # r = 1: x and the stash are both act(z)
]


@pytest.mark.parametrize("act", ["relu", "relu6", "none"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_act_stash_forward(gf, shape, dtype, act):
    N, C, H, W, r = shape
    dt = workloads.torch_dtype(dtype)
    g = torch.Generator(device="cpu")
    g.manual_seed(9000 + r)
    z = (torch.randn((N, C, H, W), generator=g) * 3.0).to(dt).contiguous()      # plenty of values beyond 0 and 6
    desc = gf.make_desc(N, C, C, H, W, 3, r=r, dtype=gf.GF_F32 if dtype == "f32" else gf.GF_BF16)
    x_ref, stash_ref = oracle.act_stash_forward(f64(z), act, r)
    x = Guarded((N, C, H, W), dt)
    stash = Guarded(gf.gf_stash_dims(desc), dt)
    gf.gf_act_stash_forward(desc, ACTS[act], z.cuda(), x.t, stash.t)
    torch.cuda.synchronize()
    assert gf.gf_last_async_status(torch.zeros(64, dtype=torch.uint8, device="cuda")) == gf.GF_OK
    x.check(); stash.check()
    assert np.array_equal(f64(x.t), x_ref)                     # max / min are exact in either dtype
    assert relerr(f64(stash.t), stash_ref) <= TOL[dtype]
    # in place: x may be z itself
    zc = z.cuda().clone()
    stash2 = torch.empty_like(stash.t)
    gf.gf_act_stash_forward(desc, ACTS[act], zc, zc, stash2)
    torch.cuda.synchronize()
    assert torch.equal(zc, x.t) and torch.equal(stash2, stash.t)


def test_act_stash_equals_separate_steps_on_a_bench_layer(gf):
    """At the size of the benchmark's depthwise layer: the fused pass gives what an element-wise
    activation followed by gf_stash_forward gives, bit for bit."""
    layer = workloads.config3(2)[1].with_(N=32)
    desc = gf.desc_for(layer)
    g = torch.Generator(device="cpu")
    g.manual_seed(5)
    z = torch.randn((layer.N, layer.C_in, layer.H, layer.W), generator=g).cuda()
    x = torch.empty_like(z)
    stash = torch.empty(gf.gf_stash_dims(desc), device="cuda")
    gf.gf_act_stash_forward(desc, gf.GF_ACT_RELU6, z, x, stash)
    ref_x = torch.clamp(z, 0.0, 6.0)
    ref_stash = torch.empty_like(stash)
    gf.gf_stash_forward(desc, ref_x, ref_stash)
    torch.cuda.synchronize()
    assert torch.equal(x, ref_x) and torch.equal(stash, ref_stash)
    x64, s64 = oracle.act_stash_forward(f64(z), "relu6", layer.r)
    assert np.array_equal(f64(x), x64) and relerr(f64(stash), s64) <= TOL["f32"]
