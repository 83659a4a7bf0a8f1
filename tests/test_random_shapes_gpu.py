"""Seeded random layer geometries through every dispatch arm of the library (dense, grouped,
depthwise; stride 1 and dividing strides; r = 1, dividing and non-dividing patch sizes; both dtypes;
both layouts) against the oracle.  A descriptor the library refuses must be refused with
GF_ERR_UNSUPPORTED before anything runs; one it accepts must give the oracle's numbers."""
import numpy as np
import pytest
import torch

import oracle
from paper_2301_00330_b200 import workloads

from parity_util import TOL, Guarded, f64, relerr

pytestmark = pytest.mark.gpu


def _draw_case(rng):
    kind = rng.choice(["dense", "dense", "dense", "grouped", "depthwise"])
    layout = rng.choice(["nchw", "nchw", "nhwc"])
    unit = 8 if (layout == "nhwc" or rng.random() < 0.6) else 1
    if kind == "depthwise":
        C_in = C_out = int(rng.integers(1, 10)) * unit
        G = C_in
    elif kind == "grouped":
        G = int(rng.choice([2, 4]))
        C_in, C_out = int(rng.integers(1, 5)) * unit * G, int(rng.integers(1, 5)) * unit * G
    else:
        G = 1
        C_in, C_out = int(rng.integers(1, 20)) * unit, int(rng.integers(1, 20)) * unit
        if rng.random() < 0.15:
            C_out = 512 + 8 * int(rng.integers(0, 5))          # long contractions
    stride = int(rng.choice([1, 1, 1, 2]))
    r = int(rng.choice([1, 2, 2, 2, 3, 4, 4, 7, 8]))
    H, W = int(rng.integers(3, 21)) * stride * 2, int(rng.integers(3, 21)) * stride * 2
    if rng.random() < 0.3:                                      # odd maps: partial patches
        H, W = H + stride, W - stride
    K = int(rng.choice([1, 3, 3, 5]))
    if r == 1:                                                  # the exact oracle is brute force: keep it small
        H, W = min(H, 12 * stride), min(W, 10 * stride)
        C_in, C_out = min(C_in, 8 * max(G, 1) if G > 1 else 24), min(C_out, 8 * max(G, 1) if G > 1 else 24)
        if G > 1 and G == C_in:
            C_out = C_in
    N = int(rng.integers(1, 6))
    dtype = str(rng.choice(["f32", "bf16"]))
    return dict(N=N, C_in=C_in, C_out=C_out, H=H, W=W, K=K, G=G, r=r, stride=stride, dtype=dtype, layout=layout)


def _cases(n, seed):
    rng = np.random.default_rng(seed)
    return [_draw_case(rng) for _ in range(n)]


def _id(c):
    return "{layout}-{dtype}-N{N}-{C_in}to{C_out}-g{G}-{H}x{W}-k{K}-r{r}-s{stride}".format(**c)


@pytest.mark.parametrize("case", _cases(90, 20240607) + _cases(110, 7), ids=_id)
def test_random_geometry(gf, case):
    c = case
    N, Cin, Cout, H, W, K, G, r, s = c["N"], c["C_in"], c["C_out"], c["H"], c["W"], c["K"], c["G"], c["r"], c["stride"]
    cl = c["layout"] == "nhwc"
    dt = workloads.torch_dtype(c["dtype"])
    desc = gf.make_desc(N, Cin, Cout, H, W, K, r=r, groups=G, stride=s, dtype=gf.GF_F32 if c["dtype"] == "f32" else gf.GF_BF16,
                        layout=gf.GF_NHWC if cl else gf.GF_NCHW)
    try:
        ws_bytes = gf.gf_backward_workspace_bytes(desc)
    except gf.GfError as e:
        assert e.status == gf.GF_ERR_UNSUPPORTED
        # refusals have stated reasons: channels-last outside its limits, or a stride that does not divide
        assert (cl and r >= 2 and (s != 1 or Cin % 8 or Cout % 8 or (G != 1 and not (G == Cin == Cout)))) or H % s or W % s
        return
    g = torch.Generator(device="cpu")
    g.manual_seed(1 + N + 3 * Cin + 5 * Cout + 7 * H + 11 * W + 13 * r)
    x = torch.randn((N, Cin, H, W), generator=g).clamp_(min=0).to(dt)
    gy = (torch.randn((N, Cout, H // s, W // s), generator=g) * 1e-2).to(dt)
    w = (torch.randn((Cout, Cin // G, K, K), generator=g) * (2.0 / (Cin // G * K * K)) ** 0.5).to(dt)

    def dev(t):
        return (t.permute(0, 2, 3, 1).contiguous() if cl else t).cuda()

    def back(t):
        return t.permute(0, 3, 1, 2) if cl else t

    n_, c_, hp, wp = gf.gf_stash_dims(desc)
    stash = Guarded((n_, hp, wp, c_) if cl else (n_, c_, hp, wp), dt)
    gW = Guarded((Cout, Cin // G, K, K), torch.float32)
    gX = Guarded((N, H, W, Cin) if cl else (N, Cin, H, W), dt)
    ws = Guarded((ws_bytes,), torch.uint8)
    gf.gf_stash_forward(desc, dev(x), stash.t)
    gf.gf_backward(desc, dev(gy), stash.t, w.cuda(), gW.t, gX.t, ws.t, ws_bytes)
    assert gf.gf_last_async_status(ws.t) == gf.GF_OK
    torch.cuda.synchronize()
    for b in (stash, gW, gX, ws):
        b.check()

    pad = (K - 1) // 2
    if r == 1:
        stash_ref = f64(x)
        if s == 1:
            gw_ref, gx_ref = oracle.exact_backward(f64(x), f64(gy), f64(w), groups=G, pad=pad)
        else:
            gw_ref, gx_ref = oracle.exact_backward_strided(f64(x), f64(gy), f64(w), s, G, pad)
    elif s == 1:
        stash_ref = oracle.stash_forward(f64(x), r)
        gw_ref, gx_ref = oracle.backward(f64(gy), stash_ref, f64(w), r, groups=G)
    else:
        stash_ref = oracle.strided_stash_forward(f64(x), r, s)
        gw_ref, gx_ref = oracle.strided_backward(f64(gy), stash_ref, f64(w), r, s, G)
    tol = TOL[c["dtype"]]
    assert relerr(f64(back(stash.t)), stash_ref) <= tol
    assert relerr(f64(gW.t), gw_ref) <= tol
    assert relerr(f64(back(gX.t)), gx_ref) <= tol
