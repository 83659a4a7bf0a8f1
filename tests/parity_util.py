"""Helpers of the GPU parity tests: run the CUDA path through the C ABI on a
seeded layer and compare with the fp64 CPU oracle on the same bits.

Error metric (both dtypes): max|gpu - ref| / max|ref| per output tensor.  An
element-wise relative error is meaningless here because the sums are zero-mean
and cancel.  Bounds: 1e-4 for fp32, 2e-2 for bf16 inputs with fp32 accumulation.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2301_00330_b200 import workloads

TOL = {"f32": 1e-4, "bf16": 2e-2}
GUARD = 256          # sentinel elements on each side of every output buffer
SENTINEL = 12345.0


def relerr(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    den = np.abs(ref).max()
    return float(np.abs(got - ref).max() / (den if den > 0 else 1.0))


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


class Guarded:
    """A device tensor with sentinel bands before and after it."""

    def __init__(self, shape, dtype, device="cuda"):
        n = int(np.prod(shape))
        # byte buffers (the workspace) start as all-ones: NaN as bf16 or fp32, so that scratch which
        # the library reads without having written it shows up in the results
        self.sentinel = 255 if dtype == torch.uint8 else SENTINEL
        self.raw = torch.full((n + 2 * GUARD,), self.sentinel, dtype=dtype, device=device)
        self.t = self.raw[GUARD:GUARD + n].view(shape)
        assert self.t.data_ptr() % 16 == 0

    def check(self):
        assert bool((self.raw[:GUARD] == self.sentinel).all()), "write before the buffer"
        assert bool((self.raw[-GUARD:] == self.sentinel).all()), "write past the buffer"


def run_gpu(gf, L: workloads.Layer, x, gy, w, stash_in=None, need_gw=True, need_gx=True):
    """stash (from gf_stash_forward unless given), g_W, g_X of layer L on cuda:0."""
    desc = gf.desc_for(L)
    dt = workloads.torch_dtype(L.dtype)
    xd, gyd, wd = x.cuda(), gy.cuda(), w.cuda()
    stash = Guarded(gf.gf_stash_dims(desc), dt)
    if stash_in is None:
        gf.gf_stash_forward(desc, xd, stash.t)
    else:
        stash.t.copy_(stash_in)
    gW = Guarded((L.C_out, L.C_ig, L.K, L.K), torch.float32)
    gX = Guarded((L.N, L.C_in, L.H, L.W), dt)
    ws_bytes = gf.gf_backward_workspace_bytes(desc)
    ws = Guarded((ws_bytes,), torch.uint8)
    before = gf.gf_kernel_launch_count()
    gf.gf_backward(desc, gyd, stash.t, wd, gW.t if need_gw else None, gX.t if need_gx else None,
                   ws.t, ws_bytes)
    assert gf.gf_last_async_status(ws.t) == gf.GF_OK
    torch.cuda.synchronize()
    assert gf.gf_kernel_launch_count() > before
    for g in (stash, gW, gX, ws):
        g.check()
    return stash.t, gW.t, gX.t


def check_layer_full(gf, L: workloads.Layer, isolate: bool = True):
    """Element-by-element parity of stash, g_W and g_X."""
    x, gy, w = workloads.make_inputs(L)
    tol = TOL[L.dtype]
    stash_ref = oracle.stash_forward(f64(x), L.r)
    gw_ref, gx_ref = oracle.backward(f64(gy), stash_ref, f64(w), L.r, groups=L.groups)
    stash, gW, gX = run_gpu(gf, L, x, gy, w)
    errs = {"stash": relerr(f64(stash), stash_ref), "gW": relerr(f64(gW), gw_ref), "gX": relerr(f64(gX), gx_ref)}
    if isolate:   # backward alone, fed the checker's stash rounded to the dtype
        st_round = torch.from_numpy(stash_ref).to(workloads.torch_dtype(L.dtype))
        gw_ref2, _ = oracle.backward(f64(gy), f64(st_round), f64(w), L.r, groups=L.groups, need_gx=False)
        _, gW2, _ = run_gpu(gf, L, x, gy, w, stash_in=st_round.cuda(), need_gx=False)
        errs["gW_isolated"] = relerr(f64(gW2), gw_ref2)
    for k, v in errs.items():
        assert v <= tol, (L.name, k, v, tol)
    return errs


def check_layer_sampled(gf, L: workloads.Layer, n_ch: int = 6, n_img: int = 2, seed: int = 0, runner=None):
    """Full-size layer: the stash in full, g_W on sampled channel pairs and g_X on
    sampled (image, channel) planes, each computed by the checker from sliced
    inputs; plus the structural properties that hold at any size."""
    x, gy, w = workloads.make_inputs(L)
    tol = TOL[L.dtype]
    stash, gW, gX = (runner or run_gpu)(gf, L, x, gy, w)      # a runner returns its tensors in NCHW order
    rng = np.random.default_rng(seed)
    errs = {}
    stash_ref = oracle.stash_forward(f64(x), L.r)
    errs["stash"] = relerr(f64(stash), stash_ref)
    del x
    gm = oracle.patch_mean(f64(gy), L.r)
    ts = oracle.kernel_sum(f64(w))
    imgs = np.sort(rng.choice(L.N, size=min(n_img, L.N), replace=False))
    if L.groups == 1:
        co = np.sort(rng.choice(L.C_out, size=min(n_ch, L.C_out), replace=False))
        ci = np.sort(rng.choice(L.C_in, size=min(n_ch, L.C_in), replace=False))
        gw_ref = oracle.reduced_gw(stash_ref[:, ci], gm[:, co], 1, L.K, L.K)
        errs["gW"] = relerr(f64(gW)[np.ix_(co, ci)], gw_ref)
        gx_ref = oracle.reduced_gx(gm[imgs], ts[:, ci], 1, L.H, L.W, L.r)
        errs["gX"] = relerr(f64(gX[torch.from_numpy(imgs).cuda()])[:, ci], gx_ref)
    else:
        assert L.groups == L.C_in == L.C_out
        c = np.sort(rng.choice(L.C_in, size=min(n_ch, L.C_in), replace=False))
        gw_ref = oracle.reduced_gw(stash_ref[:, c], gm[:, c], len(c), L.K, L.K)
        errs["gW"] = relerr(f64(gW)[c], gw_ref)
        gx_ref = oracle.reduced_gx(gm[imgs][:, c], ts[c], len(c), L.H, L.W, L.r)
        errs["gX"] = relerr(f64(gX[torch.from_numpy(imgs).cuda()])[:, c], gx_ref)
    for k, v in errs.items():
        assert v <= tol, (L.name, k, v, tol)
    # properties at any size: all taps equal; g_X constant on every patch
    assert bool((gW == gW[:, :, :1, :1]).all())
    if L.H % L.r == 0 and L.W % L.r == 0:
        blocks = gX.reshape(L.N, L.C_in, L.Hp, L.r, L.Wp, L.r)
        assert bool((blocks == blocks[:, :, :, :1, :, :1]).all())
    return errs
