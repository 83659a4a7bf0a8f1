"""GPU parity of the error diagnostics (Section 4.1: SNR of a filtered gradient, Eq. (snr_g3); DC/AC
energy ratio of a kernel, Eq. (dcac_ratio)) against the fp64 CPU oracle on the same seeded inputs,
through the C ABI.  The sums run in fp64 on both sides, so the bound is 1e-9 relative (the order of
the additions differs); the ratio array is fp32: 1e-5."""
import numpy as np
import pytest
import torch

import oracle
from paper_2301_00330_b200 import workloads
from paper_2301_00330_b200.workloads import Layer

from parity_util import f64

pytestmark = pytest.mark.gpu


def _draw(shape, seed, dtype, scale=1.0):
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return (torch.randn(shape, generator=g) * scale).to(dtype).contiguous()


def _terms(gf, fn, *args):
    out = torch.full((2,), float("nan"), dtype=torch.float64, device="cuda")
    fn(*args, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("shape,r", [((2, 3, 8, 8), 2), ((3, 5, 14, 14), 4), ((2, 4, 7, 9), 2), ((1, 2, 5, 5), 8),
                                     ((4, 16, 28, 28), 2), ((2, 3, 12, 9), 3), ((2, 2, 16, 16), 1), ((64, 96, 28, 28), 4)])
def test_filter_snr_terms(gf, shape, r, dtype):
    g = _draw(shape, 77 + r, dtype, 1e-2)
    got = _terms(gf, lambda t, out: gf.gf_filter_snr_terms(t, r, out), g.cuda())
    s, n = oracle.filter_snr_terms(f64(g), r)
    assert got[0] == pytest.approx(s, rel=1e-9)
    if r == 1:
        assert got[1] == 0.0 and n == 0.0
    else:
        assert got[1] == pytest.approx(n, rel=1e-9)


def test_filter_snr_of_a_patch_constant_map_is_infinite(gf):
    base = _draw((2, 3, 7, 7), 5, torch.float32)
    g = base.repeat_interleave(4, 2).repeat_interleave(4, 3).contiguous()
    got = _terms(gf, lambda t, out: gf.gf_filter_snr_terms(t, 4, out), g.cuda())
    s, n = oracle.filter_snr_terms(f64(g), 4)
    assert got[0] == pytest.approx(s, rel=1e-9)
    assert n <= 1e-20 * s and got[1] <= 1e-12 * got[0]            # nothing is lost: the quotient diverges


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("count", [1, 1000, 262144 + 37, 5_000_000])
def test_snr_terms(gf, count, dtype):
    ref = _draw((count,), 1, dtype)
    approx = (ref.float() + _draw((count,), 2, torch.float32, 0.1)).to(dtype)
    got = _terms(gf, lambda a, b, out: gf.gf_snr_terms(a, b, out), ref.cuda(), approx.cuda())
    s, n = oracle.snr_terms_fast(f64(ref), f64(approx))
    assert got[0] == pytest.approx(s, rel=1e-9) and got[1] == pytest.approx(n, rel=1e-9)


def test_snr_of_the_filtered_input_gradient_end_to_end(gf):
    """SNR of g~_x against the exact g_x of the same layer, every step on the GPU (exact backward =
    patch size 1), against the oracle's own exact and filtered backward; Proposition 1's two SNRs."""
    layer = Layer("snr_e2e", 0, 0, 4, 24, 40, 16, 16, 3, 1, 2, "f32", "relu", 1e-2)
    x, gy, w = workloads.make_inputs(layer)
    d_r, d_1 = gf.desc_for(layer), gf.desc_for(layer.with_(r=1))
    xd, gyd, wd = x.cuda(), gy.cuda(), w.cuda()
    b_r, b_1 = gf.alloc_layer(d_r), gf.alloc_layer(d_1)
    gf.gf_stash_forward(d_r, xd, b_r.stash)
    gf.gf_backward(d_r, gyd, b_r.stash, wd, None, b_r.g_X, b_r.workspace)
    gf.gf_stash_forward(d_1, xd, b_1.stash)
    gf.gf_backward(d_1, gyd, b_1.stash, wd, None, b_1.g_X, b_1.workspace)
    got_x = _terms(gf, lambda a, b, out: gf.gf_snr_terms(a, b, out), b_1.g_X, b_r.g_X)
    got_y = _terms(gf, lambda t, out: gf.gf_filter_snr_terms(t, 2, out), gyd)
    _, gx_exact = oracle.exact_backward(f64(x), f64(gy), f64(w), 1, 1, need_gw=False)
    _, gx_filt = oracle.backward(f64(gy), oracle.stash_forward(f64(x), 2), f64(w), 2, need_gw=False)
    sx, nx = oracle.snr_terms_fast(gx_exact, gx_filt)
    sy, ny = oracle.filter_snr_terms(f64(gy), 2)
    assert got_x[0] / got_x[1] == pytest.approx(sx / nx, rel=1e-3)       # fp32 g_X on the GPU side
    assert got_y[0] / got_y[1] == pytest.approx(sy / ny, rel=1e-9)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("shape,dft", [((8, 6, 3, 3), (0, 0)), ((5, 7, 5, 5), (0, 0)), ((4, 4, 3, 3), (4, 4)),
                                       ((3, 2, 1, 7), (0, 0)), ((6, 3, 1, 1), (0, 0)), ((2, 3, 3, 3), (8, 6)),
                                       ((64, 96, 3, 3), (0, 0))])
def test_dcac_ratio(gf, shape, dft, dtype):
    w = _draw(shape, 31, dtype, 0.2) + 0.05                       # a DC offset, as trained kernels have
    w = w.to(dtype).contiguous()
    ratio = torch.full(shape[:2], float("nan"), dtype=torch.float32, device="cuda")
    gf.gf_dcac_ratio(w.cuda(), ratio, dft)
    torch.cuda.synchronize()
    ref = oracle.dcac_ratio(f64(w), None if dft == (0, 0) else dft)
    got = ratio.cpu().numpy().astype(np.float64)
    if shape[2] * shape[3] == 1 and dft == (0, 0):
        assert np.isinf(got).all() and np.isinf(ref).all()
    else:
        assert np.allclose(got, ref, rtol=1e-5, atol=0.0)
