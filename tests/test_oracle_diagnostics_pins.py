"""Pins of the diagnostics oracle (oracle/gf_diagnostics.py): what the paper and the mathematics fix,
checked without a GPU.  Section 4.1 (SNR of the filtered gradient, Eq. (snr_g3), Eq. (dcac_ratio))
and the supplement's proof of Proposition 1."""
import numpy as np
import pytest

import oracle


def rng(seed):
    return np.random.default_rng(seed)


# ---- SNR terms -------------------------------------------------------------------------------

def test_snr_terms_loop_equals_numpy_sums():
    a, b = rng(0).normal(size=(2, 3, 4, 5)), rng(1).normal(size=(2, 3, 4, 5))
    s1, n1 = oracle.snr_terms(a, b)
    s2, n2 = oracle.snr_terms_fast(a, b)
    assert s1 == pytest.approx(s2, rel=1e-13) and n1 == pytest.approx(n2, rel=1e-13)
    assert s1 == pytest.approx(float((a ** 2).sum()), rel=1e-13)


def test_filter_noise_is_within_patch_variance():
    """Closed form: per patch sum (g - mean)^2 = sum g^2 - |P| mean^2; with partial edge patches."""
    for (H, W, r) in [(8, 8, 2), (7, 9, 4), (6, 6, 3), (5, 5, 8)]:
        g = rng(H * W + r).normal(size=(2, 3, H, W))
        signal, noise = oracle.filter_snr_terms(g, r)
        expect = 0.0
        for n in range(2):
            for c in range(3):
                for a in range(0, H, r):
                    for b in range(0, W, r):
                        blk = g[n, c, a:a + r, b:b + r]
                        expect += float((blk ** 2).sum()) - blk.size * float(blk.mean()) ** 2
        assert signal == pytest.approx(float((g ** 2).sum()), rel=1e-12)
        assert noise == pytest.approx(expect, rel=1e-10)


def test_filter_snr_equals_frequency_domain_ratio():
    """Parseval: the first line of Eq. (snr_g3), evaluated with the library FFT on every patch,
    gives the spatial-domain quotient.  The filtered patch keeps the DC bin and drops the rest."""
    r = 4
    g = rng(5).normal(size=(2, 2, 8, 12))
    signal, noise = oracle.filter_snr_terms(g, r)
    num = den = 0.0
    for n in range(2):
        for c in range(2):
            for a in range(0, 8, r):
                for b in range(0, 12, r):
                    G = np.fft.fft2(g[n, c, a:a + r, b:b + r])
                    Gt = np.zeros_like(G)
                    Gt[0, 0] = G[0, 0]
                    num += float((np.abs(G) ** 2).sum())
                    den += float((np.abs(G - Gt) ** 2).sum())
    assert signal / noise == pytest.approx(num / den, rel=1e-10)
    # and as a fraction of DC energy: 1 / SNR = 1 - (DC energy / total energy), patch by patch pooled
    dc = sum(float(np.abs(np.fft.fft2(g[n, c, a:a + r, b:b + r])[0, 0]) ** 2)
             for n in range(2) for c in range(2) for a in range(0, 8, r) for b in range(0, 12, r))
    assert noise / signal == pytest.approx(1.0 - dc / num, rel=1e-10)


def test_filter_snr_special_cases():
    base = rng(3).normal(size=(1, 2, 3, 3))
    const = np.repeat(np.repeat(base, 2, axis=2), 2, axis=3)          # patch-constant: nothing is lost
    s, n = oracle.filter_snr_terms(const, 2)
    assert n == pytest.approx(0.0, abs=1e-24) and s > 0
    g = rng(4).normal(size=(1, 1, 4, 4))
    s1, n1 = oracle.filter_snr_terms(g, 1)                             # r = 1: the filter is the identity
    assert n1 == 0.0
    zero_mean = g.copy()
    for a in range(0, 4, 2):
        for b in range(0, 4, 2):
            zero_mean[0, 0, a:a + 2, b:b + 2] -= zero_mean[0, 0, a:a + 2, b:b + 2].mean()
    s2, n2 = oracle.filter_snr_terms(zero_mean, 2)                     # filtered map is zero: SNR = 1
    assert n2 == pytest.approx(s2, rel=1e-12)


def test_filter_snr_terms_agree_with_the_method_oracle():
    """The filtered map used here is expand(patch_mean(g)) of the method's oracle."""
    g = rng(11).normal(size=(2, 3, 7, 10))
    for r in (2, 3, 4):
        approx = oracle.expand(oracle.patch_mean(g, r), 7, 10, r)
        s, n = oracle.snr_terms_fast(g, approx)
        s2, n2 = oracle.filter_snr_terms(g, r)
        assert s == pytest.approx(s2, rel=1e-13) and n == pytest.approx(n2, rel=1e-12)


# ---- DC / AC energy ratio ----------------------------------------------------------------------

def test_dcac_ratio_equals_library_fft():
    theta = rng(7).normal(size=(3, 4, 3, 5))
    for size in (None, (4, 8), (7, 7)):
        got = oracle.dcac_ratio(theta, size)
        for co in range(3):
            for ci in range(4):
                E = np.abs(np.fft.fft2(theta[co, ci], s=size)) ** 2
                dc = E[0, 0]
                E = E.copy()
                E[0, 0] = -1.0
                assert got[co, ci] == pytest.approx(dc / E.max(), rel=1e-10)


def test_dcac_ratio_closed_forms():
    K = 3
    ones = np.ones((1, 1, K, K))
    assert oracle.dcac_ratio(ones)[0, 0] > 1e20                        # all energy in the DC bin (AC: rounding only)
    delta = np.zeros((1, 1, K, K)); delta[0, 0, 0, 0] = 1.0
    assert oracle.dcac_ratio(delta)[0, 0] == pytest.approx(1.0, rel=1e-12)     # flat spectrum
    alt = np.array([[[[1.0, -1.0], [-1.0, 1.0]]]])
    assert oracle.dcac_ratio(alt)[0, 0] == 0.0                         # no DC component
    one_tap = np.full((2, 2, 1, 1), 0.5)
    assert np.isinf(oracle.dcac_ratio(one_tap)).all()                  # no AC component exists
    # a + b cos(2 pi j / 4) along one axis: DC bin 4a, bins +-1 each 2b
    a, b = 1.5, 0.5
    row = a + b * np.cos(2 * np.pi * np.arange(4) / 4)
    assert oracle.dcac_ratio(row.reshape(1, 1, 1, 4))[0, 0] == pytest.approx((4 * a) ** 2 / (2 * b) ** 2, rel=1e-10)
    # scale invariance and invariance under the 180-degree rotation of the backward pass
    th = rng(9).normal(size=(2, 2, 3, 3))
    assert np.allclose(oracle.dcac_ratio(3.0 * th), oracle.dcac_ratio(th), rtol=1e-12)
    assert np.allclose(oracle.dcac_ratio(th[:, :, ::-1, ::-1]), oracle.dcac_ratio(th), rtol=1e-10)


def test_proposition_1_on_one_patch():
    """Setting of the proof (one channel, one r x r patch, circular convolution): when the DC bin of
    the kernel's r x r spectrum is its largest, the SNR of the filtered input gradient is at least
    that of the filtered output gradient."""
    r = 4
    checked = 0
    for seed in range(40):
        g = rng(100 + seed).normal(size=(r, r))
        k = np.abs(rng(200 + seed).normal(size=(3, 3))) + 0.2          # positive taps: DC-dominated
        ratio = oracle.dcac_ratio(k.reshape(1, 1, 3, 3), (r, r))[0, 0]
        if ratio < 1.0:
            continue
        checked += 1
        Th = np.fft.fft2(k, s=(r, r))
        gx = np.real(np.fft.ifft2(np.conj(Th) * np.fft.fft2(g)))       # rotated kernel: Theta[-u,-v]
        gt = np.full_like(g, g.mean())
        gx_t = np.real(np.fft.ifft2(np.conj(Th) * np.fft.fft2(gt)))
        sy, ny = oracle.snr_terms(g, gt)
        sx, nx = oracle.snr_terms(gx, gx_t)
        assert sx / nx >= sy / ny * (1 - 1e-9)
    assert checked >= 20
