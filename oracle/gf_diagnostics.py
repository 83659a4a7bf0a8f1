"""fp64 CPU oracle of the paper's error diagnostics (Section 4.1 and the supplement's proof of
Proposition 1).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests, the smoke check and the benchmark's
CPU-baseline leg may import this module.  It never touches the CUDA library.

  snr_terms(ref, approx)   signal energy sum ref^2 and noise energy sum (ref - approx)^2.  The
                           signal-to-noise ratio of an approximate gradient is their quotient: the
                           first line of Eq. (snr_g3) (and of the supplement's Eq. (basic_snr_gy)),
                           which by Parseval's theorem has the same value in the spatial and in
                           the frequency domain.
  filter_snr_terms(g, r)   the same for the gradient filter itself: ref = g_y, approx = g_y with
                           every r x r patch replaced by its average (Section 3.3).
  dcac_ratio(theta, size)  Eq. (dcac_ratio): for every (c_o, c_i) kernel, the energy of the DC
                           component of its 2-D DFT over the largest energy of any other
                           component.  `size` is the extent of the DFT (the kernel is zero-padded
                           to it); the default is the kernel's own extent.

Readings.  (1) The closed form printed as the second line of Eq. (snr_g3), with its factor
(2 r^2 - 1) / r^4, does not follow from the first line under the usual unnormalised DFT (the
average filter leaves the DC component as it is and removes the others); the first line -- the
definition -- is what is computed here.  (2) The table of energy ratios gives one number per model
family without saying how the per-kernel ratios are combined; this oracle returns the per-kernel
ratios.  (3) A kernel with a single tap (1 x 1, DFT size 1) has no AC component: its ratio is +inf.
"""
from __future__ import annotations

import numpy as np


def snr_terms(ref, approx) -> tuple[float, float]:
    ref = np.asarray(ref, dtype=np.float64)
    approx = np.asarray(approx, dtype=np.float64)
    assert ref.shape == approx.shape
    signal = 0.0
    noise = 0.0
    for a, b in zip(ref.reshape(-1), approx.reshape(-1)):
        signal += a * a
        noise += (a - b) * (a - b)
    return signal, noise


def snr_terms_fast(ref, approx) -> tuple[float, float]:
    """snr_terms with the two sums taken by numpy (for tensors too large for a Python loop)."""
    ref = np.asarray(ref, dtype=np.float64)
    approx = np.asarray(approx, dtype=np.float64)
    assert ref.shape == approx.shape
    d = ref - approx
    return float(np.sum(ref * ref)), float(np.sum(d * d))


def filter_snr_terms(g, r: int) -> tuple[float, float]:
    """Signal and noise energy of the gradient filter on g [N, C, H, W] (partial edge patches
    average over the elements they have, as everywhere in this oracle)."""
    g = np.asarray(g, dtype=np.float64)
    N, C, H, W = g.shape
    filtered = np.empty_like(g)
    for a in range(0, H, r):
        for b in range(0, W, r):
            block = g[:, :, a:a + r, b:b + r]
            filtered[:, :, a:a + r, b:b + r] = block.mean(axis=(2, 3), keepdims=True)
    return snr_terms_fast(g, filtered)


def dcac_ratio(theta, size: tuple[int, int] | None = None) -> np.ndarray:
    """[C_out, C_ig] array of |Theta[0,0]|^2 / max_{(u,v) != (0,0)} |Theta[u,v]|^2, the DFT written
    out as its defining double sum."""
    theta = np.asarray(theta, dtype=np.float64)
    Cout, Cig, KH, KW = theta.shape
    Sh, Sw = (KH, KW) if size is None else size
    assert Sh >= KH and Sw >= KW
    out = np.empty((Cout, Cig), dtype=np.float64)
    i = np.arange(KH).reshape(KH, 1)
    j = np.arange(KW).reshape(1, KW)
    for co in range(Cout):
        for ci in range(Cig):
            k = theta[co, ci]
            dc = 0.0
            ac = -1.0
            for u in range(Sh):
                for v in range(Sw):
                    phase = -2.0 * np.pi * (u * i / Sh + v * j / Sw)
                    re = float(np.sum(k * np.cos(phase)))
                    im = float(np.sum(k * np.sin(phase)))
                    e = re * re + im * im
                    if u == 0 and v == 0:
                        dc = e
                    elif e > ac:
                        ac = e
            if ac < 0.0:
                out[co, ci] = np.inf            # a single component: no AC part
            elif ac == 0.0:
                out[co, ci] = np.inf if dc > 0.0 else np.nan
            else:
                out[co, ci] = dc / ac
    return out
