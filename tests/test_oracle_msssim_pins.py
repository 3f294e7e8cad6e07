"""Pins of the oracle's multi-scale SSIM against closed forms, brute force and invariants."""
import numpy as np
import pytest

from oracle import pcr_oracle as O

C1, C2 = (0.01 * 255.0) ** 2, (0.03 * 255.0) ** 2


def _rand(h, w, seed):
    return np.random.default_rng(seed).integers(0, 256, size=(h, w, 3), dtype=np.uint8)


def test_identical_images_score_one():
    a = _rand(200, 180, 1)
    assert O.msssim(a, a) == pytest.approx(1.0, abs=1e-12)


def test_constant_images_closed_form():
    # no variance anywhere: every contrast-structure term is 1, the luminance term is the closed
    # form of two constants, raised to the last scale's weight
    a = np.full((192, 176, 3), 100, dtype=np.uint8)
    b = np.full((192, 176, 3), 140, dtype=np.uint8)
    lum = (2 * 100.0 * 140.0 + C1) / (100.0 ** 2 + 140.0 ** 2 + C1)
    assert O.msssim_scales(176, 192) == 5
    assert O.msssim(a, b) == pytest.approx(lum ** 0.1333, rel=1e-12)


def test_scale_count_and_weight_rescaling_on_small_images():
    assert O.msssim_scales(32, 32) == 2 and O.msssim_scales(10, 50) == 0 and O.msssim_scales(175, 400) == 4
    a = np.full((32, 32, 3), 60, dtype=np.uint8)
    b = np.full((32, 32, 3), 90, dtype=np.uint8)
    lum = (2 * 60.0 * 90.0 + C1) / (60.0 ** 2 + 90.0 ** 2 + C1)
    w_last = 0.2856 / (0.0448 + 0.2856)
    assert O.msssim(a, b) == pytest.approx(lum ** w_last, rel=1e-12)
    assert np.isnan(O.msssim(a[:8], b[:8]))


def test_single_scale_against_brute_force_windows():
    # an image with one scale only (sides 11..21): the direct double loop over windows with the
    # two-dimensional Gaussian weights
    a, b = _rand(15, 19, 2), _rand(15, 19, 3)
    x, y = O.luminance(a), O.luminance(b)
    g = O.gaussian_window()
    w2 = np.outer(g, g)
    cs, lum = [], []
    for r in range(15 - 10):
        for c in range(19 - 10):
            px, py = x[r:r + 11, c:c + 11], y[r:r + 11, c:c + 11]
            mx, my = (w2 * px).sum(), (w2 * py).sum()
            sxx, syy = (w2 * (px - mx) ** 2).sum(), (w2 * (py - my) ** 2).sum()
            sxy = (w2 * (px - mx) * (py - my)).sum()
            cs.append((2 * sxy + C2) / (sxx + syy + C2))
            lum.append((2 * mx * my + C1) / (mx * mx + my * my + C1))
    want = max(np.mean(cs), 0.0) * max(np.mean(lum), 0.0)      # one scale: weight 1
    assert O.msssim(a, b) == pytest.approx(want, rel=1e-9)


def test_window_is_normalised_and_symmetric_and_luminance_weights():
    g = O.gaussian_window()
    assert g.sum() == pytest.approx(1.0) and np.allclose(g, g[::-1]) and g[5] == g.max()
    assert g[4] / g[5] == pytest.approx(np.exp(-1 / (2 * 1.5 ** 2)))
    px = np.array([[[255, 0, 0], [0, 255, 0], [0, 0, 255], [10, 20, 30]]], dtype=np.uint8)
    assert np.allclose(O.luminance(px)[0], [76.245, 149.685, 29.07, 2.99 + 11.74 + 3.42])


def test_symmetry_and_monotone_degradation():
    a = _rand(180, 200, 4)
    rng = np.random.default_rng(5)
    def noisy(s):
        return np.clip(a.astype(np.float64) + rng.normal(0, s, a.shape), 0, 255).astype(np.uint8)
    b1, b2 = noisy(3), noisy(25)
    assert O.msssim(a, b1) == pytest.approx(O.msssim(b1, a), rel=1e-12)
    assert 1.0 > O.msssim(a, b1) > O.msssim(a, b2) > 0.0


def test_second_scale_is_the_block_average():
    # two images that differ only by a pattern the 2x2 average removes: a checkerboard of +-d.
    # On 32x32 (two scales) the second scale then sees identical images: its terms are exactly 1,
    # and the result is the first scale's contrast-structure mean to its weight.
    base = np.full((32, 32), 120.0)
    yy, xx = np.mgrid[0:32, 0:32]
    chk = np.where((yy + xx) % 2 == 0, 10, -10)
    a = np.repeat(base[..., None], 3, axis=2).astype(np.uint8)
    b = np.repeat((base + chk)[..., None], 3, axis=2).astype(np.uint8)
    x, y = O.luminance(a), O.luminance(b)
    g = O.gaussian_window()
    mx, my = O._valid_filter(x, g), O._valid_filter(y, g)
    sxx = O._valid_filter(x * x, g) - mx * mx
    syy = O._valid_filter(y * y, g) - my * my
    sxy = O._valid_filter(x * y, g) - mx * my
    cs1 = ((2 * sxy + C2) / (sxx + syy + C2)).mean()
    assert O.msssim(a, b) == pytest.approx(cs1 ** (0.0448 / (0.0448 + 0.2856)), rel=1e-9)
