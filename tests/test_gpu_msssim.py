"""GPU parity of pcr_msssim (through the C ABI) against the oracle's multi-scale SSIM.

Tolerance.  The kernels evaluate a window's statistics in single precision on luminance minus
128 (|value| <= 128, squares <= 2^14, so a variance carries an absolute error of about 1e-3 next
to C2 = 58.5: 2e-5 relative per window, averaged over thousands of windows) and sum a scale in
double precision; the oracle works in double throughout.  Scores agree to 2e-4."""
import numpy as np
import pytest

import pcr_synth
from oracle import pcr_oracle as O

pytestmark = pytest.mark.gpu
TOL = 2e-4


def _scores(rec, k_a, k_b):
    import torch
    from paper_1911_00472_b200 import Decoder
    dec = Decoder(rec.bytes)
    try:
        a = dec.decode(k_a, dec.alloc_out())
        b = dec.decode(k_b, dec.alloc_out())
        s = dec.msssim(a, b)
        torch.cuda.synchronize()
        assert dec.status() == (-1, 0)
        return s.cpu().numpy()
    finally:
        dec.close()


def _check(rec, k, images):
    G = 10
    got = _scores(rec, k, G)
    for i in images:
        _, lo = O.decode_image(rec.bytes, i, k)
        _, hi = O.decode_image(rec.bytes, i, G)
        want = O.msssim(lo, hi)
        assert abs(float(got[i]) - want) <= TOL, (i, k, float(got[i]), want)
    return got


def test_tiny_record_two_scales(rec0):
    for k in (1, 2, 6):
        _check(rec0, k, range(rec0.n_images))


def test_imagenet_shaped_five_scales(rec1_small):
    s1 = _check(rec1_small, 1, range(0, rec1_small.n_images, 3))
    s5 = _check(rec1_small, 5, range(1, rec1_small.n_images, 3))
    assert np.all(s5 > s1)                      # more scan groups, closer to the full image


def test_celeba_shaped_odd_sizes(rec2_small):
    _check(rec2_small, 2, range(rec2_small.n_images))


def test_identical_decodes_score_one_twice(rec1_small):
    # two calls in a row on the same scratch: the sums are cleared by every call
    import torch
    from paper_1911_00472_b200 import Decoder
    dec = Decoder(rec1_small.bytes)
    try:
        a = dec.decode(10, dec.alloc_out())
        for _ in range(2):
            s = dec.msssim(a, a)
            torch.cuda.synchronize()
            assert np.allclose(s.cpu().numpy(), 1.0, atol=1e-6)
    finally:
        dec.close()


def test_images_too_small_for_a_window_give_nan():
    dims = [(8, 8), (40, 24), (10, 64)]
    coeffs = [np.zeros((pcr_synth.num_blocks(w, h), 64), dtype=np.int16) for w, h in dims]
    for c in coeffs:
        c[:, 0] = 5
    rec = pcr_synth.record_from_coeffs(dims, coeffs)
    got = _scores(rec, 1, 10)
    assert np.isnan(got[0]) and np.isnan(got[2])
    _, lo = O.decode_image(rec.bytes, 1, 1)
    _, hi = O.decode_image(rec.bytes, 1, 10)
    assert abs(float(got[1]) - O.msssim(lo, hi)) <= TOL
