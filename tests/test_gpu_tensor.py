"""GPU parity of the training-tensor path (pcr_decode_tensor through the C ABI) against the
CPU oracle: oracle decode of the image, then the oracle's crop / flip / bilinear / normalise.

Tolerance.  The kernel evaluates the interpolation and the normalisation in single precision
(relative error of a few 2^-24 on values below 4), the oracle in double; both round once to
the output type.  Half-precision results may therefore differ by one unit in the last place
where the exact value lies next to a rounding boundary: 2^-9 for magnitudes in [2, 4), the
largest this normalisation produces.  Single-precision results must agree to 1e-5."""
import numpy as np
import pytest

import pcr_synth
from oracle import pcr_oracle as O

pytestmark = pytest.mark.gpu

MEAN = (0.485, 0.456, 0.406)
STD = (0.229, 0.224, 0.225)
HALF_ULP_TOL = 2.0 ** -9
BF16_ULP_TOL = 2.0 ** -6          # one unit in the last place of bfloat16 (8 significant bits) in [2, 4)
SINGLE_TOL = 1e-5


def _check(rec, k, crops, size, images, dtype_name="float16"):
    import torch
    from paper_1911_00472_b200 import Decoder
    dec = Decoder(rec.bytes)
    try:
        dtype = getattr(torch, dtype_name)
        t = dec.decode_tensor(k, crops, size, MEAN, STD, dtype=dtype)
        torch.cuda.synchronize()
        assert dec.status() == (-1, 0)
        assert tuple(t.shape) == (rec.n_images, 3, size, size) and t.dtype == dtype
        got = t.float().cpu().numpy().astype(np.float64)       # exact widening of every output type
        tol = {"float16": HALF_ULP_TOL, "bfloat16": BF16_ULP_TOL, "float32": SINGLE_TOL}[dtype_name]
        for i in images:
            _, rgb = O.decode_image(rec.bytes, i, k)
            want = O.training_tensor(rgb, crops[i], size, MEAN, STD, dtype=np.float16 if dtype_name == "float16" else np.float32)
            if dtype_name == "bfloat16":       # numpy has no bfloat16: round the oracle's float32 result with torch on the CPU
                want = torch.from_numpy(want).to(torch.bfloat16).float().numpy()
            err = np.abs(got[i] - want.astype(np.float64)).max()
            assert err <= tol, (i, k, crops[i], err)
    finally:
        dec.close()


def _dims(rec):
    return [(int(w), int(h)) for w, h in rec.dims]


def test_tiny_record_random_crops_every_k(rec0):
    crops = pcr_synth.random_resized_crops(_dims(rec0), 11)
    for k in (1, 5, 10):
        _check(rec0, k, crops, 24, range(rec0.n_images))


def test_widths_that_are_no_multiple_of_sixteen_dc_only():
    # k = 1 takes the DC-only pixel kernel; with such widths an output row starts at any byte address
    rec = pcr_synth.make_record(2, n_images=6)
    assert any(w % 16 for w, _ in _dims(rec))
    crops = pcr_synth.random_resized_crops(_dims(rec), 5)
    _check(rec, 1, crops, 32, range(rec.n_images))


def test_full_image_identity_size(rec0):
    # crop = whole image, size = image size: the tensor is the normalised decode itself
    crops = np.array([[0, 0, w, h, i & 1] for i, (w, h) in enumerate(_dims(rec0))], dtype=np.uint32)
    _check(rec0, 10, crops, 32, range(rec0.n_images), "float32")
    _check(rec0, 10, crops, 32, range(rec0.n_images), "float16")
    _check(rec0, 10, crops, 32, range(rec0.n_images), "bfloat16")


def test_imagenet_shaped_224_and_160(rec1_small):
    crops = pcr_synth.random_resized_crops(_dims(rec1_small), 12)
    _check(rec1_small, 10, crops, 224, range(0, rec1_small.n_images, 5))
    _check(rec1_small, 5, crops, 160, range(1, rec1_small.n_images, 7))


def test_odd_sizes_one_pixel_crops_and_edges(rec2_small):
    dims = _dims(rec2_small)
    crops = pcr_synth.random_resized_crops(dims, 13)
    W, H = dims[0]
    crops[0] = (W - 1, H - 1, 1, 1, 0)           # a single pixel in the corner
    crops[1] = (0, 0, W, 1, 1)                   # one row, mirrored
    crops[2] = (W // 2, 0, 1, H, 0)              # one column
    crops[3] = (15, 15, 2, 2, 0)                 # straddles four MCUs
    _check(rec2_small, 10, crops, 17, range(rec2_small.n_images))
    _check(rec2_small, 7, crops, 3, range(0, rec2_small.n_images, 3), "float32")


def test_bad_arguments_are_rejected(rec0):
    import torch
    from paper_1911_00472_b200 import Decoder, PcrError
    dec = Decoder(rec0.bytes)
    try:
        crops = pcr_synth.random_resized_crops(_dims(rec0), 14)
        bad = crops.copy()
        bad[3] = (30, 0, 3, 3, 0)                # reaches past the right edge of a 32x32 image
        with pytest.raises(PcrError):
            dec.decode_tensor(10, bad, 8, MEAN, STD)
        bad = crops.copy()
        bad[0, 4] = 2
        with pytest.raises(PcrError):
            dec.decode_tensor(10, bad, 8, MEAN, STD)
        with pytest.raises(PcrError):
            dec.decode_tensor(10, crops, 0, MEAN, STD)
        with pytest.raises(PcrError):
            dec.decode_tensor(10, crops, 8, MEAN, (0.2, 0.0, 0.2))
        with pytest.raises(PcrError):
            dec.decode_tensor(11, crops, 8, MEAN, STD)
        # rows outside the crops are not decoded: the fidelity of such a decode cannot be raised
        dec.decode_tensor(5, crops, 8, MEAN, STD)
        with pytest.raises(PcrError):
            dec.decode_more(10)
        # a plain decode afterwards is complete again
        out = dec.decode(10)
        torch.cuda.synchronize()
        want_c, want = O.decode_image(rec0.bytes, 7, 10)
        assert np.array_equal(dec.image(out, 7).cpu().numpy(), want)
        assert np.array_equal(dec.coeffs(7).cpu().numpy(), want_c)
        torch.cuda.synchronize()
    finally:
        dec.close()
