"""Pins of the oracle's training-tensor epilogue (crop, flip, bilinear resize, normalise)
against things other than itself: closed forms, a hand-computed case and torch's CPU
interpolation routine."""
import numpy as np
import pytest

from oracle import pcr_oracle as O

MEAN = (0.485, 0.456, 0.406)
STD = (0.229, 0.224, 0.225)


def _rand_rgb(h, w, seed):
    return np.random.default_rng(seed).integers(0, 256, size=(h, w, 3), dtype=np.uint8)


def test_identity_when_crop_and_size_equal_the_image():
    rgb = _rand_rgb(24, 24, 1)
    out = O.training_tensor(rgb, (0, 0, 24, 24, 0), 24, MEAN, STD, dtype=np.float64)
    want = (rgb.astype(np.float64).transpose(2, 0, 1) / 255.0 - np.array(MEAN).reshape(3, 1, 1)) / np.array(STD).reshape(3, 1, 1)
    assert np.allclose(out, want, rtol=0, atol=1e-12)


def test_flip_mirrors_the_columns():
    rgb = _rand_rgb(40, 56, 2)
    crop = (5, 3, 37, 30)
    a = O.training_tensor(rgb, crop + (0,), 16, MEAN, STD, dtype=np.float64)
    b = O.training_tensor(rgb, crop + (1,), 16, MEAN, STD, dtype=np.float64)
    assert np.array_equal(b, a[:, :, ::-1])


def test_affine_images_are_reproduced():
    # bilinear interpolation is exact on functions that are affine in x and y: away from the
    # clamped border the output equals the function at the source coordinate
    H, W = 64, 80
    y, x = np.mgrid[0:H, 0:W]
    rgb = np.stack([2 * x + 10, 3 * y + 5, x + y], axis=-1).astype(np.uint8)
    x0, y0, cw, ch, S = 7, 4, 60, 50, 20
    out = O.training_tensor(rgb, (x0, y0, cw, ch, 0), S, (0, 0, 0), (1 / 255.0,) * 3, dtype=np.float64)
    ox = np.arange(S)
    fx = x0 + (ox + 0.5) * cw / S - 0.5
    fy = y0 + (ox + 0.5) * ch / S - 0.5
    assert np.allclose(out[0], np.broadcast_to(2 * fx + 10, (S, S)), atol=1e-9)
    assert np.allclose(out[1], np.broadcast_to((3 * fy + 5)[:, None], (S, S)), atol=1e-9)
    assert np.allclose(out[2], fx[None, :] + fy[:, None], atol=1e-9)


def test_hand_computed_upscale():
    # 2x2 -> 4x4: source coordinates -0.25 (clamped to 0), 0.25, 0.75, 1.25 (clamped to 1)
    g = np.array([[0, 100], [200, 40]], dtype=np.uint8)
    rgb = np.stack([g, g, g], axis=-1)
    out = O.training_tensor(rgb, (0, 0, 2, 2, 0), 4, (0, 0, 0), (1 / 255.0,) * 3, dtype=np.float64)[0]
    row0 = np.array([0.0, 25.0, 75.0, 100.0])
    row3 = np.array([200.0, 160.0, 80.0, 40.0])
    want = np.stack([row0, 0.75 * row0 + 0.25 * row3, 0.25 * row0 + 0.75 * row3, row3])
    assert np.allclose(out, want, atol=1e-9)


@pytest.mark.parametrize("crop,size", [((3, 2, 50, 41, 0), 16), ((0, 0, 33, 47, 1), 24), ((10, 10, 9, 7, 0), 32), ((0, 0, 64, 48, 0), 7)])
def test_against_torch_cpu_interpolate(crop, size):
    torch = pytest.importorskip("torch")
    rgb = _rand_rgb(48, 64, 3)
    x0, y0, cw, ch, flip = crop
    region = torch.from_numpy(rgb[y0:y0 + ch, x0:x0 + cw].astype(np.float64)).permute(2, 0, 1)[None]
    ref = torch.nn.functional.interpolate(region, size=(size, size), mode="bilinear", align_corners=False, antialias=False)[0].numpy()
    if flip:
        ref = ref[:, :, ::-1]
    out = O.training_tensor(rgb, crop, size, (0, 0, 0), (1 / 255.0,) * 3, dtype=np.float64)
    assert np.allclose(out, ref, atol=1e-9)


def test_constant_image_and_half_precision_rounding():
    rgb = np.full((20, 30, 3), 77, dtype=np.uint8)
    out = O.training_tensor(rgb, (2, 3, 11, 13, 1), 8, MEAN, STD)
    assert out.dtype == np.float16
    want = ((77 / 255.0 - np.array(MEAN)) / np.array(STD)).astype(np.float16)
    assert np.array_equal(out, np.broadcast_to(want.reshape(3, 1, 1), (3, 8, 8)))


def test_crop_outside_the_image_is_rejected():
    rgb = _rand_rgb(8, 8, 4)
    with pytest.raises(ValueError):
        O.training_tensor(rgb, (4, 0, 5, 8, 0), 4, MEAN, STD)
    with pytest.raises(ValueError):
        O.training_tensor(rgb, (0, 0, 0, 8, 0), 4, MEAN, STD)


def test_seeded_crops_are_inside_and_reproducible():
    import pcr_synth
    dims = [(256, 496), (31, 17), (600, 450), (1, 1)]
    a = pcr_synth.random_resized_crops(dims, 5)
    b = pcr_synth.random_resized_crops(dims, 5)
    assert np.array_equal(a, b)
    for (W, H), (x0, y0, w, h, f) in zip(dims, a):
        assert w >= 1 and h >= 1 and x0 + w <= W and y0 + h <= H and f in (0, 1)
    assert not np.array_equal(a, pcr_synth.random_resized_crops(dims, 6))
