"""Pins of the oracle on the other chroma samplings: 4:4:4, 4:2:2, 4:4:0 and greyscale (the
paper's per-scan example for HAM10000 is a 4:4:4 file by the arithmetic of its printed sizes).
Each pin ties the oracle to something other than itself: the generator's ground truth, the
closed-form mask of the scan script, a third-party decoder and encoder (Pillow) in both
directions, chroma planes included where no upsampling intervenes, and brute-force pixel formulas."""
import io

import numpy as np
import pytest

import pcr_synth
from oracle import pcr_oracle as O

from helpers import block_grids, mask_truth_script

SAMPLINGS = {"444": (1, 1, 3), "422": (2, 1, 3), "440": (1, 2, 3), "420": (2, 2, 3), "grey": (1, 1, 1)}
TEN = [((0, 1, 2), 0, 0, 0, 1), ((0,), 1, 5, 0, 2), ((2,), 1, 63, 0, 1), ((1,), 1, 63, 0, 1), ((0,), 6, 63, 0, 2),
       ((0,), 1, 63, 2, 1), ((0, 1, 2), 0, 0, 1, 0), ((2,), 1, 63, 1, 0), ((1,), 1, 63, 1, 0), ((0,), 1, 63, 1, 0)]
GREY = [((0,), Ss, Se, Ah, Al) for comps, Ss, Se, Ah, Al in TEN if 0 in comps]


def _script(samp):
    return GREY if samp[2] == 1 else TEN


def _record(name, config=2, n=3, **kw):
    with pcr_synth.sampling(*SAMPLINGS[name]):
        return pcr_synth.make_record(config, n_images=n, **kw)


@pytest.mark.parametrize("name", sorted(SAMPLINGS))
@pytest.mark.parametrize("restart_rows", [True, False])
def test_ground_truth_and_script_mask_every_k(name, restart_rows):
    samp = SAMPLINGS[name]
    rec = _record(name, restart_rows=restart_rows)
    n, G = O.record_info(rec.bytes)
    assert G == len(_script(samp))
    for i in range(n):
        W, H = rec.dims[i]
        assert O.image_sampling(rec.bytes, i) == samp
        t = rec.truth(i)
        assert t.shape[0] == O.num_blocks(W, H, samp) == sum(a * b for a, b in block_grids(W, H, samp)[2])
        for k in range(1, G + 1):
            got, _ = O.decode_image(rec.bytes, i, k, False)
            want = t if k == G else mask_truth_script(t, W, H, _script(samp), k, samp)
            assert np.array_equal(got, want), (name, i, k)


@pytest.mark.parametrize("name", sorted(SAMPLINGS))
def test_odd_sizes_round_trip(name):
    samp = SAMPLINGS[name]
    dims = [(1, 1), (8, 8), (9, 17), (17, 9), (16, 16), (31, 33), (100, 7)]
    rng = np.random.default_rng(5)
    with pcr_synth.sampling(*samp):
        coeffs = []
        for W, H in dims:
            nb = pcr_synth.num_blocks(W, H)
            c = (rng.integers(-40, 41, size=(nb, 64)) * (rng.random((nb, 64)) < 0.3)).astype(np.int16)
            c[:, 0] = rng.integers(-500, 500, size=nb)
            coeffs.append(c)
        rec = pcr_synth.record_from_coeffs(dims, coeffs)
    _, G = O.record_info(rec.bytes)
    for i in range(len(dims)):
        got, _ = O.decode_image(rec.bytes, i, G, False)
        assert np.array_equal(got, rec.truth(i)), (name, dims[i])


def _pillow_planes(jpeg_bytes):
    from PIL import Image
    im = Image.open(io.BytesIO(jpeg_bytes))
    im.draft("YCbCr", im.size)
    im.load()
    return im.mode, np.asarray(im)


def test_444_files_in_a_third_party_decoder_all_three_planes():
    """Without chroma subsampling nothing but the inverse DCT separates the coefficients from the
    YCbCr samples a stock decoder returns: luminance AND both chroma planes agree within one level
    (the two integer transforms round differently), which ties the chroma path of the entropy
    decode and the component order to a third party."""
    rec = _record("444", config=2, n=3)
    for i in range(3):
        W, H = rec.dims[i]
        mode, ycc = _pillow_planes(rec.jpeg(i))
        assert mode == "YCbCr" and ycc.shape == (H, W, 3)
        coef, rgb, (Y, Cb, Cr) = O.jpeg_decode(rec.jpeg(i), want_planes=True)
        for c, plane in enumerate((Y, Cb, Cr)):
            d = np.abs(plane[:H, :W].astype(int) - ycc[:, :, c].astype(int))
            assert d.max() <= 1, (i, c, d.max())
        # and the colour conversion on top: our RGB against the stock decoder's RGB
        from PIL import Image
        ref = np.asarray(Image.open(io.BytesIO(rec.jpeg(i))).convert("RGB")).astype(int)
        assert np.abs(rgb.astype(int) - ref).max() <= 3


def test_grey_files_in_a_third_party_decoder():
    from PIL import Image
    rec = _record("grey", config=2, n=2)
    for i in range(2):
        im = Image.open(io.BytesIO(rec.jpeg(i)))
        assert im.mode == "L"
        ref = np.asarray(im).astype(int)
        _, rgb = O.jpeg_decode(rec.jpeg(i))
        assert np.array_equal(rgb[:, :, 0], rgb[:, :, 1]) and np.array_equal(rgb[:, :, 0], rgb[:, :, 2])
        assert np.abs(rgb[:, :, 0].astype(int) - ref).max() <= 1


@pytest.mark.parametrize("subsampling,samp", [(0, (1, 1, 3)), (1, (2, 1, 3)), (2, (2, 2, 3))])
def test_oracle_decodes_a_third_party_encoder(subsampling, samp):
    """Progressive files written by Pillow with its own tables: the oracle's luminance (and at 4:4:4
    its chroma planes) within one level of Pillow's own decode."""
    from PIL import Image
    spec = pcr_synth.make_specs(2, 0, 1)[0]
    img = Image.fromarray(pcr_synth.image_rgb(spec))
    buf = io.BytesIO()
    img.save(buf, "JPEG", quality=92, progressive=True, subsampling=subsampling, optimize=True)
    data = buf.getvalue()
    W, H, got_samp = O.jpeg_info(data)
    assert got_samp == samp
    mode, ycc = _pillow_planes(data)
    coef, rgb, planes = O.jpeg_decode(data, want_planes=True)
    assert np.abs(planes[0][:H, :W].astype(int) - ycc[:, :, 0].astype(int)).max() <= 1
    if subsampling == 0:
        for c in (1, 2):
            assert np.abs(planes[c][:H, :W].astype(int) - ycc[:, :, c].astype(int)).max() <= 1


def test_oracle_decodes_a_third_party_greyscale_file():
    from PIL import Image
    spec = pcr_synth.make_specs(2, 0, 1)[0]
    img = Image.fromarray(pcr_synth.image_rgb(spec)).convert("L")
    buf = io.BytesIO()
    img.save(buf, "JPEG", quality=90, progressive=True)
    data = buf.getvalue()
    assert O.jpeg_info(data)[2] == (1, 1, 1)
    _, rgb = O.jpeg_decode(data)
    ref = np.asarray(Image.open(io.BytesIO(data))).astype(int)
    assert np.abs(rgb[:, :, 1].astype(int) - ref).max() <= 1


@pytest.mark.parametrize("name", ["444", "422", "440", "420"])
def test_replication_by_the_per_pixel_formula(name):
    """Pixel (x, y) takes chroma sample (x // hs, y // vs): brute force over an odd-sized image."""
    hs, vs, nc = SAMPLINGS[name]
    W, H = 37, 21
    rng = np.random.default_rng(9)
    nb = O.num_blocks(W, H, (hs, vs, nc))
    coef = np.zeros((nb, 64), dtype=np.int16)
    coef[:, 0] = rng.integers(-300, 300, size=nb)
    coef[:, 1:4] = rng.integers(-20, 21, size=(nb, 3))
    q = np.full(64, 2, dtype=np.uint16)
    rgb, (Y, Cb, Cr) = O.pixels_from_coeffs(coef, W, H, q, q, want_planes=True, sampling=(hs, vs, nc))
    for y in range(H):
        for x in range(W):
            want = O.ycc_to_rgb(int(Y[y, x]), int(Cb[y // vs, x // hs]), int(Cr[y // vs, x // hs]))
            assert tuple(int(v) for v in rgb[y, x]) == want, (x, y)


def test_greyscale_pixels_are_the_luminance_samples():
    W, H = 19, 11
    rng = np.random.default_rng(3)
    nb = O.num_blocks(W, H, (1, 1, 1))
    assert nb == 3 * 2
    coef = np.zeros((nb, 64), dtype=np.int16)
    coef[:, 0] = rng.integers(-300, 300, size=nb)
    coef[:, 1:6] = rng.integers(-30, 31, size=(nb, 5))
    q = np.full(64, 3, dtype=np.uint16)
    rgb, (Y,) = O.pixels_from_coeffs(coef, W, H, q, q, want_planes=True, sampling=(1, 1, 1))
    for c in range(3):
        assert np.array_equal(rgb[:, :, c], Y[:H, :W])
    # block by block the samples are the single-block transform
    for b in range(nb):
        by, bx = divmod(b, 3)
        assert np.array_equal(Y[8 * by:8 * by + 8, 8 * bx:8 * bx + 8], O.block_idct(coef[b], q))


def test_scan7_size_of_the_papers_444_example():
    """The paper's printed per-scan sizes for its 600 x 450 example: scan 7 minus scan 6 is one bit per
    block of a 4:4:4 image.  The generator's 4:4:4 file of that size has exactly that DC refinement scan."""
    from helpers import jpeg_segments
    with pcr_synth.sampling(1, 1, 3):
        rec = pcr_synth.record_from_specs([pcr_synth.ImageSpec(600, 450, 0, 90, 2.0, 0.1, 2.0, 0, 0, 5)], restart_rows=False)
    data = rec.jpeg(0)
    sos = [s for s in jpeg_segments(data) if s[0] == 0xDA]
    start = sos[6][1] + sos[6][2]
    ent = data[start:start + sos[6][3]]
    blocks = 3 * 75 * 57
    assert len(ent) - ent.count(b"\xff\x00") == (blocks + 7) // 8
