"""Pins of the CPU oracle against things other than itself (CPU only).

Each test names what it ties the oracle to: the encoder's ground truth, a closed form,
a third-party JPEG implementation, double-precision arithmetic, or brute force.
"""
import io
import os

import numpy as np
import pytest

import pcr_synth
from oracle import pcr_oracle as O

from helpers import (block_grids, comp_of_block, idct_double, jpeg_segments, mask_truth, pillow_y,
                     zigzag_natural)

G = 10


def _qzz(quality):
    zz = zigzag_natural()
    return pcr_synth.quant_table(quality, False)[zz].astype(np.uint16), pcr_synth.quant_table(quality, True)[zz].astype(np.uint16)


# ---------------------------------------------------------------------------------------
# entropy decode: round trip and the closed-form mask (paper Section 2: scans are disjoint
# deltas holding the same information as sequential JPEG; Section 3: all groups = full data)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("fix", ["rec0", "rec1_small", "rec2_small", "rec3_small"])
def test_full_decode_equals_ground_truth(fix, request):
    rec = request.getfixturevalue(fix)
    for i in range(rec.n_images):
        coef, _ = O.decode_image(rec.bytes, i, G, want_rgb=False)
        assert np.array_equal(coef, rec.truth(i)), f"image {i}"


@pytest.mark.parametrize("fix", ["rec0", "rec1_small", "rec2_small", "rec3_small"])
@pytest.mark.parametrize("k", range(1, G + 1))
def test_truncated_decode_equals_masked_truth(fix, k, request):
    rec = request.getfixturevalue(fix)
    n = rec.n_images if fix == "rec0" else min(rec.n_images, 3)
    for i in range(n):
        W, H = rec.dims[i]
        coef, _ = O.decode_image(rec.bytes, i, k, want_rgb=False)
        want = mask_truth(rec.truth(i), W, H, k)
        assert np.array_equal(coef, want), f"image {i} k {k}"


def _random_coeffs(rng, W, H, density, amp):
    nb = pcr_synth.num_blocks(W, H)
    c = np.zeros((nb, 64), dtype=np.int16)
    m = rng.random((nb, 64)) < density
    mag = np.minimum(np.floor(rng.exponential(amp, size=(nb, 64))) + 1, 1023)
    c[m] = (mag * rng.choice([-1, 1], size=(nb, 64)))[m].astype(np.int16)
    c[:, 0] = rng.integers(-1023, 1024, size=nb)
    return c


@pytest.mark.parametrize("seed", range(6))
def test_random_coefficient_fields_round_trip(seed):
    """Arbitrary (not DCT-derived) coefficient fields, odd sizes, all restart modes."""
    rng = np.random.default_rng(seed)
    dims = [(int(rng.integers(1, 70)), int(rng.integers(1, 70))) for _ in range(5)] + [(8, 8), (16, 16), (17, 9), (1, 1)]
    density = [0.02, 0.1, 0.3, 0.6, 0.9, 1.0][seed]
    amp = [1.0, 2.0, 4.0, 20.0, 100.0, 300.0][seed]
    coeffs = [_random_coeffs(rng, W, H, density, amp) for W, H in dims]
    mode = [dict(restart_rows=True), dict(restart_rows=False), dict(restart_rows=False, restart_fixed=1),
            dict(restart_rows=False, restart_fixed=3), dict(restart_rows=True), dict(restart_rows=False)][seed]
    rec = pcr_synth.record_from_coeffs(dims, coeffs, quality=90, **mode)
    for i, (W, H) in enumerate(dims):
        truth = rec.truth(i)
        for k in (1, 2, 3, 4, 5, 6, 7, 8, 9, 10):
            coef, _ = O.decode_image(rec.bytes, i, k, want_rgb=False)
            assert np.array_equal(coef, mask_truth(truth, W, H, k)), (seed, i, k)


def test_many_stuffed_bytes_round_trip():
    """Coefficient fields chosen so the entropy-coded bytes are full of 0xFF (stuffing path)."""
    rng = np.random.default_rng(11)
    W, H = 48, 32
    nb = pcr_synth.num_blocks(W, H)
    c = np.zeros((nb, 64), dtype=np.int16)
    c[:, 1:] = -1                      # sign bit 0 ... with every coefficient new in the last scans
    c[:, 0] = rng.integers(-5, 5, size=nb)
    c2 = np.full((nb, 64), 1023, dtype=np.int16)
    rec = pcr_synth.record_from_coeffs([(W, H), (W, H)], [c, c2])
    n_ff = int((rec.bytes == 0xFF).sum())
    assert n_ff > 100
    for i in range(2):
        coef, _ = O.decode_image(rec.bytes, i, G, want_rgb=False)
        assert np.array_equal(coef, rec.truth(i))


def test_restart_modes_give_identical_output(rec0):
    """Same coefficients with no restarts, every MCU, every MCU row: same planes and pixels."""
    dims = rec0.dims[:4]
    coeffs = [rec0.truth(i) for i in range(4)]
    outs = []
    for mode in (dict(restart_rows=False), dict(restart_rows=False, restart_fixed=1), dict(restart_rows=True)):
        r = pcr_synth.record_from_coeffs(dims, coeffs, quality=90, **mode)
        outs.append([O.decode_image(r.bytes, i, k) for i in range(4) for k in (1, 5, 6, 10)])
    for a, b in zip(outs[0], outs[1]):
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    for a, b in zip(outs[0], outs[2]):
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


# ---------------------------------------------------------------------------------------
# record semantics (paper Section 3 and Section 5 "Decoding")
# ---------------------------------------------------------------------------------------
def test_reassembled_full_file_is_the_encoders_file(rec0):
    for i in range(rec0.n_images):
        assert O.reassemble(rec0.bytes, i, G) == rec0.jpeg(i)


@pytest.mark.parametrize("k", [1, 4, 7])
def test_prefix_property(rec0, k):
    """decode(k) reads nothing at or beyond the end of scan group k."""
    pre = O.prefix_bytes(rec0.bytes, k)
    poisoned = rec0.bytes.copy()
    poisoned[pre:] = 0xA7
    cut = rec0.bytes[:pre].copy()
    for i in (0, 13, 31):
        a = O.decode_image(rec0.bytes, i, k)
        b = O.decode_image(poisoned, i, k)
        c = O.decode_image(cut, i, k)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
        assert np.array_equal(a[0], c[0]) and np.array_equal(a[1], c[1])
    with pytest.raises(O.OracleError):
        O.decode_image(cut, 0, k + 1)


def test_truncated_files_render_in_a_stock_decoder(rec0):
    """Scans 1..k plus an EOI token parse as a JPEG in a stock decoder, for every k."""
    from PIL import Image
    for k in range(1, G + 1):
        im = Image.open(io.BytesIO(O.reassemble(rec0.bytes, 3, k)))
        im.load()
        assert im.size == rec0.dims[3]


def test_scan_script_and_one_bit_dc_refinement(rec1_small):
    """Ten SOS segments with the expected script; scan 7 carries one bit per block, which is
    also what the paper's printed per-scan file sizes show (golden file)."""
    i = 0
    W, H = rec1_small.dims[i]
    data = rec1_small.jpeg(i)
    sos = [(off, ln, ent) for (mk, off, ln, ent) in jpeg_segments(data) if mk == 0xDA]
    assert len(sos) == 10
    script = []
    for off, ln, ent in sos:
        ns = data[off]
        comps = tuple(data[off + 1 + 2 * j] for j in range(ns))
        ss, se, ahal = data[off + 1 + 2 * ns], data[off + 2 + 2 * ns], data[off + 3 + 2 * ns]
        script.append((comps, ss, se, ahal >> 4, ahal & 15))
    assert script == [((1, 2, 3), 0, 0, 0, 1), ((1,), 1, 5, 0, 2), ((3,), 1, 63, 0, 1), ((2,), 1, 63, 0, 1),
                      ((1,), 6, 63, 0, 2), ((1,), 1, 63, 2, 1), ((1, 2, 3), 0, 0, 1, 0), ((3,), 1, 63, 1, 0),
                      ((2,), 1, 63, 1, 0), ((1,), 1, 63, 1, 0)]
    mx, my = (W + 15) // 16, (H + 15) // 16
    # one MCU row = 6*mx bits, byte padded, plus a 2-byte RST marker between rows
    start = sos[6][0] + sos[6][1]
    stuffed = data[start:start + sos[6][2]].count(b"\xff\x00")
    assert sos[6][2] - stuffed == my * ((6 * mx + 7) // 8) + 2 * (my - 1)
    # the paper's numbers: scan7 - scan6 equals blocks/8 bytes for the two images whose size is known
    rows = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_scan_sizes.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            t = line.split()
            rows[t[0]] = (int(t[1]), int(t[2]), t[3], [float(v) for v in t[4:]])
    w, h, samp, s = rows["celebahq"]
    blocks = (w // 8) * (h // 8) * 3 // 2          # 4:2:0
    assert abs((s[6] - s[5]) * 1024 - blocks / 8) < 0.1 * 1024 + 64   # two sizes printed to 0.1 KiB, plus headers
    w, h, samp, s = rows["ham10000"]
    blocks = 3 * ((w + 7) // 8) * ((h + 7) // 8)   # 4:4:4
    assert abs((s[6] - s[5]) * 1024 - blocks / 8) < 0.1 * 1024 + 64


def test_size_ratio_shape_of_the_paper_tables(rec1_small):
    """Table 1 of the paper: the ratio full size / size of the prefix up to scan group k falls with
    k and is 1 at k = 10 for every data set.  The synthetic record has the same shape (its values
    are reported by the benchmark, not asserted: the content recipe is not the paper's data)."""
    rows = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_tables.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            t = line.split()
            rows[t[0]] = [float(v) for v in t[1:5]]
    assert set(rows) == {"imagenet", "ham10000", "cars", "celebahq"}
    for name, r in rows.items():
        assert r[0] > r[1] > r[2] > r[3] == 1.0, name
    rec = rec1_small.bytes
    data0 = O.prefix_bytes(rec, 1) - sum(len(O.reassemble(rec, i, 1)) - 2 for i in range(rec1_small.n_images))
    full = O.prefix_bytes(rec, 10) - data0          # scan-group bytes without header and index
    ratios = [full / (O.prefix_bytes(rec, k) - data0) for k in (1, 2, 5, 10)]
    assert ratios[0] > ratios[1] > ratios[2] > ratios[3] == 1.0
    assert ratios[0] > 4.0                          # the first scan group is a small fraction of the image


def test_quant_tables_match_a_stock_encoder():
    """The typed-in base tables and the quality scaling agree with a stock encoder's tables."""
    from PIL import Image
    zz = zigzag_natural()
    for q in (50, 75, 90, 95):
        buf = io.BytesIO()
        Image.new("RGB", (16, 16)).save(buf, "JPEG", quality=q)
        im = Image.open(io.BytesIO(buf.getvalue()))
        t = im.quantization
        mine_y, mine_c = pcr_synth.quant_table(q, False), pcr_synth.quant_table(q, True)
        # Pillow returns tables in natural order on recent versions, zigzag on older ones
        ty, tc = np.array(t[0]), np.array(t[1])
        assert np.array_equal(ty, mine_y) or np.array_equal(ty, mine_y[zz])
        assert np.array_equal(tc, mine_c) or np.array_equal(tc, mine_c[zz])
    assert pcr_synth.quant_table(90, False)[0] == 3 and pcr_synth.quant_table(95, False)[0] == 2


# ---------------------------------------------------------------------------------------
# third-party cross checks, both directions (guards against encoder and oracle sharing a
# misreading of the stream syntax)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("fix", ["rec0", "rec1_small", "rec2_small", "rec3_small"])
def test_stock_decoder_luminance_agrees(fix, request):
    rec = request.getfixturevalue(fix)
    for i in range(min(rec.n_images, 4)):
        W, H = rec.dims[i]
        _, _, (Y, _, _) = O.jpeg_decode(O.reassemble(rec.bytes, i, G), want_planes=True)
        ref = pillow_y(rec.jpeg(i))
        d = np.abs(Y[:H, :W].astype(int) - ref.astype(int))
        assert d.max() <= 1, f"image {i}: {d.max()}"


@pytest.mark.parametrize("restart_rows", [0, 1, 2])
@pytest.mark.parametrize("size", [(64, 64), (178, 218), (33, 17)])
def test_oracle_decodes_stock_encoder_streams(restart_rows, size):
    """A stock encoder's progressive stream (its own tables and restart intervals)."""
    from PIL import Image
    spec = pcr_synth.ImageSpec(size[0], size[1], 0, 90, 1.0, 0.3, 4.0, 0, 0, 1234 + restart_rows)
    rgb = pcr_synth.image_rgb(spec)
    buf = io.BytesIO()
    kw = dict(restart_marker_rows=restart_rows) if restart_rows else {}
    Image.fromarray(rgb).save(buf, "JPEG", quality=90, progressive=True, subsampling=2, optimize=True, **kw)
    data = buf.getvalue()
    assert sum(1 for s in jpeg_segments(data) if s[0] == 0xDA) == 10
    _, _, (Y, _, _) = O.jpeg_decode(data, want_planes=True)
    ref = pillow_y(data)
    d = np.abs(Y[:size[1], :size[0]].astype(int) - ref.astype(int))
    assert d.max() <= 1


# ---------------------------------------------------------------------------------------
# pixels: inverse DCT, constants, colour, upsampling, crop
# ---------------------------------------------------------------------------------------
def test_idct_within_one_of_double_precision():
    rng = np.random.default_rng(5)
    qy, qc = _qzz(90)
    worst = 0.0
    for t in range(400):
        q = qy if t % 2 == 0 else qc
        # a legal block: quantised forward transform of random samples
        s = rng.integers(0, 256, size=(8, 8)).astype(np.float64) if t % 3 else rng.choice([0, 255], size=(8, 8)).astype(np.float64)
        n = np.arange(8)
        B = np.cos((2 * n[:, None] + 1) * n[None, :] * np.pi / 16) * np.where(n[None, :] == 0, np.sqrt(0.5), 1.0) * 0.5
        F = B.T @ (s - 128.0) @ B
        zz = zigzag_natural()
        coef = np.rint(F.reshape(64)[zz] / q).astype(np.int16)
        got = O.block_idct(coef, q).astype(np.float64)
        ref = np.clip(idct_double(coef, q), 0, 255)
        worst = max(worst, np.abs(got - ref).max())
    assert worst <= 1.0, worst


def test_idct_dc_only_and_zero_block_closed_form():
    q = np.ones(64, dtype=np.uint16)
    assert np.all(O.block_idct(np.zeros(64, np.int16), q) == 128)
    for c in range(-128, 128):
        coef = np.zeros(64, np.int16)
        coef[0] = 8 * c                      # gain of the DC term is 1/8
        assert np.all(O.block_idct(coef, q) == c + 128), c
    # one basis function against double precision, all positions
    for k in range(64):
        coef = np.zeros(64, np.int16)
        coef[k] = 100
        assert np.abs(O.block_idct(coef, q) - np.clip(idct_double(coef, q), 0, 255)).max() <= 1


def test_idct_is_not_transposed():
    """A horizontal-frequency coefficient must vary along x only (guards a transposed operand)."""
    q = np.ones(64, dtype=np.uint16)
    coef = np.zeros(64, np.int16)
    coef[1] = 200                            # zigzag 1 = row 0, column 1 = horizontal frequency
    out = O.block_idct(coef, q).astype(int)
    assert np.all(out == out[0:1, :]) and out[0, 0] > out[0, 7]
    coef[:] = 0
    coef[2] = 200                            # zigzag 2 = row 1, column 0 = vertical frequency
    out = O.block_idct(coef, q).astype(int)
    assert np.all(out == out[:, 0:1]) and out[0, 0] > out[7, 0]


@pytest.mark.parametrize("grey", [128, 131, 200, 17, 255, 0])
def test_constant_images_reproduce_their_constant(grey):
    """A constant image is DC-only; with DC quantiser 3 (quality 90) the decode returns the
    constant exactly when 8*(g-128) is a multiple of 3, at full fidelity; before the DC
    refinement (k < 7) it returns the constant of the floor-halved DC."""
    W, H = 40, 24
    rgb = np.full((H, W, 3), grey, dtype=np.uint8)
    coef = pcr_synth.rgb_to_coeffs(rgb, 90)
    assert np.all(coef[:, 1:] == 0)
    rec = pcr_synth.record_from_coeffs([(W, H)], [coef], quality=90)
    qdc = 3
    dc = int(coef[0, 0])
    for k in range(1, G + 1):
        c, out = O.decode_image(rec.bytes, 0, k)
        dck = dc if k >= 7 else (dc >> 1) << 1
        val = dck * qdc / 8.0 + 128
        expect = int(np.clip(np.floor(val + 0.5), 0, 255))
        assert np.all(out == expect), (k, grey, out[0, 0], expect)
        if k >= 7 and (8 * (grey - 128)) % qdc == 0:
            assert expect == grey


def test_colour_cube_against_double_precision():
    Y, Cb, Cr = np.meshgrid(np.arange(256), np.arange(256), np.arange(0, 256), indexing="ij")
    ycc = np.stack([Y.ravel(), Cb.ravel(), Cr.ravel()], axis=1).astype(np.uint8)
    got = O.ycc_to_rgb_array(ycc).astype(np.float64)
    y, cb, cr = ycc[:, 0].astype(np.float64), ycc[:, 1].astype(np.float64) - 128, ycc[:, 2].astype(np.float64) - 128
    ref = np.stack([y + 1.402 * cr, y - 0.344136 * cb - 0.714136 * cr, y + 1.772 * cb], axis=1)
    ref = np.clip(ref, 0, 255)
    assert np.abs(got - ref).max() <= 1.0
    grey = ycc[(ycc[:, 1] == 128) & (ycc[:, 2] == 128)]
    out = O.ycc_to_rgb_array(grey)
    assert np.array_equal(out, np.repeat(grey[:, :1], 3, axis=1))
    # a few hand-computed points (guards swapped channels / wrong sign)
    assert O.ycc_to_rgb(128, 128, 255) == (255, 37, 128)      # strong Cr -> red up, green down
    assert O.ycc_to_rgb(128, 255, 128) == (128, 84, 255)      # strong Cb -> blue up, green down


@pytest.mark.parametrize("size", [(17, 9), (1, 1), (8, 8), (16, 16), (31, 33)])
def test_upsample_and_crop_brute_force(size):
    """RGB(x, y) comes from Y(x, y) and the chroma sample at (x >> 1, y >> 1), cropped to W x H."""
    W, H = size
    spec = pcr_synth.ImageSpec(W, H, 0, 90, 1.0, 0.8, 4.0, 0, 0, 99)
    rec = pcr_synth.record_from_specs([spec])
    _, rgb, (Y, Cb, Cr) = O.jpeg_decode(rec.jpeg(0), want_planes=True)
    assert rgb.shape == (H, W, 3)
    for y in range(H):
        for x in range(W):
            assert tuple(rgb[y, x]) == O.ycc_to_rgb(Y[y, x], Cb[y >> 1, x >> 1], Cr[y >> 1, x >> 1])


def test_full_decode_equals_sequential_decode_of_same_coefficients(rec1_small):
    """All scan groups == pixels computed directly from the ground-truth coefficients."""
    qy, qc = _qzz(90)
    for i in range(3):
        W, H = rec1_small.dims[i]
        _, rgb = O.decode_image(rec1_small.bytes, i, G)
        assert np.array_equal(rgb, O.pixels_from_coeffs(rec1_small.truth(i), W, H, qy, qc))


def test_padding_only_blocks_never_get_ac(rec2_small):
    """178x218: the 24th luminance block column exists only as MCU padding."""
    W, H = rec2_small.dims[0]
    mx, my, padded, off = block_grids(W, H)
    coef, _ = O.decode_image(rec2_small.bytes, 0, G, want_rgb=False)
    ycoef = coef[:off[1]].reshape(padded[0][1], padded[0][0], 64)
    assert (W + 7) // 8 == 23 and padded[0][0] == 24
    assert np.all(ycoef[:, 23, 1:] == 0) and np.any(ycoef[:, 23, 0] != 0)


# ---------------------------------------------------------------------------------------
# malformed input is an error, not a crash
# ---------------------------------------------------------------------------------------
def test_malformed_records_are_rejected(rec0):
    b = rec0.bytes.copy()
    b[0] = ord("X")
    with pytest.raises(O.OracleError):
        O.record_info(b)
    with pytest.raises(O.OracleError):
        O.decode_image(rec0.bytes, 0, 11)
    with pytest.raises(O.OracleError):
        O.decode_image(rec0.bytes, 32, 1)
    # flip entropy-coded bytes of image 0's first scan: either an error or a different result, never a crash
    pre0 = O.prefix_bytes(rec0.bytes, 1)
    c = rec0.bytes.copy()
    c[pre0 - 40:pre0 - 20] ^= 0x5A
    try:
        O.decode_image(c, rec0.n_images - 1, 1)
    except O.OracleError:
        pass
