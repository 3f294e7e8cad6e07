"""Other scan scripts than the ten-scan default (the paper, Section 4.2: scans that are not used
can be left out; a record is one scan per group whatever the script).  The oracle is pinned on
them against the generator's ground truth and the script's own meaning; the CUDA path is then
compared with the oracle at every fidelity."""
import numpy as np
import pytest

import pcr_synth
from oracle import pcr_oracle as O

from helpers import mask_truth, mask_truth_script

SCRIPTS = {"spectral4": pcr_synth.SCRIPT_SPECTRAL_4, "mixed6": pcr_synth.SCRIPT_MIXED_6, "deep14": pcr_synth.SCRIPT_DEEP_14}
TEN = [((0, 1, 2), 0, 0, 0, 1), ((0,), 1, 5, 0, 2), ((2,), 1, 63, 0, 1), ((1,), 1, 63, 0, 1), ((0,), 6, 63, 0, 2),
       ((0,), 1, 63, 2, 1), ((0, 1, 2), 0, 0, 1, 0), ((2,), 1, 63, 1, 0), ((1,), 1, 63, 1, 0), ((0,), 1, 63, 1, 0)]


def _record(name, config=2, n=3, **kw):
    with pcr_synth.scan_script(SCRIPTS[name]):
        return pcr_synth.make_record(config, n_images=n, **kw)


def test_general_mask_agrees_with_the_ten_scan_closed_form(rec2_small):
    W, H = rec2_small.dims[0]
    t = rec2_small.truth(0)
    for k in range(1, 11):
        assert np.array_equal(mask_truth_script(t, W, H, TEN, k), mask_truth(t, W, H, k))


@pytest.mark.parametrize("name", sorted(SCRIPTS))
def test_oracle_on_other_scripts_every_k(name):
    rec = _record(name)
    n, G = O.record_info(rec.bytes)
    assert G == len(SCRIPTS[name])
    for i in range(n):
        W, H = rec.dims[i]
        for k in range(1, G + 1):
            got = O.decode_image(rec.bytes, i, k, False)
            got = got[0] if isinstance(got, tuple) else got
            assert np.array_equal(got, mask_truth_script(rec.truth(i), W, H, SCRIPTS[name], k)), (name, i, k)


@pytest.mark.parametrize("name", sorted(SCRIPTS))
def test_oracle_other_scripts_without_restart_markers(name):
    rec = _record(name, config=0, n=4, restart_rows=False)
    _, G = O.record_info(rec.bytes)
    for i in range(4):
        got = O.decode_image(rec.bytes, i, G, False)
        got = got[0] if isinstance(got, tuple) else got
        assert np.array_equal(got, rec.truth(i))


@pytest.mark.gpu
@pytest.mark.parametrize("name", sorted(SCRIPTS))
@pytest.mark.parametrize("restart_rows", [True, False])
def test_gpu_other_scripts_every_k(name, restart_rows):
    import torch
    from paper_1911_00472_b200 import Decoder, pcr_image_blocks
    rec = _record(name, config=2, n=5, restart_rows=restart_rows)
    dec = Decoder(rec.bytes)
    try:
        G = dec.n_groups
        assert G == len(SCRIPTS[name])
        for k in range(1, G + 1):
            out = dec.decode(k)
            torch.cuda.synchronize()
            assert dec.status() == (-1, 0), (name, k)
            coef = dec.coeffs().cpu().numpy()
            out_h = out.cpu().numpy()
            for i in range(rec.n_images):
                want_c, want_rgb = O.decode_image(rec.bytes, i, k)
                a, b = pcr_image_blocks(dec.handle, i)
                assert np.array_equal(coef[a:a + b], want_c), (name, i, k)
                inf = dec.info[i]
                got = out_h[inf.out_offset:inf.out_offset + inf.out_bytes].reshape(inf.height, inf.width, 3)
                assert np.array_equal(got, want_rgb), (name, i, k)
        # raising the fidelity step by step ends at the same pixels
        dec.decode(1)
        for k in range(2, G + 1):
            out = dec.decode_more(k)
        torch.cuda.synchronize()
        full = dec.decode(G, dec.alloc_out())
        torch.cuda.synchronize()
        for i in range(rec.n_images):
            assert torch.equal(dec.image(out, i), dec.image(full, i)), (name, i)
    finally:
        dec.close()


# ---- baseline (sequential) JPEG records: the paper's Table 2 compares progressive decoding with it
def _baseline(config, n, **kw):
    with pcr_synth.scan_script(pcr_synth.SCRIPT_BASELINE):
        return pcr_synth.make_record(config, n_images=n, **kw)


@pytest.mark.parametrize("config,restart_rows", [(0, True), (2, True), (2, False), (3, False)])
def test_oracle_on_baseline_records_matches_ground_truth(config, restart_rows):
    rec = _baseline(config, 3, restart_rows=restart_rows)
    n, G = O.record_info(rec.bytes)
    assert G == 1
    for i in range(n):
        got, _ = O.decode_image(rec.bytes, i, 1)
        assert np.array_equal(got, rec.truth(i))


def test_baseline_files_cross_checked_with_pillow():
    """Pillow decodes this generator's baseline files and the oracle decodes Pillow's: luminance
    planes within one level both ways (chroma upsampling differs by design, luminance does not)."""
    PIL = pytest.importorskip("PIL.Image")
    import io
    from helpers import pillow_y
    rec = _baseline(2, 2)
    for i in range(2):
        jpg = rec.jpeg(i)
        assert not PIL.open(io.BytesIO(jpg)).info.get("progressive")
        W, H = rec.dims[i]
        _, _, (Y, _, _) = O.jpeg_decode(jpg, want_planes=True)
        assert np.abs(pillow_y(jpg).astype(int) - Y[:H, :W].astype(int)).max() <= 1
    rng = np.random.default_rng(3)
    img = np.clip(np.cumsum(rng.normal(0, 4, (70, 90, 3)), axis=1) + 128, 0, 255).astype(np.uint8)
    for opt, rst in ((True, 0), (False, 0), (True, 1)):
        buf = io.BytesIO()
        kw = {"restart_marker_rows": rst} if rst else {}
        PIL.fromarray(img).save(buf, "JPEG", quality=90, subsampling=2, progressive=False, optimize=opt, **kw)
        jpg = buf.getvalue()
        _, _, (Y, _, _) = O.jpeg_decode(jpg, want_planes=True)
        assert np.abs(pillow_y(jpg).astype(int) - Y[:70, :90].astype(int)).max() <= 1


@pytest.mark.gpu
@pytest.mark.parametrize("config,n,restart_rows", [(0, 32, True), (1, 6, True), (2, 5, True), (2, 5, False), (3, 2, False)])
def test_gpu_baseline_records(config, n, restart_rows):
    """A record of baseline JPEGs (one scan group): coefficients and pixels bit-equal to the oracle,
    and the training-tensor path on top of it."""
    import torch
    from paper_1911_00472_b200 import Decoder, pcr_image_blocks
    rec = _baseline(config, n, restart_rows=restart_rows)
    dec = Decoder(rec.bytes)
    try:
        assert dec.n_groups == 1
        out = dec.decode(1)
        torch.cuda.synchronize()
        assert dec.status() == (-1, 0)
        coef = dec.coeffs().cpu().numpy()
        out_h = out.cpu().numpy()
        for i in range(rec.n_images):
            want_c, want_rgb = O.decode_image(rec.bytes, i, 1)
            a, b = pcr_image_blocks(dec.handle, i)
            assert np.array_equal(coef[a:a + b], want_c), (config, i)
            inf = dec.info[i]
            got = out_h[inf.out_offset:inf.out_offset + inf.out_bytes].reshape(inf.height, inf.width, 3)
            assert np.array_equal(got, want_rgb), (config, i)
        crops = pcr_synth.random_resized_crops([(int(w), int(h)) for w, h in rec.dims], 31)
        mean, std = (0.485, 0.456, 0.406), (0.229, 0.224, 0.225)
        t = dec.decode_tensor(1, crops, 24, mean, std)
        torch.cuda.synchronize()
        got_t = t.cpu().numpy().astype(np.float64)
        for i in range(0, rec.n_images, 3):
            _, rgb = O.decode_image(rec.bytes, i, 1)
            want = O.training_tensor(rgb, crops[i], 24, mean, std).astype(np.float64)
            assert np.abs(got_t[i] - want).max() <= 2.0 ** -9, (config, i)
    finally:
        dec.close()


@pytest.mark.gpu
def test_gpu_baseline_record_with_damaged_bytes_is_flagged():
    """Damaged entropy-coded bytes in a baseline record: the decode completes, the image is flagged,
    its neighbours are untouched."""
    import torch
    from paper_1911_00472_b200 import Decoder
    rec = _baseline(0, 32)
    ref = Decoder(rec.bytes)
    good = ref.decode(1).clone()
    torch.cuda.synchronize()
    b = rec.bytes.copy()
    N = rec.n_images
    index_off = int(np.frombuffer(b[32:40].tobytes(), dtype="<u8")[0])
    ent = index_off + 8 * 2 + 16 * (0 * N + 5)                 # chunk (group 1, image 5)
    off = int(np.frombuffer(b[ent:ent + 8].tobytes(), dtype="<u8")[0])
    ln = int(np.frombuffer(b[ent + 8:ent + 12].tobytes(), dtype="<u4")[0])
    b[off + ln - 40:off + ln] = 0                              # wipes the last restart marker and the data around it
    dec = Decoder(b)
    try:
        out = dec.decode(1)
        torch.cuda.synchronize()
        bad, code = dec.status()
        assert bad == 5 and code == -3
        for i in (4, 6):
            inf = dec.info[i]
            assert torch.equal(out[inf.out_offset:inf.out_offset + inf.out_bytes], good[inf.out_offset:inf.out_offset + inf.out_bytes])
    finally:
        dec.close(); ref.close()
