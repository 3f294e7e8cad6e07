"""Records written without restart markers: every scan of an image is one long entropy-coded
segment (the HAM10000-shaped workload).  Such scans take kernels of their own: first passes are
decoded from 32 speculative entry points that re-synchronise, AC refinements by one chain per warp,
DC refinements bit-parallel.  Here those kernels are compared with the oracle bit for bit at every
fidelity, also on inputs far smaller than the ones they are meant for (the size threshold that
routes a scan to them is lowered through PCR_LONG_MIN_BYTES, read when a record is opened), so that
empty subsequences, blocks shared by neighbouring lanes and images of a single block are covered."""
import numpy as np
import pytest

import pcr_synth
from oracle import pcr_oracle as O

pytestmark = pytest.mark.gpu


def _compare_every_k(rec, min_bytes, monkeypatch):
    import torch
    from paper_1911_00472_b200 import Decoder, pcr_image_blocks
    monkeypatch.setenv("PCR_LONG_MIN_BYTES", str(min_bytes))
    dec = Decoder(rec.bytes)
    monkeypatch.delenv("PCR_LONG_MIN_BYTES")
    try:
        G = dec.n_groups
        for k in range(1, G + 1):
            dec.out = torch.zeros(dec.out_bytes, dtype=torch.uint8, device="cuda")
            out = dec.decode(k)
            torch.cuda.synchronize()
            assert dec.status() == (-1, 0), k
            coef = dec.coeffs().cpu().numpy()
            out_h = out.cpu().numpy()
            for i in range(rec.n_images):
                want_c, want_rgb = O.decode_image(rec.bytes, i, k)
                a, b = pcr_image_blocks(dec.handle, i)
                assert np.array_equal(coef[a:a + b], want_c), (i, k, np.argwhere(coef[a:a + b] != want_c)[:4])
                inf = dec.info[i]
                got = out_h[inf.out_offset:inf.out_offset + inf.out_bytes].reshape(inf.height, inf.width, 3)
                assert np.array_equal(got, want_rgb), (i, k)
        # raising the fidelity scan group by scan group ends at the same pixels
        want = out.clone()
        dec.decode(1)
        for k in range(2, G + 1):
            out = dec.decode_more(k)
        torch.cuda.synchronize()
        assert dec.status() == (-1, 0)
        assert torch.equal(out, want)
    finally:
        dec.close()


@pytest.mark.parametrize("min_bytes", [0, 1 << 20])
def test_ham_shaped_small(rec3_small, min_bytes, monkeypatch):
    _compare_every_k(rec3_small, min_bytes, monkeypatch)


@pytest.mark.parametrize("config", [0, 1, 2])
def test_other_shapes_without_restart_markers(config, monkeypatch):
    rec = pcr_synth.make_record(config, n_images=6, restart_rows=False)
    _compare_every_k(rec, 0, monkeypatch)


@pytest.mark.parametrize("seed", range(6))
def test_random_coefficient_fields_without_restart_markers(seed, monkeypatch):
    rng = np.random.default_rng(300 + seed)
    dims = [(int(rng.integers(1, 200)), int(rng.integers(1, 200))) for _ in range(5)] + [(8, 8), (16, 16), (17, 9), (1, 1), (129, 40), (600, 20)]
    density = [0.02, 0.1, 0.3, 0.6, 0.9, 1.0][seed]
    amp = [1.0, 2.0, 4.0, 20.0, 100.0, 300.0][seed]
    coeffs = []
    for W, H in dims:
        nb = pcr_synth.num_blocks(W, H)
        c = np.zeros((nb, 64), dtype=np.int16)
        m = rng.random((nb, 64)) < density
        mag = np.minimum(np.floor(rng.exponential(amp, size=(nb, 64))) + 1, 1023)
        c[m] = (mag * rng.choice([-1, 1], size=(nb, 64)))[m].astype(np.int16)
        c[:, 0] = rng.integers(-1023, 1024, size=nb)
        coeffs.append(c)
    rec = pcr_synth.record_from_coeffs(dims, coeffs, quality=[90, 50, 95, 100, 75, 90][seed], restart_rows=False)
    _compare_every_k(rec, 0, monkeypatch)


def test_all_zero_and_saturated_streams(monkeypatch):
    """Long end-of-band runs (all-zero AC: a whole scan is a handful of run symbols) and streams
    full of stuffed 0xFF bytes."""
    W, H = 304, 208
    nb = pcr_synth.num_blocks(W, H)
    zero = np.zeros((nb, 64), dtype=np.int16)
    zero[:, 0] = 37
    ones = np.zeros((nb, 64), dtype=np.int16)
    ones[:, 1:] = -1
    big = np.full((nb, 64), 1023, dtype=np.int16)
    sparse = np.zeros((nb, 64), dtype=np.int16)
    sparse[::97, 63] = 5
    sparse[::89, 1] = -3
    rec = pcr_synth.record_from_coeffs([(W, H)] * 4, [zero, ones, big, sparse], restart_rows=False)
    _compare_every_k(rec, 0, monkeypatch)


# four AC refinements of the luminance (the most one call decodes per component), two of each chroma component
SCRIPT_FOUR_LEVELS = [((0, 1, 2), 0, 0, 0, 0), ((0,), 1, 63, 0, 4), ((1,), 1, 63, 0, 2), ((2,), 1, 63, 0, 2),
                      ((0,), 1, 63, 4, 3), ((0,), 1, 63, 3, 2), ((1,), 1, 63, 2, 1), ((2,), 1, 63, 2, 1),
                      ((0,), 1, 63, 2, 1), ((0,), 1, 63, 1, 0), ((1,), 1, 63, 1, 0), ((2,), 1, 63, 1, 0)]


@pytest.mark.parametrize("name", ["spectral4", "mixed6", "deep14", "four_levels"])
def test_other_scripts_without_restart_markers(name, monkeypatch):
    scripts = {"spectral4": pcr_synth.SCRIPT_SPECTRAL_4, "mixed6": pcr_synth.SCRIPT_MIXED_6, "deep14": pcr_synth.SCRIPT_DEEP_14,
               "four_levels": SCRIPT_FOUR_LEVELS}
    with pcr_synth.scan_script(scripts[name]):
        rec = pcr_synth.make_record(3, n_images=2, restart_rows=False)
    _compare_every_k(rec, 0, monkeypatch)


def test_damaged_long_scan_is_flagged_not_fatal(rec3_small):
    """Bytes of a long scan overwritten: the image is flagged (or decodes to something), the call
    returns, other images are untouched, and nothing is written out of bounds."""
    import torch
    from paper_1911_00472_b200 import Decoder
    good = Decoder(rec3_small.bytes)
    want = good.decode(10).clone()
    torch.cuda.synchronize()
    for group, fill in ((2, 0x00), (5, 0xFF), (6, 0xA5), (10, 0x00)):
        dec = Decoder(rec3_small.bytes)
        lo, hi = dec.prefix_bytes(group - 1) if group > 1 else dec.prefix_bytes(1) // 2, dec.prefix_bytes(group)
        # damage the tail of the scan group: the last image's chunk lies there
        a = hi - min(600, (hi - lo) // 4)
        dec.host[a:hi - 16] = fill
        dec.out = torch.zeros(dec.out_bytes, dtype=torch.uint8, device="cuda")
        out = dec.decode(10)
        torch.cuda.synchronize()
        bad, code = dec.status()
        assert code in (0, -3)
        # the first image's chunks were not touched
        inf = dec.info[0]
        assert torch.equal(out[inf.out_offset:inf.out_offset + inf.out_bytes], want[inf.out_offset:inf.out_offset + inf.out_bytes])
        dec.close()
    good.close()


def test_bounded_wait_gives_up_and_the_context_survives(rec0):
    """A refinement warp waits for the warp that decodes the earlier refinement of its component;
    the wait counts its polls.  Pointed at a flag that nothing sets it must end by its limit, the
    kernel must return, and the device must still decode afterwards."""
    import torch
    from paper_1911_00472_b200 import Decoder, binding
    assert binding.pcr_selftest_bounded_wait() is True
    assert binding.strerror(binding.PCR_E_TIMEOUT) == "device-side wait timed out"
    dec = Decoder(rec0.bytes)
    dec.decode(10)
    torch.cuda.synchronize()
    assert dec.status() == (-1, 0)
    dec.close()
