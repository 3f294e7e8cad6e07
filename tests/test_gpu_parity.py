"""GPU parity: the CUDA path through the C ABI against the CPU oracle, element by element,
on the same seeded records.  Bit exact: int16 coefficients and uint8 pixels, at every k."""
import numpy as np
import pytest

import pcr_synth
from oracle import pcr_oracle as O

pytestmark = pytest.mark.gpu

G = 10


def _gpu_decode(dec, k):
    import torch
    out = dec.decode(k)
    torch.cuda.synchronize()
    bad, code = dec.status()
    return out, dec.coeffs(), bad, code


def _compare(rec, ks, images=None):
    import torch
    from paper_1911_00472_b200 import Decoder
    dec = Decoder(rec.bytes)
    assert dec.n_images == rec.n_images and dec.n_groups == G
    idx = range(rec.n_images) if images is None else images
    try:
        for k in ks:
            out, coef, bad, code = _gpu_decode(dec, k)
            assert (bad, code) == (-1, 0), (k, bad, code)
            out_h = out.cpu().numpy()
            coef_h = coef.cpu().numpy()
            for i in idx:
                want_c, want_rgb = O.decode_image(rec.bytes, i, k)
                inf = dec.info[i]
                a, b = dec_blocks(dec, i)
                got_c = coef_h[a:a + b]
                assert np.array_equal(got_c, want_c), f"coefficients differ: image {i} k {k}: {np.argwhere(got_c != want_c)[:4]}"
                got = out_h[inf.out_offset:inf.out_offset + inf.out_bytes].reshape(inf.height, inf.width, 3)
                assert np.array_equal(got, want_rgb), f"pixels differ: image {i} k {k}: {np.argwhere(got != want_rgb)[:4]}"
    finally:
        dec.close()


def dec_blocks(dec, i):
    from paper_1911_00472_b200 import pcr_image_blocks
    return pcr_image_blocks(dec.handle, i)


def test_tiny_record_every_k(rec0):
    _compare(rec0, range(1, G + 1))


def test_imagenet_shaped_small(rec1_small):
    _compare(rec1_small, range(1, G + 1))


def test_celeba_shaped_small_unpadded_grid(rec2_small):
    _compare(rec2_small, range(1, G + 1))


def test_ham_shaped_small_no_restarts(rec3_small):
    _compare(rec3_small, (1, 5, 10))


@pytest.mark.parametrize("seed", range(6))
def test_random_coefficient_fields(seed):
    rng = np.random.default_rng(100 + seed)
    dims = [(int(rng.integers(1, 90)), int(rng.integers(1, 90))) for _ in range(6)] + [(8, 8), (16, 16), (17, 9), (1, 1), (129, 40), (300, 20)]
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
    mode = [dict(restart_rows=True), dict(restart_rows=False), dict(restart_rows=False, restart_fixed=1),
            dict(restart_rows=False, restart_fixed=3), dict(restart_rows=True), dict(restart_rows=False, restart_fixed=40)][seed]
    rec = pcr_synth.record_from_coeffs(dims, coeffs, quality=[90, 50, 95, 100, 75, 90][seed], **mode)
    _compare(rec, range(1, G + 1))


def test_stuffed_bytes():
    W, H = 48, 32
    nb = pcr_synth.num_blocks(W, H)
    c = np.zeros((nb, 64), dtype=np.int16)
    c[:, 1:] = -1
    c2 = np.full((nb, 64), 1023, dtype=np.int16)
    c3 = np.full((nb, 64), -1023, dtype=np.int16)
    rec = pcr_synth.record_from_coeffs([(W, H)] * 3, [c, c2, c3])
    _compare(rec, range(1, G + 1))


def test_prefix_property_on_the_device(rec0):
    """Bytes at or beyond the end of scan group k never influence decode(k)."""
    import torch
    from paper_1911_00472_b200 import Decoder
    for k in (1, 4, 7):
        poisoned = rec0.bytes.copy()
        dec0 = Decoder(rec0.bytes)
        pre = dec0.prefix_bytes(k)
        assert pre == O.prefix_bytes(rec0.bytes, k)
        out0, c0, bad, code = _gpu_decode(dec0, k)
        out0 = out0.clone()
        dec0.close()
        # the header/index stay intact (they precede group 1); everything past the prefix is junk
        poisoned[pre:] = 0xA7
        dec1 = Decoder.__new__(Decoder)
        # opening needs the full record's index to validate, so open on the intact bytes and
        # poison the pinned host copy afterwards: the decode copies from that buffer
        dec1.__init__(rec0.bytes)
        dec1.host[pre:] = 0xA7
        out1, c1, bad, code = _gpu_decode(dec1, k)
        assert (bad, code) == (-1, 0)
        assert torch.equal(c0, c1)
        for i in range(rec0.n_images):                     # the images' bytes (the buffer's spare tail is not written)
            assert torch.equal(dec1.image(out0, i), dec1.image(out1, i))
        dec1.close()


def test_incremental_prefix_copy_and_evict(rec0):
    """Raising k copies only the missing groups; evict forces a full copy; results identical."""
    import torch
    from paper_1911_00472_b200 import Decoder
    dec = Decoder(rec0.bytes)
    outs = {}
    for k in (2, 5, 10, 3):
        out, c, bad, code = _gpu_decode(dec, k)
        outs[k] = (out.clone(), c)
    dec.evict()
    for k in (10, 3):
        out, c, bad, code = _gpu_decode(dec, k)
        assert torch.equal(out, outs[k][0]) and torch.equal(c, outs[k][1])
    dec.close()


def test_argument_and_format_errors(rec0):
    import torch
    from paper_1911_00472_b200 import Decoder, PcrError, binding
    dec = Decoder(rec0.bytes)
    out = dec.alloc_out()
    for k in (0, 11, -1):
        with pytest.raises(PcrError) as e:
            binding.pcr_decode(dec.handle, k, out.data_ptr(), 0)
        assert e.value.code == binding.PCR_E_ARG
    with pytest.raises(PcrError) as e:
        binding.pcr_decode(dec.handle, 1, out.data_ptr() + 4, 0)
    assert e.value.code == binding.PCR_E_ARG
    assert dec.prefix_bytes(0) == 0 and dec.prefix_bytes(11) == 0
    dec.close()
    # malformed records: bad magic, truncated, offsets past the end, non-monotone group table
    b = rec0.bytes.copy(); b[0] = ord("X")
    with pytest.raises(PcrError) as e:
        Decoder(b)
    assert e.value.code == binding.PCR_E_FORMAT
    with pytest.raises(PcrError):
        Decoder(rec0.bytes[:len(rec0.bytes) // 2].copy())
    b = rec0.bytes.copy()
    index_off = int(np.frombuffer(b[32:40].tobytes(), dtype="<u8")[0])
    b[index_off + 8:index_off + 16] = np.frombuffer(np.uint64(2 ** 40).tobytes(), dtype=np.uint8)
    with pytest.raises(PcrError):
        Decoder(b)
    # a frame header that disagrees with the record metadata
    b = rec0.bytes.copy()
    meta_off = int(np.frombuffer(b[24:32].tobytes(), dtype="<u8")[0])
    b[meta_off + 4] = 48
    with pytest.raises(PcrError):
        Decoder(b)


def test_corrupt_entropy_data_sets_status_not_a_fault(rec0):
    """Damaged entropy-coded bytes: the decode completes, the image is flagged (or happens to
    decode to something else); neighbouring images are untouched."""
    import torch
    from paper_1911_00472_b200 import Decoder
    ref = Decoder(rec0.bytes)
    good, cgood, _, _ = _gpu_decode(ref, 10)
    good = good.clone()
    b = rec0.bytes.copy()
    # remove image 5's restart markers in scan 10 by overwriting its chunk tail with zeros
    N = rec0.n_images
    index_off = int(np.frombuffer(b[32:40].tobytes(), dtype="<u8")[0])
    ent = index_off + 8 * 11 + 16 * (9 * N + 5)
    off = int(np.frombuffer(b[ent:ent + 8].tobytes(), dtype="<u8")[0])
    ln = int(np.frombuffer(b[ent + 8:ent + 12].tobytes(), dtype="<u4")[0])
    b[off + ln - 30:off + ln] = 0
    dec = Decoder(b)
    out, c, bad, code = _gpu_decode(dec, 10)
    assert bad == 5 and code == -3
    for i in (4, 6):
        inf = dec.info[i]
        assert torch.equal(out[inf.out_offset:inf.out_offset + inf.out_bytes], good[inf.out_offset:inf.out_offset + inf.out_bytes])
    dec.close(); ref.close()


def test_widths_multiple_of_16_odd_heights_dc_only_path():
    """Images 16-pixel aligned in width (the DC-only pixel kernel's condition) with heights that
    end inside an MCU row, random coefficient fields: every k, k = 1 included."""
    rng = np.random.default_rng(7)
    dims = [(48, 37), (16, 1), (64, 100), (32, 8), (496, 23)]
    coeffs = []
    for w, h in dims:
        c = np.zeros((pcr_synth.num_blocks(w, h), 64), dtype=np.int16)
        c[:, 0] = rng.integers(-300, 300, c.shape[0])
        hit = rng.random(c.shape) < 0.08
        hit[:, 0] = False
        c[hit] = rng.integers(-12, 13, int(hit.sum()))
        coeffs.append(c)
    rec = pcr_synth.record_from_coeffs(dims, coeffs)
    _compare(rec, (1, 2, 7, 10))


@pytest.mark.parametrize("slices", ["2", "3"])
def test_sliced_pipelines_on_small_records(monkeypatch, slices, rec1_small, rec2_small):
    """The multi-slice path (image slices on their own streams in width-sorted order, index of the
    later waves on the side stream) on records small enough to compare every image: the slice
    count is read when a record is opened."""
    monkeypatch.setenv("PCR_SLICES", slices)
    _compare(rec1_small, (1, 2, 5, 6, 7, 9, 10))
    _compare(rec2_small, range(1, G + 1))


def test_two_records_in_flight_on_two_streams(monkeypatch, rec1_small, rec2_small):
    """A loader keeps two records in flight (the paper's double buffering): both decodes are enqueued
    on their own streams before either is waited for, each opened from its own host thread."""
    import threading
    import torch
    from paper_1911_00472_b200 import Decoder
    monkeypatch.setenv("PCR_SLICES", "2")
    decs = [None, None]

    def opener(j, rec):
        torch.cuda.set_device(0)
        decs[j] = Decoder(rec.bytes)

    ths = [threading.Thread(target=opener, args=(j, r)) for j, r in enumerate((rec1_small, rec2_small))]
    for t in ths:
        t.start()
    for t in ths:
        t.join()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    try:
        for k in (5, 10):
            outs = [d.decode(k, d.alloc_out(), stream=s) for d, s in zip(decs, streams)]
            torch.cuda.synchronize()
            for d, rec, out in zip(decs, (rec1_small, rec2_small), outs):
                assert d.status() == (-1, 0)
                for i in range(0, rec.n_images, 2):
                    _, want = O.decode_image(rec.bytes, i, k)
                    assert np.array_equal(d.image(out, i).cpu().numpy(), want), (k, i)
    finally:
        for d in decs:
            if d is not None:
                d.close()


def test_record_cache_reopens_the_same_record_and_only_that(rec0, rec1_small):
    """With the cache of closed records on, reopening the same bytes gives a fresh handle that
    decodes to the same result; other bytes, or the same bytes changed in what pcr_open reads, are
    parsed anew."""
    import torch
    from paper_1911_00472_b200 import Decoder, binding
    binding.pcr_set_record_cache(1 << 30)
    try:
        dec = Decoder(rec0.bytes)
        host = dec.host                                   # keep the pinned bytes: the identity includes their address
        dec.out = torch.zeros(dec.out_bytes, dtype=torch.uint8, device="cuda")    # bytes between images are never written
        want = dec.decode(7).clone()
        torch.cuda.synchronize()
        dec.close()
        n0 = binding.pcr_launch_count()
        h = binding.pcr_open(host.data_ptr(), host.numel())      # a hit: no set-up kernel is launched
        assert binding.pcr_launch_count() == n0
        out = torch.zeros_like(want)
        with pytest.raises(binding.PcrError):             # a fresh handle: nothing decoded yet
            binding.pcr_decode_more(h, 9, out.data_ptr(), 0)
        binding.pcr_decode(h, 7, out.data_ptr(), 0)
        torch.cuda.synchronize()
        assert binding.pcr_status(h) == (-1, 0)
        assert torch.equal(out, want)
        binding.pcr_close(h)
        # a label changes (sample metadata is part of what pcr_open reads): parsed anew, new label seen
        host[64] ^= 0x5A
        n1 = binding.pcr_launch_count()
        h = binding.pcr_open(host.data_ptr(), host.numel())
        assert binding.pcr_launch_count() == n1 + 1        # the set-up kernel of a real open
        assert binding.pcr_get_image(h, 0).label == (dec.info[0].label ^ 0x5A)
        binding.pcr_close(h)
        host[64] ^= 0x5A
        # another record is not confused with it
        other = Decoder(rec1_small.bytes)
        assert other.n_images == rec1_small.n_images
        other.close()
    finally:
        binding.pcr_set_record_cache(0)


def test_samples_near_the_end_of_the_32_bit_range():
    """Coefficients no image produces: a luminance DC of 2040 under a quantiser of 128 gives a sample of
    32644 before the level shift, so the second transform pass ends within 128 << 16 of 2^31.  The oracle
    rounds, shifts, adds 128 and clamps (255); a kernel that folds the 128 into the rounding constant
    wraps there (0).  Dense +-1023 fields at odd sizes beside it (4:2:0 and 4:4:0)."""
    import torch
    from paper_1911_00472_b200 import Decoder
    rng = np.random.default_rng(21)
    qy = np.ones(64, dtype=np.uint8); qy[0] = 128
    qc = np.ones(64, dtype=np.uint8)
    for samp in ((2, 2, 3), (1, 2, 3)):
        with pcr_synth.sampling(*samp):
            dims = [(24, 16), (183, 70), (61, 35)]
            coeffs = []
            for n, (w, h) in enumerate(dims):
                nb = pcr_synth.num_blocks(w, h)
                if n == 0:
                    c = np.zeros((nb, 64), dtype=np.int16)
                    c[:, 0] = 2040
                else:
                    c = rng.integers(-1023, 1024, size=(nb, 64)).astype(np.int16)
                coeffs.append(c)
            rec = pcr_synth.record_from_coeffs(dims, coeffs, qtables=(qy, qc))
            rec2 = pcr_synth.record_from_coeffs(dims[1:], coeffs[1:])
        for r in (rec, rec2):
            dec = Decoder(r.bytes)
            try:
                for k in (1, dec.n_groups):
                    out = dec.decode(k).cpu().numpy()
                    assert dec.status() == (-1, 0)
                    for i in range(r.n_images):
                        _, want = O.decode_image(r.bytes, i, k)
                        inf = dec.info[i]
                        got = out[inf.out_offset:inf.out_offset + inf.out_bytes].reshape(inf.height, inf.width, 3)
                        assert np.array_equal(got, want), (samp, i, k, np.argwhere(got != want)[:3])
            finally:
                dec.close()
    _, rgb = O.decode_image(rec.bytes, 0, 10)
    assert rgb[0, 0, 0] == 255          # (the case is the one described: the oracle saturates high)
