"""GPU parity on the other chroma samplings (4:4:4, 4:2:2, 4:4:0, greyscale): int16 coefficients and
uint8 pixels bit for bit against the oracle at every fidelity, with and without restart markers,
through the kernels for long scans too, on odd sizes, after raising the fidelity, for baseline
(sequential) records and through the training-tensor call."""
import numpy as np
import pytest

import pcr_synth
from oracle import pcr_oracle as O

pytestmark = pytest.mark.gpu

SAMPLINGS = {"444": (1, 1, 3), "422": (2, 1, 3), "440": (1, 2, 3), "grey": (1, 1, 1)}


def _compare_every_k(rec, samp):
    import torch
    from paper_1911_00472_b200 import Decoder, binding, pcr_image_blocks
    dec = Decoder(rec.bytes)
    try:
        assert binding.pcr_get_sampling(dec.handle) == samp
        G = dec.n_groups
        assert G == O.record_info(rec.bytes)[1]
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
                assert b == want_c.shape[0]
                assert np.array_equal(coef[a:a + b], want_c), (i, k, np.argwhere(coef[a:a + b] != want_c)[:4])
                inf = dec.info[i]
                got = out_h[inf.out_offset:inf.out_offset + inf.out_bytes].reshape(inf.height, inf.width, 3)
                assert np.array_equal(got, want_rgb), (i, k, np.argwhere(got != want_rgb)[:4])
        want = out.clone()
        dec.decode(1)
        for k in range(2, G + 1):
            out = dec.decode_more(k)
        torch.cuda.synchronize()
        assert dec.status() == (-1, 0)
        assert torch.equal(out, want)
    finally:
        dec.close()


@pytest.mark.parametrize("name", sorted(SAMPLINGS))
@pytest.mark.parametrize("config", [0, 1, 2])
def test_with_restart_markers(name, config):
    with pcr_synth.sampling(*SAMPLINGS[name]):
        rec = pcr_synth.make_record(config, n_images=5)
    _compare_every_k(rec, SAMPLINGS[name])


@pytest.mark.parametrize("name", sorted(SAMPLINGS))
@pytest.mark.parametrize("min_bytes", [0, 1 << 20])
def test_without_restart_markers(name, min_bytes, monkeypatch):
    with pcr_synth.sampling(*SAMPLINGS[name]):
        rec = pcr_synth.make_record(3, n_images=2, restart_rows=False)
        rec_small = pcr_synth.make_record(0, n_images=4, restart_rows=False)
    monkeypatch.setenv("PCR_LONG_MIN_BYTES", str(min_bytes))
    _compare_every_k(rec, SAMPLINGS[name])
    _compare_every_k(rec_small, SAMPLINGS[name])


@pytest.mark.parametrize("name", sorted(SAMPLINGS))
def test_odd_sizes_and_random_fields(name):
    samp = SAMPLINGS[name]
    rng = np.random.default_rng(11)
    dims = [(1, 1), (8, 8), (9, 17), (17, 9), (16, 16), (31, 33), (129, 40), (300, 20), (255, 257)]
    with pcr_synth.sampling(*samp):
        coeffs = []
        for W, H in dims:
            nb = pcr_synth.num_blocks(W, H)
            c = np.zeros((nb, 64), dtype=np.int16)
            m = rng.random((nb, 64)) < 0.3
            mag = np.minimum(np.floor(rng.exponential(6.0, size=(nb, 64))) + 1, 1023)
            c[m] = (mag * rng.choice([-1, 1], size=(nb, 64)))[m].astype(np.int16)
            c[:, 0] = rng.integers(-1023, 1024, size=nb)
            coeffs.append(c)
        rec = pcr_synth.record_from_coeffs(dims, coeffs, restart_fixed=3, restart_rows=False)
        rec2 = pcr_synth.record_from_coeffs(dims, coeffs)
    _compare_every_k(rec, samp)
    _compare_every_k(rec2, samp)


@pytest.mark.parametrize("name", sorted(SAMPLINGS))
def test_baseline_records(name):
    import torch
    from paper_1911_00472_b200 import Decoder, pcr_image_blocks
    with pcr_synth.sampling(*SAMPLINGS[name]), pcr_synth.scan_script(pcr_synth.SCRIPT_BASELINE):
        recs = [pcr_synth.make_record(2, n_images=4), pcr_synth.make_record(0, n_images=5, restart_rows=False)]
    for rec in recs:
        dec = Decoder(rec.bytes)
        out = dec.decode(1)
        torch.cuda.synchronize()
        assert dec.status() == (-1, 0)
        coef = dec.coeffs().cpu().numpy()
        out_h = out.cpu().numpy()
        for i in range(rec.n_images):
            want_c, want_rgb = O.decode_image(rec.bytes, i, 1)
            a, b = pcr_image_blocks(dec.handle, i)
            assert np.array_equal(coef[a:a + b], want_c) and np.array_equal(want_c, rec.truth(i))
            inf = dec.info[i]
            assert np.array_equal(out_h[inf.out_offset:inf.out_offset + inf.out_bytes].reshape(inf.height, inf.width, 3), want_rgb)
        dec.close()


@pytest.mark.parametrize("name", sorted(SAMPLINGS))
def test_training_tensor_and_refusals(name):
    import torch
    from paper_1911_00472_b200 import Decoder, PcrError, binding
    with pcr_synth.sampling(*SAMPLINGS[name]):
        rec = pcr_synth.make_record(1, n_images=4)
    dec = Decoder(rec.bytes)
    mean, std = (0.485, 0.456, 0.406), (0.229, 0.224, 0.225)
    crops = pcr_synth.random_resized_crops([(int(w), int(h)) for w, h in rec.dims], 5)
    G = dec.n_groups                                   # six scan groups for greyscale, ten otherwise
    t = dec.decode_tensor(G, crops, 96, mean, std, dtype=torch.float32)
    torch.cuda.synchronize()
    assert dec.status() == (-1, 0)
    got = t.cpu().numpy().astype(np.float64)
    for i in range(rec.n_images):
        _, rgb = O.decode_image(rec.bytes, i, G)
        want = O.training_tensor(rgb, crops[i], 96, mean, std, dtype=np.float32).astype(np.float64)
        assert np.abs(got[i] - want).max() <= 1e-5, i
    with pytest.raises(PcrError) as e:                 # the triangle filter is built for 4:2:0
        dec.set_upsampling(True)
    assert e.value.code == binding.PCR_E_ARG
    dec.close()
