"""Randomised records against the oracle: scan script, chroma sampling, image sizes, restart-marker
layout, the statistics of the coefficient field and the fidelities are drawn from a seed; int16
coefficients and uint8 pixels must agree bit for bit, also after raising the fidelity of a resident
decode.  The fields include ones no encoder produces (dense +-1023, one block repeated, symbols of
one length): they reach the wrap-around ends of the fixed-point arithmetic and streams that do not
re-synchronise."""
import contextlib
import os

import numpy as np
import pytest

import pcr_synth
from oracle import pcr_oracle as O

pytestmark = pytest.mark.gpu

FOUR_LEVELS = [((0, 1, 2), 0, 0, 0, 0), ((0,), 1, 63, 0, 4), ((1,), 1, 63, 0, 2), ((2,), 1, 63, 0, 2),
               ((0,), 1, 63, 4, 3), ((0,), 1, 63, 3, 2), ((1,), 1, 63, 2, 1), ((2,), 1, 63, 2, 1),
               ((0,), 1, 63, 2, 1), ((0,), 1, 63, 1, 0), ((1,), 1, 63, 1, 0), ((2,), 1, 63, 1, 0)]
SCRIPTS = [None, pcr_synth.SCRIPT_DEEP_14, FOUR_LEVELS, pcr_synth.SCRIPT_MIXED_6, pcr_synth.SCRIPT_SPECTRAL_4, pcr_synth.SCRIPT_BASELINE]
SAMPLINGS = [(2, 2, 3), (2, 2, 3), (1, 1, 3), (2, 1, 3), (1, 2, 3), (1, 1, 1)]


def _field(rng, nb, kind):
    if kind == 0:      # sparse, like an image's
        c = (rng.integers(-60, 61, size=(nb, 64)) * (rng.random((nb, 64)) < rng.uniform(0.02, 0.4))).astype(np.int16)
    elif kind == 1:    # dense small values: symbols of one length
        c = rng.integers(-3, 4, size=(nb, 64)).astype(np.int16)
    elif kind == 2:    # dense and as large as the format allows
        c = rng.integers(-1023, 1024, size=(nb, 64)).astype(np.int16)
    elif kind == 3:    # the same block everywhere
        c = np.tile(rng.integers(-9, 10, size=64), (nb, 1)).astype(np.int16)
    else:              # empty but for rare spikes
        c = np.zeros((nb, 64), dtype=np.int16)
        idx = rng.integers(0, nb, size=max(1, nb // 50))
        c[idx, rng.integers(0, 64, size=idx.size)] = rng.integers(-500, 500, size=idx.size)
    if kind != 3:
        c[:, 0] = rng.integers(-800, 800, size=nb)
    return c


def _one(seed, monkeypatch):
    import torch
    from paper_1911_00472_b200 import Decoder, pcr_image_blocks
    rng = np.random.default_rng(seed)
    script = SCRIPTS[rng.integers(0, len(SCRIPTS))]
    samp = SAMPLINGS[rng.integers(0, len(SAMPLINGS))]
    n = int(rng.integers(1, 7))
    dims = [(int(rng.integers(1, 260)), int(rng.integers(1, 200))) for _ in range(n)]
    if rng.random() < 0.3:
        dims[0] = (int(rng.integers(300, 700)), int(rng.integers(200, 500)))
    restart_rows = bool(rng.random() < 0.4)
    restart_fixed = 0 if restart_rows else int(rng.choice([0, 0, 0, 1, 5, 40]))
    cm = pcr_synth.scan_script(script) if script is not None else contextlib.nullcontext()
    with cm, pcr_synth.sampling(*samp):
        coeffs = [_field(rng, pcr_synth.num_blocks(w, h), int(rng.integers(0, 5))) for w, h in dims]
        rec = pcr_synth.record_from_coeffs(dims, coeffs, restart_rows=restart_rows, restart_fixed=restart_fixed)
    monkeypatch.setenv("PCR_LONG_MIN_BYTES", str(int(rng.choice([0, 64, 64, 1 << 20]))))
    dec = Decoder(rec.bytes)
    monkeypatch.delenv("PCR_LONG_MIN_BYTES")
    try:
        G = dec.n_groups
        for k in sorted(set([1, G] + [int(x) for x in rng.integers(1, G + 1, size=2)])):
            dec.out = torch.zeros(dec.out_bytes, dtype=torch.uint8, device="cuda")
            out = dec.decode(k)
            torch.cuda.synchronize()
            assert dec.status() == (-1, 0), (seed, k)
            coef = dec.coeffs().cpu().numpy()
            out_h = out.cpu().numpy()
            for i in range(rec.n_images):
                want_c, want_rgb = O.decode_image(rec.bytes, i, k)
                a, b = pcr_image_blocks(dec.handle, i)
                assert np.array_equal(coef[a:a + b], want_c), (seed, i, k)
                inf = dec.info[i]
                got = out_h[inf.out_offset:inf.out_offset + inf.out_bytes].reshape(inf.height, inf.width, 3)
                assert np.array_equal(got, want_rgb), (seed, i, k, np.argwhere(got != want_rgb)[:3])
        k0 = int(rng.integers(1, G + 1))
        dec.decode(k0)
        out2 = (dec.decode_more(G) if k0 < G else dec.decode(G)).cpu().numpy()
        assert dec.status() == (-1, 0)
        for i in range(rec.n_images):
            _, want_rgb = O.decode_image(rec.bytes, i, G)
            inf = dec.info[i]
            got = out2[inf.out_offset:inf.out_offset + inf.out_bytes].reshape(inf.height, inf.width, 3)
            assert np.array_equal(got, want_rgb), (seed, i, "raised from", k0)
    finally:
        dec.close()


@pytest.mark.parametrize("first", [0, 60, 120])
def test_random_records(first, monkeypatch):
    for seed in range(first, first + 60):
        _one(seed, monkeypatch)
