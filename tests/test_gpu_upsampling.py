"""GPU parity of triangle chroma upsampling (pcr_set_upsampling) against the oracle: bit exact."""
import numpy as np
import pytest

import pcr_synth
from oracle import pcr_oracle as O

pytestmark = pytest.mark.gpu


def _check(rec, ks, images=None):
    import torch
    from paper_1911_00472_b200 import Decoder
    dec = Decoder(rec.bytes)
    try:
        dec.set_upsampling(True)
        for k in ks:
            out = dec.decode(k)
            torch.cuda.synchronize()
            assert dec.status() == (-1, 0)
            for i in (range(rec.n_images) if images is None else images):
                _, want = O.decode_image_upsampled(rec.bytes, i, k, True)
                assert np.array_equal(dec.image(out, i).cpu().numpy(), want), (k, i)
        # back to replication: the plain decode again
        dec.set_upsampling(False)
        out = dec.decode(ks[-1])
        torch.cuda.synchronize()
        _, want = O.decode_image(rec.bytes, 0, ks[-1])
        assert np.array_equal(dec.image(out, 0).cpu().numpy(), want)
    finally:
        dec.close()


def test_tiny_record_every_k(rec0):
    _check(rec0, list(range(1, 11)))


def test_imagenet_and_celeba_shaped(rec1_small, rec2_small):
    _check(rec1_small, [1, 2, 5, 10], range(0, rec1_small.n_images, 3))
    _check(rec2_small, [2, 6, 10])


def test_sliced_record_and_fidelity_raise(monkeypatch, rec2_small):
    import torch
    from paper_1911_00472_b200 import Decoder, PcrError
    monkeypatch.setenv("PCR_SLICES", "2")
    dec = Decoder(rec2_small.bytes)
    try:
        dec.set_upsampling(True)
        dec.decode(3)
        out = dec.decode_more(10)
        torch.cuda.synchronize()
        for i in range(rec2_small.n_images):
            _, want = O.decode_image_upsampled(rec2_small.bytes, i, 10, True)
            assert np.array_equal(dec.image(out, i).cpu().numpy(), want), i
        crops = pcr_synth.random_resized_crops([(int(w), int(h)) for w, h in rec2_small.dims], 1)
        with pytest.raises(PcrError):
            dec.decode_tensor(10, crops, 8, (0.5, 0.5, 0.5), (0.2, 0.2, 0.2))
    finally:
        dec.close()
