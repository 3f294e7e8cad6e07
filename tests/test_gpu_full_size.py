"""GPU parity at the full sizes of the workloads, in the launch configuration the benchmark
times (default image slices and streams): every image's coefficients against the generator's
ground truth at full fidelity, and sampled images against the oracle (coefficients and pixels,
bit exact) at the scan groups each workload names."""
import numpy as np
import pytest

import pcr_synth
from oracle import pcr_oracle as O

from helpers import mask_truth

pytestmark = pytest.mark.gpu


def _check(config, ks, n_sample, full_truth_k=10):
    import torch
    from paper_1911_00472_b200 import Decoder, pcr_image_blocks
    rec = pcr_synth.make_record(config, 0)
    assert rec.n_images == pcr_synth.WORKLOADS[config].images_per_record
    dec = Decoder(rec.bytes)
    rng = np.random.default_rng(config)
    sample = sorted(set([0, rec.n_images - 1] + [int(v) for v in rng.integers(0, rec.n_images, n_sample)]))
    try:
        for k in ks:
            out = dec.decode(k)
            torch.cuda.synchronize()
            assert dec.status() == (-1, 0), (config, k)
            coef = dec.coeffs().cpu().numpy()
            out_h = out.cpu().numpy()
            if k == full_truth_k:
                # all scan groups = the full-quality data (paper Section 3): every image, every block
                for i in range(rec.n_images):
                    a, b = pcr_image_blocks(dec.handle, i)
                    assert np.array_equal(coef[a:a + b], rec.truth(i)), f"config {config} image {i}"
            for i in sample:
                a, b = pcr_image_blocks(dec.handle, i)
                W, H = rec.dims[i]
                want_c, want_rgb = O.decode_image(rec.bytes, i, k)
                assert np.array_equal(coef[a:a + b], want_c), f"config {config} image {i} k {k}"
                assert np.array_equal(want_c, mask_truth(rec.truth(i), W, H, k))
                inf = dec.info[i]
                got = out_h[inf.out_offset:inf.out_offset + inf.out_bytes].reshape(inf.height, inf.width, 3)
                assert np.array_equal(got, want_rgb), f"config {config} image {i} k {k}"
    finally:
        dec.close()


def test_imagenet_shaped_full_record():
    _check(1, (1, 2, 5, 10), 20)


def test_celeba_shaped_full_record_every_k():
    _check(2, range(1, 11), 10)


def test_ham_shaped_full_record_no_restart_markers():
    _check(3, (1, 5, 10), 6)


def test_imagenet_shaped_full_record_training_tensor():
    """The fixed-size training batch at full record size, in the benchmark's configuration:
    sampled images against the oracle, and for every image the mirror property (the same crop
    with the flip flag toggled gives the column-reversed tensor, bit for bit)."""
    import torch
    from paper_1911_00472_b200 import Decoder
    rec = pcr_synth.make_record(1, 0)
    dec = Decoder(rec.bytes)
    mean, std = (0.485, 0.456, 0.406), (0.229, 0.224, 0.225)
    crops = pcr_synth.random_resized_crops([(int(w), int(h)) for w, h in rec.dims], 21)
    try:
        for k, size in ((10, 224), (2, 160)):
            t = dec.decode_tensor(k, crops, size, mean, std).clone()
            torch.cuda.synchronize()
            assert dec.status() == (-1, 0)
            flipped = crops.copy()
            flipped[:, 4] ^= 1
            t2 = dec.decode_tensor(k, flipped, size, mean, std)
            torch.cuda.synchronize()
            assert torch.equal(t2, torch.flip(t, dims=[3]))
            got = t.cpu().numpy().astype(np.float64)
            for i in (0, 511, rec.n_images - 1):
                _, rgb = O.decode_image(rec.bytes, i, k)
                want = O.training_tensor(rgb, crops[i], size, mean, std).astype(np.float64)
                assert np.abs(got[i] - want).max() <= 2.0 ** -9, (k, i)
    finally:
        dec.close()


def test_imagenet_shaped_full_record_msssim():
    """pcr_msssim at full record size: sampled images against the oracle, every score in (0, 1],
    more scan groups never score lower on average."""
    import torch
    from paper_1911_00472_b200 import Decoder
    rec = pcr_synth.make_record(1, 0)
    dec = Decoder(rec.bytes)
    try:
        full = dec.decode(10, dec.alloc_out())
        means = []
        for k in (1, 5):
            part = dec.decode(k, dec.alloc_out())
            s = dec.msssim(part, full)
            torch.cuda.synchronize()
            v = s.cpu().numpy()
            assert np.all(v > 0) and np.all(v <= 1.0 + 1e-6)
            means.append(v.mean())
            for i in (3, 700):
                _, lo = O.decode_image(rec.bytes, i, k)
                _, hi = O.decode_image(rec.bytes, i, 10)
                assert abs(float(v[i]) - O.msssim(lo, hi)) <= 2e-4, (k, i)
        assert means[1] > means[0]
    finally:
        dec.close()
