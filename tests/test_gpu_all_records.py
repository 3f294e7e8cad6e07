"""GPU parity over every record of the multi-record workloads, and over every pixel of a full
record (the paper's loader reads every record of a data set; Section 3: all scan groups are the
full-quality data, a prefix is the data masked to its bands and bit planes).

  * every record of the CelebA-shaped (4), HAM10000-shaped (2) and sweep (16) workloads: the int16
    coefficient planes of ALL images against the generator's ground truth at k = G and against the
    closed-form mask of the scan script at one k < G per record;
  * record 0 of the ImageNet-, CelebA- and HAM10000-shaped workloads: the pixels of ALL images at
    k = 10 and k = 5 against the CPU oracle (run on a process pool), byte for byte.
"""
import multiprocessing as mp
import os
import tempfile

import numpy as np
import pytest

import pcr_synth

from helpers import mask_truth, oracle_record_pixels

pytestmark = pytest.mark.gpu

G = 10
RECORDS = [(2, r) for r in range(4)] + [(3, r) for r in range(2)] + [(4, r) for r in range(16)]


@pytest.mark.parametrize("config,record", RECORDS)
def test_every_record_coefficients(config, record):
    import torch
    from paper_1911_00472_b200 import Decoder, pcr_image_blocks
    rec = pcr_synth.make_record(config, record)
    assert rec.n_images == pcr_synth.WORKLOADS[config].images_per_record
    dec = Decoder(rec.bytes)
    k_low = 1 + (3 * record + config) % (G - 1)          # a different prefix per record, all of 1..9 over the sweep
    try:
        for k in (G, k_low):
            dec.decode(k)
            torch.cuda.synchronize()
            assert dec.status() == (-1, 0), (config, record, k)
            coef = dec.coeffs().cpu().numpy()
            for i in range(rec.n_images):
                a, b = pcr_image_blocks(dec.handle, i)
                W, H = rec.dims[i]
                truth = rec.truth(i)
                want = truth if k == G else mask_truth(truth, W, H, k)
                assert np.array_equal(coef[a:a + b], want), f"config {config} record {record} image {i} k {k}"
    finally:
        dec.close()


@pytest.fixture(scope="module")
def oracle_pool():
    workers = max(1, min(len(os.sched_getaffinity(0)), 32))
    with mp.get_context("spawn").Pool(workers) as pool:
        yield pool, workers


@pytest.mark.parametrize("config", [1, 2, 3])
def test_full_record_every_pixel(config, oracle_pool):
    import torch
    from paper_1911_00472_b200 import Decoder
    pool, workers = oracle_pool
    rec = pcr_synth.make_record(config, 0)
    dec = Decoder(rec.bytes)
    offsets = [int(inf.out_offset) for inf in dec.info]
    try:
        with tempfile.TemporaryDirectory() as td:
            for k in (10, 5, 1):
                want = oracle_record_pixels(pool, workers, rec.bytes, td, offsets, dec.out_bytes, k)
                dec.out = torch.zeros(dec.out_bytes, dtype=torch.uint8, device="cuda")     # gaps between images stay zero
                got = dec.decode(k)
                torch.cuda.synchronize()
                assert dec.status() == (-1, 0), (config, k)
                got = got.cpu().numpy()
                if not np.array_equal(got, want):
                    for i, inf in enumerate(dec.info):
                        a, b = int(inf.out_offset), int(inf.out_offset + inf.out_bytes)
                        assert np.array_equal(got[a:b], want[a:b]), f"config {config} k {k}: image {i} differs"
                    raise AssertionError(f"config {config} k {k}: bytes between images differ")
    finally:
        dec.close()
