"""The allocation-free pixel entry point against the regular decode (GPU).

Some callers of this library run where device memory cannot be allocated any more: inside
another framework's memory pool, or after the training job has taken the whole device.
`pcr_pixels_noalloc` serves them: it keeps its small tables in a fixed array inside the
library instead of cudaMalloc'd buffers.  Here it must reproduce, byte for byte, the pixels
that `pcr_decode` writes for the same coefficients, on two calls in a row (the second call
reuses the array the first one filled, with a different image size), and both must equal what
the CPU oracle makes of the same coefficients.

This file sorts last on purpose, so a run that stops at the first failure has already run
every other test.
"""
import numpy as np
import pytest

import pcr_synth
from oracle import pcr_oracle as O

pytestmark = pytest.mark.gpu


def _zigzag_quantisers(quality):
    zz = pcr_synth.zigzag()
    qy = pcr_synth.quant_table(quality, False)[zz].astype(np.uint16)
    qc = pcr_synth.quant_table(quality, True)[zz].astype(np.uint16)
    return np.ascontiguousarray(np.concatenate([qy, qc, qc]))


def test_noalloc_pixels_match_decode_on_two_calls_in_a_row():
    import torch
    from paper_1911_00472_b200 import Decoder, binding
    # two shapes: a width that is not a multiple of 16 (ragged rows) and a 16-multiple one
    specs = [pcr_synth.ImageSpec(178, 218, 0, 95, 1.0, 0.3, 3.0, 1, 0, 71),
             pcr_synth.ImageSpec(272, 304, 1, 95, 1.0, 0.3, 4.0, 0, 0, 72)]
    rec = pcr_synth.record_from_specs(specs)
    dec = Decoder(rec.bytes)
    out = dec.decode(10)
    torch.cuda.synchronize()
    assert dec.status() == (-1, 0)
    q = _zigzag_quantisers(95)
    stream = torch.cuda.current_stream()
    results = []
    for i in (0, 1):
        inf = dec.info[i]
        coef = dec.coeffs(i).contiguous()                       # device copy of image i's planes
        rgb = torch.full((inf.height * inf.width * 3,), 0xEE, dtype=torch.uint8, device="cuda")
        binding.pcr_pixels_noalloc(coef.data_ptr(), inf.width, inf.height, q.ctypes.data, rgb.data_ptr(), stream.cuda_stream)
        results.append((i, rgb))
    torch.cuda.synchronize()
    for i, rgb in results:
        inf = dec.info[i]
        want = out[inf.out_offset:inf.out_offset + inf.out_bytes]
        assert torch.equal(rgb, want), f"image {i}"
        # ... and the oracle's pixels from the same coefficients (which are the ground truth at k = 10)
        coef_h = dec.coeffs(i).cpu().numpy()
        assert np.array_equal(coef_h, rec.truth(i)), f"image {i}"
        want_o = O.pixels_from_coeffs(coef_h, inf.width, inf.height, q[:64], q[64:128])
        assert np.array_equal(rgb.cpu().numpy().reshape(inf.height, inf.width, 3), want_o), f"image {i}"
    # sizes beyond the fixed array are refused with a clear error, nothing is launched
    with pytest.raises(binding.PcrError) as e:
        binding.pcr_pixels_noalloc(results[0][1].data_ptr(), 4112, 16, q.ctypes.data, results[0][1].data_ptr(), 0)
    assert e.value.code == binding.PCR_E_ARG
    # the kernel reads the coefficients as 16-byte vectors: a pointer that is only 4-byte aligned
    # is refused before anything is launched
    coef = dec.coeffs(0).contiguous()
    inf = dec.info[0]
    for shift in (4, 8, 12):
        with pytest.raises(binding.PcrError) as e:
            binding.pcr_pixels_noalloc(coef.data_ptr() + shift, inf.width, inf.height, q.ctypes.data,
                                       results[0][1].data_ptr(), stream.cuda_stream)
        assert e.value.code == binding.PCR_E_ARG
    torch.cuda.synchronize()
    dec.close()
