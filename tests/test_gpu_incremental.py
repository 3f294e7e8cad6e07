"""Raising the fidelity of a resident decode (paper Section 3: reading subsequent scan groups
raises the fidelity without re-encoding): pcr_decode(k1) followed by pcr_decode_more(k2) must give
exactly what pcr_decode(k2) gives, which the other tests tie to the oracle."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _snapshot(dec, out):
    import torch
    torch.cuda.synchronize()
    assert dec.status() == (-1, 0)
    return out.clone(), dec.coeffs()


@pytest.mark.parametrize("fix", ["rec0", "rec1_small", "rec3_small"])
def test_decode_more_equals_decode_from_scratch(fix, request):
    import torch
    from paper_1911_00472_b200 import Decoder
    from oracle import pcr_oracle as O
    rec = request.getfixturevalue(fix)
    ref = Decoder(rec.bytes)
    inc = Decoder(rec.bytes)
    # zeroed output buffers: the padding between images is never written
    ref.out = torch.zeros_like(ref.alloc_out())
    inc.out = torch.zeros_like(inc.alloc_out())
    want = {}
    for k in range(1, 11):
        want[k] = _snapshot(ref, ref.decode(k))
    # what the chains are compared with is itself the oracle's result, for every image and k
    from paper_1911_00472_b200 import pcr_image_blocks
    oracle = {k: [O.decode_image(rec.bytes, i, k) for i in range(rec.n_images)] for k in range(1, 11)}

    def assert_oracle(snap, k, what):
        out_h, coef_h = snap[0].cpu().numpy(), snap[1].cpu().numpy()
        for i in range(rec.n_images):
            inf = ref.info[i]
            a, b = pcr_image_blocks(ref.handle, i)
            want_c, want_rgb = oracle[k][i]
            assert np.array_equal(coef_h[a:a + b], want_c), (fix, what, k, i)
            assert np.array_equal(out_h[inf.out_offset:inf.out_offset + inf.out_bytes].reshape(inf.height, inf.width, 3), want_rgb), (fix, what, k, i)

    for k in range(1, 11):
        assert_oracle(want[k], k, "from scratch")
    # one scan group at a time, and a few jumps (from DC only, across the refinement waves)
    chains = [list(range(1, 11)), [1, 10], [2, 6, 7], [5, 8, 10], [4, 9]]
    for chain in chains:
        out = inc.decode(chain[0])
        got = _snapshot(inc, out)
        assert torch.equal(got[0], want[chain[0]][0]) and torch.equal(got[1], want[chain[0]][1])
        for k in chain[1:]:
            out = inc.decode_more(k)
            got = _snapshot(inc, out)
            assert torch.equal(got[0], want[k][0]), (fix, chain, k)
            assert torch.equal(got[1], want[k][1]), (fix, chain, k)
        assert_oracle(got, chain[-1], chain)             # the end of every chain against the oracle directly
    # the end of the longest chain against the oracle directly
    coef, rgb = O.decode_image(rec.bytes, 0, 10)
    inf = inc.info[0]
    out = inc.decode(3); out = inc.decode_more(10)
    torch.cuda.synchronize()
    got = out[inf.out_offset:inf.out_offset + inf.out_bytes].view(inf.height, inf.width, 3).cpu().numpy()
    assert np.array_equal(got, rgb)
    ref.close(); inc.close()


def test_decode_more_argument_errors(rec0):
    from paper_1911_00472_b200 import Decoder, PcrError, binding
    dec = Decoder(rec0.bytes)
    out = dec.alloc_out()
    with pytest.raises(PcrError) as e:               # nothing decoded yet
        binding.pcr_decode_more(dec.handle, 3, out.data_ptr(), 0)
    assert e.value.code == binding.PCR_E_ARG
    dec.decode(4, out)
    for k in (4, 2, 11, 0):                          # not above the current fidelity / out of range
        with pytest.raises(PcrError):
            binding.pcr_decode_more(dec.handle, k, out.data_ptr(), 0)
    dec.close()


def test_decode_more_copies_only_the_missing_groups(rec0):
    """The later scan groups may arrive in host memory after the first decode: they are read only
    when the fidelity is raised."""
    import torch
    from paper_1911_00472_b200 import Decoder
    full = Decoder(rec0.bytes)
    full.out = torch.zeros_like(full.alloc_out())
    want = full.decode(10).clone()
    torch.cuda.synchronize()
    dec = Decoder(rec0.bytes)
    dec.out = torch.zeros_like(dec.alloc_out())
    pre = dec.prefix_bytes(5)
    saved = dec.host[pre:].clone()
    dec.host[pre:] = 0x5A                            # groups 6..10 "not read from storage yet"
    out = dec.decode(5)
    torch.cuda.synchronize()
    dec.host[pre:] = saved                           # now they are
    out = dec.decode_more(10)
    torch.cuda.synchronize()
    assert torch.equal(out, want)
    full.close(); dec.close()
