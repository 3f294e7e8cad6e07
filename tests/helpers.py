"""Closed forms and brute-force references used by the tests (numpy only; no decoder code)."""
from __future__ import annotations

import io
import struct

import numpy as np


def block_grids(W, H, sampling=(2, 2, 3)):
    """MCU grid, padded block grid per component and block offsets; sampling = (hs, vs, components):
    hs x vs luminance blocks per MCU, one block per chroma component; one component = no MCU padding."""
    hs, vs, nc = sampling
    mx, my = (W + 8 * hs - 1) // (8 * hs), (H + 8 * vs - 1) // (8 * vs)
    padded = [(hs * mx, vs * my)] + [(mx, my)] * (nc - 1)
    off = [0, hs * vs * mx * my, (hs * vs + 1) * mx * my][:nc]
    return mx, my, padded, off


def comp_of_block(W, H, sampling=(2, 2, 3)):
    """Component index (0 Y, 1 Cb, 2 Cr) of every block of the canonical layout."""
    hs, vs, nc = sampling
    mx, my, _, _ = block_grids(W, H, sampling)
    parts = [np.zeros(hs * vs * mx * my, int)]
    if nc == 3:
        parts += [np.ones(mx * my, int), 2 * np.ones(mx * my, int)]
    return np.concatenate(parts)


def _trunc(c, bits):
    """Keep the magnitude bits above `bits` low ones, sign kept (shift toward zero)."""
    a = np.abs(c.astype(np.int32))
    return (np.sign(c) * ((a >> bits) << bits)).astype(np.int16)


def mask_truth(truth: np.ndarray, W: int, H: int, k: int) -> np.ndarray:
    """What a decoder holds after scan groups 1..k of the ten-scan script
    (DC: floor shift; AC: magnitude shift), written straight from the script:

      1: DC all, Al=1          6: Y  1..63 refine to Al=1
      2: Y  1..5  Al=2         7: DC refine to Al=0
      3: Cr 1..63 Al=1         8: Cr 1..63 refine to Al=0
      4: Cb 1..63 Al=1         9: Cb 1..63 refine to Al=0
      5: Y  6..63 Al=2        10: Y  1..63 refine to Al=0
    """
    comp = comp_of_block(W, H)
    out = np.zeros_like(truth)
    t = truth.astype(np.int32)
    # DC: point transform is an arithmetic shift (floor)
    out[:, 0] = (t[:, 0] if k >= 7 else ((t[:, 0] >> 1) << 1)).astype(np.int16)
    y, cb, cr = comp == 0, comp == 1, comp == 2

    def ac(sel, lo, hi, first, mid, full):
        """band lo..hi of blocks `sel`: absent before scan `first`; coarse (2 bits dropped) until
        `mid` if mid is given; 1 bit dropped until `full`; exact from `full` on."""
        if k < first:
            return
        sub = truth[sel][:, lo:hi + 1]
        if k >= full:
            v = sub
        elif mid is not None and k < mid:
            v = _trunc(sub, 2)
        else:
            v = _trunc(sub, 1)
        blk = out[sel]
        blk[:, lo:hi + 1] = v
        out[sel] = blk

    ac(y, 1, 5, 2, 6, 10)
    ac(y, 6, 63, 5, 6, 10)
    ac(cr, 1, 63, 3, None, 8)
    ac(cb, 1, 63, 4, None, 9)
    return out


def mask_truth_script(truth: np.ndarray, W: int, H: int, script, k: int, sampling=(2, 2, 3)) -> np.ndarray:
    """What a decoder holds after scans 1..k of an arbitrary script, written from the meaning of
    the script alone: a coefficient is known to the precision Al of the last scan <= k that
    covers its component and zigzag position (DC: floor shift, AC: magnitude shift toward zero),
    and is zero if no such scan exists.  script: [(components, Ss, Se, Ah, Al)]."""
    comp = comp_of_block(W, H, sampling)
    out = np.zeros_like(truth)
    for comps, Ss, Se, _Ah, Al in script[:k]:
        for c in comps:
            sel = comp == c
            sub = truth[sel][:, Ss:Se + 1].astype(np.int32)
            if Ss == 0:
                v = ((sub >> Al) << Al).astype(np.int16)
            else:
                v = _trunc(sub, Al)
            blk = out[sel]
            blk[:, Ss:Se + 1] = v
            out[sel] = blk
    return out


def zigzag_natural():
    """zigzag position -> natural index, from the definition (sort by anti-diagonal, alternating)."""
    order = sorted(range(64), key=lambda i: (i // 8 + i % 8, (i // 8) if (i // 8 + i % 8) % 2 else (i % 8)))
    return np.array(order)


def idct_double(coef_zz: np.ndarray, q_zz: np.ndarray) -> np.ndarray:
    """8x8 inverse DCT in double precision, by definition; returns unrounded samples + 128."""
    zz = zigzag_natural()
    F = np.zeros(64)
    F[zz] = coef_zz.astype(np.float64) * q_zz.astype(np.float64)
    F = F.reshape(8, 8)
    n = np.arange(8)
    B = np.cos((2 * n[:, None] + 1) * n[None, :] * np.pi / 16) * np.where(n[None, :] == 0, np.sqrt(0.5), 1.0) * 0.5
    return B @ F @ B.T + 128.0


def jpeg_segments(data: bytes):
    """Walk a JPEG byte string: list of (marker, payload_offset, payload_len, entropy_len)."""
    out = []
    p = 2
    assert data[:2] == b"\xff\xd8"
    n = len(data)
    while p < n:
        assert data[p] == 0xFF, (p, data[p])
        mk = data[p + 1]
        if mk == 0xD9:
            out.append((mk, p + 2, 0, 0))
            break
        L = struct.unpack(">H", data[p + 2:p + 4])[0]
        ent = 0
        if mk == 0xDA:
            q = p + 2 + L
            while True:
                j = data.find(b"\xff", q)
                if j < 0 or j + 1 >= n:
                    q = n
                    break
                if data[j + 1] == 0 or 0xD0 <= data[j + 1] <= 0xD7:
                    q = j + 2
                    continue
                q = j
                break
            ent = q - (p + 2 + L)
        out.append((mk, p + 4, L - 2, ent))
        p += 2 + L + ent
    return out


def pillow_y(jpeg_bytes: bytes) -> np.ndarray:
    """Luminance plane of a JPEG as a third-party decoder (Pillow) produces it, no colour
    conversion or chroma upsampling involved."""
    from PIL import Image
    im = Image.open(io.BytesIO(jpeg_bytes))
    im.draft("YCbCr", im.size)
    im.load()
    assert im.mode == "YCbCr"
    return np.asarray(im)[:, :, 0]


def oracle_rgb_shard(args):
    """Process-pool worker (module level so that spawned children can import it): decodes images
    lo..hi-1 of the record saved at rec_path with the CPU oracle at fidelity k and writes each
    image's pixels at its offset into the uint8 file out_path (the GPU output buffer's layout)."""
    rec_path, out_path, out_bytes, offsets, k, lo, hi = args
    from oracle import pcr_oracle as O
    rec = np.load(rec_path)
    out = np.memmap(out_path, dtype=np.uint8, mode="r+", shape=(out_bytes,))
    for i in range(lo, hi):
        _, rgb = O.decode_image(rec, i, k)
        out[offsets[i]:offsets[i] + rgb.size] = rgb.reshape(-1)
    out.flush()
    return hi - lo


def oracle_record_pixels(pool, workers, rec_bytes, tmpdir, offsets, out_bytes, k):
    """All images of a record at fidelity k through the oracle on a process pool: a uint8 array
    laid out like the output buffer of the decode (bytes between images zero)."""
    import os
    rec_path = os.path.join(tmpdir, "rec.npy")
    if not os.path.exists(rec_path):
        np.save(rec_path, rec_bytes)
    out_path = os.path.join(tmpdir, f"oracle_k{k}.u8")
    np.memmap(out_path, dtype=np.uint8, mode="w+", shape=(out_bytes,)).flush()
    n = len(offsets)
    per = max(1, (n + 4 * workers - 1) // (4 * workers))
    shards = [(rec_path, out_path, out_bytes, offsets, k, lo, min(lo + per, n)) for lo in range(0, n, per)]
    assert sum(pool.map(oracle_rgb_shard, shards)) == n
    return np.array(np.memmap(out_path, dtype=np.uint8, mode="r", shape=(out_bytes,)))
