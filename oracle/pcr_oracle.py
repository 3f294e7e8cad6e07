"""ctypes front end of the CPU oracle (`pcr_oracle.c`).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU-baseline leg may
import this; the CUDA library and its Python binding never do.  The C file is compiled on
first use with the host compiler; it links nothing but libm.

Follows the paper's Section 3 (record = metadata + scan groups, prefix read = fidelity k)
and Section 5 "Decoding" (reassemble scans 1..k, terminate with EOI, JPEG-decode).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pcr_oracle.c")
_LIB = os.path.join(_HERE, "libpcr_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = C.CDLL(build())
            vp, sz = C.c_void_p, C.c_size_t
            lib.oracle_record_info.argtypes = [vp, sz, C.POINTER(C.c_int), C.POINTER(C.c_int)]
            lib.oracle_image_info.argtypes = [vp, sz, C.c_int, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), C.POINTER(C.c_int32)]
            lib.oracle_prefix_bytes.restype = C.c_longlong
            lib.oracle_prefix_bytes.argtypes = [vp, sz, C.c_int]
            lib.oracle_reassemble.restype = C.c_longlong
            lib.oracle_reassemble.argtypes = [vp, sz, C.c_int, C.c_int, vp, sz]
            lib.oracle_decode_image.argtypes = [vp, sz, C.c_int, C.c_int, vp, sz, vp]
            lib.oracle_jpeg_decode.argtypes = [vp, sz, vp, sz, vp, vp, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
            lib.oracle_jpeg_dims.argtypes = [vp, sz, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
            lib.oracle_pixels_from_coeffs.argtypes = [vp, C.c_uint32, C.c_uint32, vp, vp, vp, vp, vp]
            lib.oracle_jpeg_info.argtypes = [vp, sz, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int)]
            lib.oracle_pixels_from_coeffs_s.argtypes = [vp, C.c_uint32, C.c_uint32, C.c_int, C.c_int, C.c_int, vp, vp, vp, vp, vp]
            lib.oracle_num_blocks_s.restype = sz
            lib.oracle_num_blocks_s.argtypes = [C.c_uint32, C.c_uint32, C.c_int, C.c_int, C.c_int]
            lib.oracle_num_blocks.restype = sz
            lib.oracle_num_blocks.argtypes = [C.c_uint32, C.c_uint32]
            lib.oracle_block_idct.argtypes = [vp, vp, vp]
            lib.oracle_ycc_to_rgb.argtypes = [C.c_int, C.c_int, C.c_int, vp]
            lib.oracle_ycc_to_rgb_array.argtypes = [vp, sz, vp]
            _lib = lib
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(f"oracle error {code}")
        self.code = code


def _chk(rc):
    if rc < 0:
        raise OracleError(rc)
    return rc


def _u8(buf) -> np.ndarray:
    a = np.frombuffer(buf, dtype=np.uint8) if not isinstance(buf, np.ndarray) else buf
    return np.ascontiguousarray(a, dtype=np.uint8)


def record_info(rec):
    """(number of images, number of scan groups)."""
    rec = _u8(rec)
    n, g = C.c_int(), C.c_int()
    _chk(_load().oracle_record_info(rec.ctypes.data, rec.size, C.byref(n), C.byref(g)))
    return n.value, g.value


def image_info(rec, i):
    """(width, height, label) of image i, from the record's sample metadata."""
    rec = _u8(rec)
    W, H, lab = C.c_uint32(), C.c_uint32(), C.c_int32()
    _chk(_load().oracle_image_info(rec.ctypes.data, rec.size, i, C.byref(W), C.byref(H), C.byref(lab)))
    return W.value, H.value, lab.value


def prefix_bytes(rec, k) -> int:
    rec = _u8(rec)
    return _chk(_load().oracle_prefix_bytes(rec.ctypes.data, rec.size, k))


def reassemble(rec, i, k) -> bytes:
    """Scans 1..k of image i followed by EOI: a JPEG file any stock decoder renders."""
    rec = _u8(rec)
    lib = _load()
    n = _chk(lib.oracle_reassemble(rec.ctypes.data, rec.size, i, k, None, 0))
    out = np.empty(n, dtype=np.uint8)
    _chk(lib.oracle_reassemble(rec.ctypes.data, rec.size, i, k, out.ctypes.data, out.size))
    return out.tobytes()


def num_blocks(W, H, sampling=(2, 2, 3)) -> int:
    """Blocks of the MCU-padded grids of all components; sampling = (hs, vs, components)."""
    return int(_load().oracle_num_blocks_s(W, H, *sampling))


def jpeg_info(jpg):
    """(W, H, (hs, vs, components)) from the frame header of a JPEG byte string."""
    a = _u8(jpg)
    W, H = C.c_uint32(), C.c_uint32()
    hs, vs, nc = C.c_int(), C.c_int(), C.c_int()
    _chk(_load().oracle_jpeg_info(a.ctypes.data, a.size, C.byref(W), C.byref(H), C.byref(hs), C.byref(vs), C.byref(nc)))
    return W.value, H.value, (hs.value, vs.value, nc.value)


def image_sampling(rec, i):
    """(hs, vs, components) of image i: read from the frame header at the head of its first chunk."""
    return jpeg_info(reassemble(rec, i, 1))[2]


def decode_image(rec, i, k, want_rgb=True):
    """Image i at fidelity k -> (coefficients (blocks, 64) int16 zigzag, RGB (H, W, 3) uint8 or None)."""
    rec = _u8(rec)
    W, H, _ = image_info(rec, i)
    coef = np.empty((num_blocks(W, H, image_sampling(rec, i)), 64), dtype=np.int16)
    rgb = np.empty((H, W, 3), dtype=np.uint8) if want_rgb else None
    _chk(_load().oracle_decode_image(rec.ctypes.data, rec.size, i, k, coef.ctypes.data, coef.size,
                                     rgb.ctypes.data if want_rgb else None))
    return coef, rgb


def _split_planes(planes, W, H, sampling):
    hs, vs, nc = sampling
    mx, my = (W + 8 * hs - 1) // (8 * hs), (H + 8 * vs - 1) // (8 * vs)
    ny = 64 * hs * vs * mx * my
    Y = planes[:ny].reshape(8 * vs * my, 8 * hs * mx)
    if nc == 1:
        return (Y,)
    Cb = planes[ny:ny + 64 * mx * my].reshape(8 * my, 8 * mx)
    Cr = planes[ny + 64 * mx * my:].reshape(8 * my, 8 * mx)
    return Y, Cb, Cr


def jpeg_decode(jpg: bytes, want_planes=False):
    """A progressive JPEG byte string -> (coefficients, RGB[, (Y, Cb, Cr) padded planes])."""
    lib = _load()
    a = _u8(jpg)
    W, H, samp = jpeg_info(a)
    nb = num_blocks(W, H, samp)
    coef = np.empty((nb, 64), dtype=np.int16)
    rgb = np.empty((H, W, 3), dtype=np.uint8)
    planes = np.empty(64 * nb, dtype=np.uint8) if want_planes else None
    _chk(lib.oracle_jpeg_decode(a.ctypes.data, a.size, coef.ctypes.data, coef.size, rgb.ctypes.data,
                                planes.ctypes.data if want_planes else None, None, None))
    if not want_planes:
        return coef, rgb
    return coef, rgb, _split_planes(planes, W, H, samp)


def pixels_from_coeffs(coef, W, H, qy_zz, qc_zz, want_planes=False, sampling=(2, 2, 3)):
    """Sequential-style decode of given coefficients: canonical (blocks, 64) int16 + zigzag-order
    quantisers -> RGB (H, W, 3)."""
    coef = np.ascontiguousarray(coef, dtype=np.int16)
    qy = np.ascontiguousarray(qy_zz, dtype=np.uint16)
    qc = np.ascontiguousarray(qc_zz, dtype=np.uint16)
    rgb = np.empty((H, W, 3), dtype=np.uint8)
    planes = np.empty(64 * num_blocks(W, H, sampling), dtype=np.uint8) if want_planes else None
    _chk(_load().oracle_pixels_from_coeffs_s(coef.ctypes.data, W, H, sampling[0], sampling[1], sampling[2],
                                             qy.ctypes.data, qc.ctypes.data, qc.ctypes.data,
                                             rgb.ctypes.data, planes.ctypes.data if want_planes else None))
    if not want_planes:
        return rgb
    return rgb, _split_planes(planes, W, H, sampling)


def block_idct(coef_zz, q_zz) -> np.ndarray:
    c = np.ascontiguousarray(coef_zz, dtype=np.int16)
    q = np.ascontiguousarray(q_zz, dtype=np.uint16)
    out = np.empty(64, dtype=np.uint8)
    _load().oracle_block_idct(c.ctypes.data, q.ctypes.data, out.ctypes.data)
    return out.reshape(8, 8)


def ycc_to_rgb(Y, cb, cr):
    out = np.empty(3, dtype=np.uint8)
    _load().oracle_ycc_to_rgb(int(Y), int(cb), int(cr), out.ctypes.data)
    return tuple(int(v) for v in out)


def ycc_to_rgb_array(ycc: np.ndarray) -> np.ndarray:
    """(n, 3) uint8 Y,Cb,Cr triples -> (n, 3) uint8 R,G,B."""
    a = np.ascontiguousarray(ycc, dtype=np.uint8).reshape(-1, 3)
    out = np.empty_like(a)
    _load().oracle_ycc_to_rgb_array(a.ctypes.data, a.shape[0], out.ctypes.data)
    return out


def decode_record(rec, k, images=None, want_rgb=True):
    """Decode every image (or the listed ones) of a record at fidelity k, one after the other."""
    n, _ = record_info(rec)
    idx = range(n) if images is None else images
    return [decode_image(rec, i, k, want_rgb) for i in idx]


def _pool_worker(args):
    path_or_bytes, k, lo, hi = args
    rec = np.load(path_or_bytes, mmap_mode="r") if isinstance(path_or_bytes, str) else _u8(path_or_bytes)
    rec = np.ascontiguousarray(rec)
    npx = 0
    for i in range(lo, hi):
        _, rgb = decode_image(rec, i, k, True)
        npx += rgb.shape[0] * rgb.shape[1]
    return hi - lo, npx


# --------------------------------------------------------------------------------------
# Training-tensor epilogue (Section 6 of the paper, experimental setup: resizing, crop and
# horizontal-flip augmentations, after which all inputs have the same size; 224x224 in the
# main experiments, 160x160 crops in the appendix's second pipeline).  The paper leaves
# the resampling filter to its frameworks; the reading taken here: plain bilinear
# interpolation with half-pixel centres inside the crop rectangle, edge pixels of the crop
# repeated, no low-pass filter, then (v / 255 - mean_c) / std_c per channel, planar layout.
# Evaluated in float64 by the definition, one output pixel = four taps.
# --------------------------------------------------------------------------------------
def training_tensor(rgb: np.ndarray, crop, size: int, mean, std, dtype=np.float16) -> np.ndarray:
    """rgb: (H, W, 3) uint8.  crop = (x0, y0, w, h, flip) in pixels of that image.
    Returns (3, size, size) of `dtype`: out[c, oy, ox] for output column ox taken from the
    crop's column u = size-1-ox when flip is set, else u = ox."""
    x0, y0, cw, ch, flip = (int(v) for v in crop)
    H, W, _ = rgb.shape
    if cw < 1 or ch < 1 or x0 < 0 or y0 < 0 or x0 + cw > W or y0 + ch > H:
        raise ValueError("crop outside the image")
    region = rgb[y0:y0 + ch, x0:x0 + cw, :].astype(np.float64)
    out = np.empty((3, size, size), dtype=np.float64)
    for oy in range(size):
        fy = (oy + 0.5) * ch / size - 0.5
        fy = min(max(fy, 0.0), ch - 1.0)
        iy = int(np.floor(fy))
        ay = fy - iy
        iy1 = min(iy + 1, ch - 1)
        for ox in range(size):
            u = size - 1 - ox if flip else ox
            fx = (u + 0.5) * cw / size - 0.5
            fx = min(max(fx, 0.0), cw - 1.0)
            ix = int(np.floor(fx))
            ax = fx - ix
            ix1 = min(ix + 1, cw - 1)
            top = (1.0 - ax) * region[iy, ix] + ax * region[iy, ix1]
            bot = (1.0 - ax) * region[iy1, ix] + ax * region[iy1, ix1]
            out[:, oy, ox] = (1.0 - ay) * top + ay * bot
    m = np.asarray(mean, dtype=np.float64).reshape(3, 1, 1)
    s = np.asarray(std, dtype=np.float64).reshape(3, 1, 1)
    return ((out / 255.0 - m) / s).astype(dtype)


# --------------------------------------------------------------------------------------
# Multi-scale structural similarity (the paper's Section 4.3 and appendix figure "reconstruction
# quality": MSSIM between the image decoded from scans 1..k and the full-fidelity image, used as
# a diagnostic for choosing k).  The measure is Wang, Simoncelli and Bovik's (2003); the paper
# does not say which implementation it ran.  Reading taken here, the common one:
#   * luminance Y = 0.299 R + 0.587 G + 0.114 B of the decoded 8-bit pixels, dynamic range L = 255;
#   * at every scale, local statistics under an 11x11 Gaussian window (sigma 1.5, normalised),
#     evaluated only where the window lies inside the image;
#   * cs = (2 s_xy + C2) / (s_x^2 + s_y^2 + C2), l = (2 m_x m_y + C1) / (m_x^2 + m_y^2 + C1),
#     C1 = (0.01 L)^2, C2 = (0.03 L)^2, averaged over the positions of the scale;
#   * next scale: 2x2 block averages (an odd last row or column is dropped);
#   * result = prod_j max(mean cs_j, 0)^w_j * max(mean l_M, 0)^w_M over the M scales with the
#     published weights (0.0448, 0.2856, 0.3001, 0.2363, 0.1333); images too small for five
#     scales (a side below 11 * 2^(M-1)) use the first M weights, rescaled to sum to one (the
#     five published weights are used as printed; they sum to 1.0001).
# Plain float64, windows written out by the definition.
# --------------------------------------------------------------------------------------
MSSSIM_WEIGHTS = (0.0448, 0.2856, 0.3001, 0.2363, 0.1333)


def gaussian_window(size: int = 11, sigma: float = 1.5) -> np.ndarray:
    x = np.arange(size, dtype=np.float64) - (size - 1) / 2.0
    g = np.exp(-(x * x) / (2.0 * sigma * sigma))
    return g / g.sum()


def luminance(rgb: np.ndarray) -> np.ndarray:
    r = rgb.astype(np.float64)
    return 0.299 * r[..., 0] + 0.587 * r[..., 1] + 0.114 * r[..., 2]


def _valid_filter(a: np.ndarray, g: np.ndarray) -> np.ndarray:
    """sum_{i,j} g[i] g[j] a[y+i, x+j] for every position where the window fits."""
    n = g.size
    H, W = a.shape
    rows = np.zeros((H, W - n + 1), dtype=np.float64)
    for j in range(n):
        rows += g[j] * a[:, j:j + W - n + 1]
    out = np.zeros((H - n + 1, W - n + 1), dtype=np.float64)
    for i in range(n):
        out += g[i] * rows[i:i + H - n + 1, :]
    return out


def msssim_scales(W: int, H: int, window: int = 11) -> int:
    m = 0
    while m < len(MSSSIM_WEIGHTS) and (min(W, H) >> m) >= window:
        m += 1
    return m


def msssim(rgb_a: np.ndarray, rgb_b: np.ndarray) -> float:
    """Multi-scale SSIM of two (H, W, 3) uint8 images of the same size (nan if a side is below 11)."""
    if rgb_a.shape != rgb_b.shape:
        raise ValueError("images differ in size")
    x, y = luminance(rgb_a), luminance(rgb_b)
    H, W = x.shape
    M = msssim_scales(W, H)
    if M == 0:
        return float("nan")
    w = np.array(MSSSIM_WEIGHTS[:M], dtype=np.float64)
    if M < len(MSSSIM_WEIGHTS):
        w = w / w.sum()
    g = gaussian_window()
    C1, C2 = (0.01 * 255.0) ** 2, (0.03 * 255.0) ** 2
    result = 1.0
    for j in range(M):
        mx, my = _valid_filter(x, g), _valid_filter(y, g)
        sxx = _valid_filter(x * x, g) - mx * mx
        syy = _valid_filter(y * y, g) - my * my
        sxy = _valid_filter(x * y, g) - mx * my
        cs = ((2.0 * sxy + C2) / (sxx + syy + C2)).mean()
        if j == M - 1:
            lum = ((2.0 * mx * my + C1) / (mx * mx + my * my + C1)).mean()
            result *= max(lum, 0.0) ** w[j]
        result *= max(cs, 0.0) ** w[j]
        if j < M - 1:
            h2, w2 = x.shape[0] // 2, x.shape[1] // 2
            x = x[:2 * h2, :2 * w2].reshape(h2, 2, w2, 2).mean(axis=(1, 3))
            y = y[:2 * h2, :2 * w2].reshape(h2, 2, w2, 2).mean(axis=(1, 3))
    return float(result)


# --------------------------------------------------------------------------------------
# Triangle ("linear") chroma upsampling, the filter stock decoders apply by default to 4:2:0
# data; the paper's decoders were stock ones (Section 5) and it does not name the filter.
# Reading taken: every pixel mixes its own chroma sample with the horizontally nearer, the
# vertically nearer and the diagonal neighbour with weights 9, 3, 3, 1 (sum 16, +8 and a shift:
# round half up); neighbours come from the decoded MCU-padded chroma planes, beyond their border
# the edge sample repeats.  Then the same colour conversion as with replication.
# --------------------------------------------------------------------------------------
def rgb_from_planes(Y: np.ndarray, Cb: np.ndarray, Cr: np.ndarray, W: int, H: int, triangle: bool) -> np.ndarray:
    """Padded sample planes (Y: 16my x 16mx, Cb/Cr: 8my x 8mx, uint8) -> (H, W, 3) uint8."""
    ch, cw = Cb.shape
    ys, xs = np.arange(H), np.arange(W)
    cy, cx = ys >> 1, xs >> 1
    if not triangle:
        cb, cr = Cb[cy][:, cx], Cr[cy][:, cx]
    else:
        ny = np.clip(cy + np.where(ys & 1, 1, -1), 0, ch - 1)
        nx = np.clip(cx + np.where(xs & 1, 1, -1), 0, cw - 1)

        def mix(P):
            P = P.astype(np.int64)
            return (9 * P[cy][:, cx] + 3 * P[cy][:, nx] + 3 * P[ny][:, cx] + P[ny][:, nx] + 8) >> 4
        cb, cr = mix(Cb), mix(Cr)
    ycc = np.stack([Y[:H, :W].astype(np.uint8), cb.astype(np.uint8), cr.astype(np.uint8)], axis=-1)
    return ycc_to_rgb_array(ycc.reshape(-1, 3)).reshape(H, W, 3)


def decode_image_upsampled(rec, i, k, triangle: bool):
    """Image i of a record at fidelity k with the chosen chroma upsampling: (coefficients, RGB)."""
    jpg = reassemble(rec, i, k)
    coef, _, (Y, Cb, Cr) = jpeg_decode(jpg, want_planes=True)
    W, H = image_info(rec, i)[:2]
    return coef, rgb_from_planes(Y, Cb, Cr, W, H, triangle)
