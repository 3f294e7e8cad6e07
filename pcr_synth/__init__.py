"""Seeded synthetic inputs for the PCR decode path.

Makes records only: synthetic images -> quantised DCT coefficients (the ground truth)
-> progressive JPEG scans -> a Progressive Compressed Record laid out as the paper's
Section 3 describes (metadata, then scan group 1 of every image, scan group 2, ...).
None of the decode arithmetic lives here; the CPU oracle and the CUDA library both
consume these bytes and share no code with this module or with each other.

The C source beside this file is compiled on first use with the host compiler.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pcr_synth.c")
_LIB = os.path.join(_HERE, "libpcr_synth.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the generator into a shared library next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class ImageSpec(C.Structure):
    _fields_ = [
        ("width", C.c_uint32), ("height", C.c_uint32), ("label", C.c_int32), ("quality", C.c_int32),
        ("beta", C.c_double), ("gamma", C.c_double), ("sigma", C.c_double),
        ("blobs", C.c_int32), ("rsvd", C.c_int32), ("seed", C.c_uint64),
    ]


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = C.CDLL(build())
            lib.synth_record_create.restype = C.c_void_p
            lib.synth_record_create.argtypes = [C.POINTER(ImageSpec), C.c_int, C.c_int, C.c_int, C.c_int]
            lib.synth_record_from_coeffs.restype = C.c_void_p
            lib.synth_record_from_coeffs.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                                     C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int]
            lib.synth_record_bytes.restype = C.c_void_p
            lib.synth_record_bytes.argtypes = [C.c_void_p, C.POINTER(C.c_size_t)]
            lib.synth_record_truth_count.restype = C.c_size_t
            lib.synth_record_truth_count.argtypes = [C.c_void_p, C.c_int]
            lib.synth_record_truth.restype = C.c_void_p
            lib.synth_record_truth.argtypes = [C.c_void_p, C.c_int]
            lib.synth_record_jpeg.restype = C.c_void_p
            lib.synth_record_jpeg.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_size_t)]
            lib.synth_record_free.argtypes = [C.c_void_p]
            lib.synth_record_num_images.restype = C.c_int
            lib.synth_record_num_images.argtypes = [C.c_void_p]
            lib.synth_record_dims.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
            lib.synth_image_rgb.argtypes = [C.POINTER(ImageSpec), C.c_void_p]
            lib.synth_quant_table.argtypes = [C.c_int, C.c_int, C.c_void_p]
            lib.synth_num_blocks.restype = C.c_size_t
            lib.synth_num_blocks.argtypes = [C.c_uint32, C.c_uint32]
            lib.synth_zigzag.argtypes = [C.c_void_p]
            lib.synth_set_script.argtypes = [C.c_void_p, C.c_int]
            lib.synth_set_sampling.argtypes = [C.c_int, C.c_int, C.c_int]
            lib.synth_rgb_to_coeffs.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
            _lib = lib
    return _lib


# --------------------------------------------------------------------------------------
# plain-Python splitmix64, used only to draw image sizes and seeds
# --------------------------------------------------------------------------------------
_M64 = (1 << 64) - 1


def splitmix64(x: int) -> int:
    z = (x + 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def _unit(x: int) -> float:
    return (splitmix64(x) >> 11) / float(1 << 53)


# --------------------------------------------------------------------------------------
# workload recipes (shapes and statistics of the paper's datasets; Table 1 and Table 3)
# --------------------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    name: str
    images_per_record: int
    n_records: int
    quality: int
    beta: float
    gamma: float
    sigma: float
    blobs: bool
    restart_rows: bool
    fixed_size: tuple | None   # (W, H) or None for the 256..496 multiples of 16
    ks: tuple


WORKLOADS = {
    0: Workload("tiny32", 32, 1, 90, 1.0, 0.3, 4.0, False, True, (32, 32), tuple(range(1, 11))),
    1: Workload("imagenet_shaped", 1024, 1, 90, 1.0, 0.3, 4.0, False, True, None, (1, 2, 5, 10)),
    2: Workload("celeba_shaped", 1024, 4, 95, 1.0, 0.3, 3.0, True, True, (178, 218), tuple(range(1, 11))),
    3: Workload("ham10000_shaped", 1024, 2, 90, 2.0, 0.1, 2.0, False, False, (600, 450), (1, 5, 10)),
    4: Workload("imagenet_shaped_sweep", 1024, 16, 90, 1.0, 0.3, 4.0, False, True, None, tuple(range(1, 11))),
}


def record_seed(config: int, record: int) -> int:
    """Seed of record `record` of workload `config`; workload 0 is seed 0."""
    if config == 0:
        return 0
    # the sweep (4) continues the ImageNet-shaped distribution of workload 1 with new records
    c = 1 if config == 4 else config
    r = record + 1 if config == 4 else record
    return splitmix64((c << 20) ^ r) >> 1


def make_specs(config: int, record: int = 0, n_images: int | None = None):
    """Per-image recipes of one record of a workload."""
    w = WORKLOADS[config]
    n = w.images_per_record if n_images is None else n_images
    base = record_seed(config, record)
    specs = (ImageSpec * n)()
    for i in range(n):
        s = (base * 1000003 + i) & _M64
        if w.fixed_size is not None:
            W, H = w.fixed_size
        else:
            W = 16 * int(round((256 + 244 * _unit(s ^ 0xA5A5)) / 16.0))
            H = 16 * int(round((256 + 244 * _unit(s ^ 0x5A5A00)) / 16.0))
        specs[i] = ImageSpec(W, H, int(splitmix64(s ^ 0x77) % 1000), w.quality, w.beta, w.gamma, w.sigma,
                             1 if w.blobs else 0, 0, s)
    return specs


class Record:
    """A synthetic PCR record plus its ground truth (owned by the C side until closed)."""

    def __init__(self, handle):
        self._lib = _load()
        self._h = C.c_void_p(handle)
        self.sampling = _sampling          # (hs, vs, components) the record was made with
        n = C.c_size_t()
        p = self._lib.synth_record_bytes(self._h, C.byref(n))
        self.n_images = self._lib.synth_record_num_images(self._h)
        # one owning copy of the record bytes (page-aligned, writable: tests poison it)
        self.bytes = np.ctypeslib.as_array(C.cast(p, C.POINTER(C.c_uint8)), shape=(n.value,)).copy()
        self.dims = []
        for i in range(self.n_images):
            W, H = C.c_uint32(), C.c_uint32()
            self._lib.synth_record_dims(self._h, i, C.byref(W), C.byref(H))
            self.dims.append((W.value, H.value))

    def truth(self, i: int) -> np.ndarray:
        """Ground-truth quantised coefficients of image i: (blocks, 64) int16, zigzag order,
        blocks ordered component, block row, block column over the MCU-padded grid."""
        n = self._lib.synth_record_truth_count(self._h, i)
        p = self._lib.synth_record_truth(self._h, i)
        return np.ctypeslib.as_array(C.cast(p, C.POINTER(C.c_int16)), shape=(n,)).copy().reshape(-1, 64)

    def jpeg(self, i: int) -> bytes:
        """The stand-alone progressive JPEG file the record's chunks of image i were cut from."""
        n = C.c_size_t()
        p = self._lib.synth_record_jpeg(self._h, i, C.byref(n))
        return C.string_at(p, n.value)

    def close(self):
        if self._h:
            self._lib.synth_record_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def make_record(config: int, record: int = 0, n_images: int | None = None, threads: int = 0,
                restart_fixed: int = 0, restart_rows: bool | None = None) -> Record:
    """Generate one record of a workload (seeded; same arguments -> same bytes)."""
    lib = _load()
    specs = make_specs(config, record, n_images)
    rr = WORKLOADS[config].restart_rows if restart_rows is None else restart_rows
    h = lib.synth_record_create(specs, len(specs), 1 if rr else 0, restart_fixed, threads)
    return Record(h)


def record_from_specs(specs, restart_rows: bool = True, restart_fixed: int = 0, threads: int = 0) -> Record:
    lib = _load()
    arr = (ImageSpec * len(specs))(*specs)
    return Record(lib.synth_record_create(arr, len(specs), 1 if restart_rows else 0, restart_fixed, threads))


def record_from_coeffs(dims, coeffs, quality: int = 90, labels=None, restart_rows: bool = True,
                       restart_fixed: int = 0, qtables=None, threads: int = 0) -> Record:
    """Encode given coefficient arrays (one (blocks, 64) int16 array per image, canonical layout)."""
    lib = _load()
    n = len(dims)
    W = np.array([d[0] for d in dims], dtype=np.uint32)
    H = np.array([d[1] for d in dims], dtype=np.uint32)
    lab = np.zeros(n, dtype=np.int32) if labels is None else np.asarray(labels, dtype=np.int32)
    if qtables is None:
        qy1, qc1 = quant_table(quality, False), quant_table(quality, True)
        qy = np.tile(qy1, (n, 1))
        qc = np.tile(qc1, (n, 1))
    else:
        qy = np.ascontiguousarray(np.broadcast_to(np.asarray(qtables[0], dtype=np.uint8).reshape(-1, 64), (n, 64)))
        qc = np.ascontiguousarray(np.broadcast_to(np.asarray(qtables[1], dtype=np.uint8).reshape(-1, 64), (n, 64)))
    keep = []
    ptrs = (C.c_void_p * n)()
    for i in range(n):
        a = np.ascontiguousarray(coeffs[i], dtype=np.int16).reshape(-1)
        assert a.size == num_blocks(*dims[i]) * 64, "coefficient array does not match the image's block grid"
        keep.append(a)
        ptrs[i] = a.ctypes.data
    h = lib.synth_record_from_coeffs(n, W.ctypes.data, H.ctypes.data, lab.ctypes.data, C.cast(ptrs, C.c_void_p),
                                     qy.ctypes.data, qc.ctypes.data, 1 if restart_rows else 0, restart_fixed, threads)
    return Record(h)


def image_rgb(spec: ImageSpec) -> np.ndarray:
    lib = _load()
    out = np.empty((spec.height, spec.width, 3), dtype=np.uint8)
    lib.synth_image_rgb(C.byref(spec), out.ctypes.data)
    return out


def rgb_to_coeffs(rgb: np.ndarray, quality: int = 90) -> np.ndarray:
    lib = _load()
    rgb = np.ascontiguousarray(rgb, dtype=np.uint8)
    H, W, _ = rgb.shape
    out = np.empty((num_blocks(W, H), 64), dtype=np.int16)
    qy, qc = quant_table(quality, False), quant_table(quality, True)
    lib.synth_rgb_to_coeffs(rgb.ctypes.data, W, H, qy.ctypes.data, qc.ctypes.data, out.ctypes.data)
    return out


def quant_table(quality: int, chroma: bool) -> np.ndarray:
    """Scaled quantisation table in natural (row-major) order."""
    lib = _load()
    out = np.empty(64, dtype=np.uint8)
    lib.synth_quant_table(quality, 1 if chroma else 0, out.ctypes.data)
    return out


def num_blocks(W: int, H: int) -> int:
    return int(_load().synth_num_blocks(W, H))


def zigzag() -> np.ndarray:
    """zigzag position -> natural index."""
    out = np.empty(64, dtype=np.int32)
    _load().synth_zigzag(out.ctypes.data)
    return out


def block_grids(W: int, H: int, sampling=(2, 2, 3)):
    """(padded, unpadded) block grids per component as [(bw, bh)] * components, and block offsets."""
    hs, vs, nc = sampling
    mx, my = (W + 8 * hs - 1) // (8 * hs), (H + 8 * vs - 1) // (8 * vs)
    padded = [(hs * mx, vs * my)] + [(mx, my)] * (nc - 1)
    cw, ch = (W + hs - 1) // hs, (H + vs - 1) // vs
    unp = [((W + 7) // 8, (H + 7) // 8)] + [((cw + 7) // 8, (ch + 7) // 8)] * (nc - 1)
    off = [0, padded[0][0] * padded[0][1], padded[0][0] * padded[0][1] + mx * my][:nc]
    return padded, unp, off


def random_resized_crops(dims, seed: int, scale=(0.08, 1.0), ratio=(3.0 / 4.0, 4.0 / 3.0)) -> np.ndarray:
    """Seeded crop rectangles and flip flags, one per image: (N, 5) uint32 rows x0, y0, w, h, flip.

    The usual ImageNet training augmentation draws: area fraction uniform in `scale`, aspect
    ratio log-uniform in `ratio`, position uniform, ten attempts then the whole image; flip
    with probability one half.  These are inputs of the decode path (the random numbers are
    drawn here, never inside it)."""
    import math
    out = np.zeros((len(dims), 5), dtype=np.uint32)
    for i, (W, H) in enumerate(dims):
        st = splitmix64((seed * 0x9E3779B97F4A7C15 + i + 1) & _M64)
        def u():
            nonlocal st
            st = splitmix64(st)
            return _unit(st)
        rect = (0, 0, int(W), int(H))
        for _ in range(10):
            area = W * H * (scale[0] + (scale[1] - scale[0]) * u())
            ar = math.exp(math.log(ratio[0]) + (math.log(ratio[1]) - math.log(ratio[0])) * u())
            w = int(round(math.sqrt(area * ar)))
            h = int(round(math.sqrt(area / ar)))
            if 0 < w <= W and 0 < h <= H:
                x0 = int(u() * (W - w + 1))
                y0 = int(u() * (H - h + 1))
                rect = (min(x0, W - w), min(y0, H - h), w, h)
                break
        out[i, :4] = rect
        out[i, 4] = 1 if u() < 0.5 else 0
    return out


# --------------------------------------------------------------------------------------
# other scan scripts (the paper, Section 4.2: unused scans can be dropped; any script that
# progressive JPEG allows makes a record, one scan per group)
# --------------------------------------------------------------------------------------
# (components, Ss, Se, Ah, Al); components: (0, 1, 2) = interleaved Y, Cb, Cr
SCRIPT_DEFAULT = None
SCRIPT_SPECTRAL_4 = [((0, 1, 2), 0, 0, 0, 0), ((0,), 1, 63, 0, 0), ((1,), 1, 63, 0, 0), ((2,), 1, 63, 0, 0)]
SCRIPT_MIXED_6 = [((0, 1, 2), 0, 0, 0, 1), ((0,), 1, 63, 0, 1), ((1,), 1, 63, 0, 0), ((2,), 1, 63, 0, 0),
                  ((0, 1, 2), 0, 0, 1, 0), ((0,), 1, 63, 1, 0)]
SCRIPT_DEEP_14 = [((0, 1, 2), 0, 0, 0, 2), ((0,), 1, 9, 0, 3), ((0,), 10, 63, 0, 3), ((1,), 1, 63, 0, 2),
                  ((2,), 1, 63, 0, 2), ((0,), 1, 63, 3, 2), ((0, 1, 2), 0, 0, 2, 1), ((0,), 1, 63, 2, 1),
                  ((1,), 1, 63, 2, 1), ((2,), 1, 63, 2, 1), ((0, 1, 2), 0, 0, 1, 0), ((0,), 1, 63, 1, 0),
                  ((1,), 1, 63, 1, 0), ((2,), 1, 63, 1, 0)]


# baseline (sequential) JPEG: one interleaved scan with the DC and all AC coefficients of every block
SCRIPT_BASELINE = [((0, 1, 2), 0, 63, 0, 0)]


_sampling = (2, 2, 3)


class sampling:
    """Context manager: records made inside have luminance sampling hs x vs (1 or 2 each; 2 x 2 =
    4:2:0, 2 x 1 = 4:2:2, 1 x 1 = 4:4:4) and `components` components (1 = greyscale: the scans of
    the chroma components drop out of the script).  Not thread safe (a process-wide setting)."""

    def __init__(self, hs: int, vs: int, components: int = 3):
        self.new = (1, 1, 1) if components == 1 else (hs, vs, components)

    def __enter__(self):
        global _sampling
        self.old = _sampling
        if _load().synth_set_sampling(*self.new) != 0:
            raise ValueError("unsupported sampling")
        _sampling = self.new
        return self

    def __exit__(self, *exc):
        global _sampling
        _load().synth_set_sampling(*self.old)
        _sampling = self.old
        return False


class scan_script:
    """Context manager: records made inside use `script` (a list of (components, Ss, Se, Ah, Al),
    at most 16 scans) instead of the ten-scan default.  Not thread safe (a process-wide setting)."""

    def __init__(self, script):
        self.script = script

    def __enter__(self):
        lib = _load()
        if self.script is None:
            lib.synth_set_script(None, 0)
            return self
        flat = []
        for comps, Ss, Se, Ah, Al in self.script:
            cs = list(comps) + [0] * (3 - len(comps))
            flat += [len(comps)] + cs + [Ss, Se, Ah, Al]
        arr = (C.c_int * len(flat))(*flat)
        if lib.synth_set_script(arr, len(self.script)) != 0:
            raise ValueError("scan script too long")
        return self

    def __exit__(self, *exc):
        _load().synth_set_script(None, 0)
        return False
