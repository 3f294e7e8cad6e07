"""ctypes binding of the C ABI declared in include/pcr.h: argument marshalling only.

Every step of the decode runs in the CUDA library; there is no CPU fallback.  Loading fails
loudly when the shared library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpcr_b200.so")

PCR_OK = 0
PCR_E_ARG, PCR_E_FORMAT, PCR_E_CORRUPT, PCR_E_TIMEOUT, PCR_E_CUDA, PCR_E_NOMEM = -1, -2, -3, -4, -5, -6

EXPORTS = ("pcr_open", "pcr_num_images", "pcr_num_groups", "pcr_get_image", "pcr_out_bytes", "pcr_prefix_bytes",
           "pcr_decode", "pcr_evict", "pcr_status", "pcr_coeffs", "pcr_image_blocks", "pcr_launch_count",
           "pcr_strerror", "pcr_close", "pcr_get_scan", "pcr_set_profiling", "pcr_get_profile",
           "pcr_pixels_noalloc", "pcr_decode_more", "pcr_release_cached_memory", "pcr_decode_tensor", "pcr_msssim", "pcr_msssim_scratch_bytes", "pcr_set_upsampling",
           "pcr_selftest_bounded_wait", "pcr_get_sampling", "pcr_set_record_cache")


class ImageInfo(C.Structure):
    _fields_ = [("width", C.c_uint32), ("height", C.c_uint32), ("label", C.c_int32), ("rsvd", C.c_uint32),
                ("out_offset", C.c_uint64), ("out_bytes", C.c_uint64)]


class ScanInfo(C.Structure):
    _fields_ = [("ncomp", C.c_int32), ("comp", C.c_int32 * 3), ("Ss", C.c_int32), ("Se", C.c_int32),
                ("Ah", C.c_int32), ("Al", C.c_int32), ("wave", C.c_int32), ("rsvd", C.c_int32), ("bytes", C.c_uint64)]


class StageTime(C.Structure):
    _fields_ = [("name", C.c_char * 24), ("ms", C.c_float), ("launches", C.c_int32)]


class PcrError(RuntimeError):
    def __init__(self, code, what=""):
        self.code = code
        super().__init__(f"{what}: {strerror(code)} ({code})")


_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it first (python -m paper_1911_00472_b200.build); "
                               "there is no fallback path")
        L = C.CDLL(LIB_PATH)
        vp = C.c_void_p
        L.pcr_open.argtypes = [vp, C.c_size_t, C.POINTER(vp)]
        L.pcr_num_images.argtypes = [vp]
        L.pcr_num_groups.argtypes = [vp]
        L.pcr_get_image.argtypes = [vp, C.c_int, C.POINTER(ImageInfo)]
        L.pcr_out_bytes.restype = C.c_size_t
        L.pcr_out_bytes.argtypes = [vp]
        L.pcr_prefix_bytes.restype = C.c_size_t
        L.pcr_prefix_bytes.argtypes = [vp, C.c_int]
        L.pcr_decode.argtypes = [vp, C.c_int, vp, vp]
        L.pcr_decode_more.argtypes = [vp, C.c_int, vp, vp]
        L.pcr_decode_tensor.argtypes = [vp, C.c_int, vp, C.c_int, vp, vp, C.c_int, vp, vp, vp]
        L.pcr_msssim_scratch_bytes.restype = C.c_size_t
        L.pcr_msssim_scratch_bytes.argtypes = [vp]
        L.pcr_msssim.argtypes = [vp, vp, vp, vp, vp, vp]
        L.pcr_set_upsampling.argtypes = [vp, C.c_int]
        L.pcr_evict.argtypes = [vp]
        L.pcr_status.argtypes = [vp, C.POINTER(C.c_int), C.POINTER(C.c_int)]
        L.pcr_coeffs.argtypes = [vp, C.POINTER(vp), C.POINTER(C.c_size_t)]
        L.pcr_image_blocks.argtypes = [vp, C.c_int, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
        L.pcr_get_scan.argtypes = [vp, C.c_int, C.POINTER(ScanInfo)]
        L.pcr_set_profiling.argtypes = [vp, C.c_int]
        L.pcr_get_profile.argtypes = [vp, C.POINTER(StageTime), C.c_int, C.POINTER(C.c_int)]
        L.pcr_pixels_noalloc.argtypes = [vp, C.c_uint32, C.c_uint32, vp, vp, vp]
        L.pcr_selftest_bounded_wait.argtypes = [C.POINTER(C.c_int)]
        L.pcr_set_record_cache.argtypes = [C.c_size_t]
        L.pcr_get_sampling.argtypes = [vp, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int)]
        L.pcr_launch_count.restype = C.c_uint64
        L.pcr_launch_count.argtypes = []
        L.pcr_strerror.restype = C.c_char_p
        L.pcr_strerror.argtypes = [C.c_int]
        L.pcr_release_cached_memory.restype = None
        L.pcr_release_cached_memory.argtypes = []
        L.pcr_close.restype = None
        L.pcr_close.argtypes = [vp]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().pcr_strerror(code).decode()


def _chk(rc, what):
    if rc != PCR_OK:
        raise PcrError(rc, what)


def pcr_open(host_ptr: int, length: int) -> int:
    h = C.c_void_p()
    _chk(lib().pcr_open(host_ptr, length, C.byref(h)), "pcr_open")
    return h.value


def pcr_close(handle: int) -> None:
    lib().pcr_close(handle)


def pcr_num_images(handle: int) -> int:
    return lib().pcr_num_images(handle)


def pcr_num_groups(handle: int) -> int:
    return lib().pcr_num_groups(handle)


def pcr_get_image(handle: int, i: int) -> ImageInfo:
    info = ImageInfo()
    _chk(lib().pcr_get_image(handle, i, C.byref(info)), "pcr_get_image")
    return info


def pcr_out_bytes(handle: int) -> int:
    return lib().pcr_out_bytes(handle)


def pcr_prefix_bytes(handle: int, k: int) -> int:
    return lib().pcr_prefix_bytes(handle, k)


def pcr_decode(handle: int, k: int, out_dev_ptr: int, stream: int = 0) -> None:
    _chk(lib().pcr_decode(handle, k, out_dev_ptr, stream), "pcr_decode")


def pcr_decode_more(handle: int, k: int, out_dev_ptr: int, stream: int = 0) -> None:
    _chk(lib().pcr_decode_more(handle, k, out_dev_ptr, stream), "pcr_decode_more")


PCR_F16, PCR_F32, PCR_BF16 = 0, 1, 2


def pcr_decode_tensor(handle: int, k: int, crops_host_ptr: int, size: int, mean_host_ptr: int, std_host_ptr: int,
                      dtype: int, rgb_dev_ptr: int, tensor_dev_ptr: int, stream: int = 0) -> None:
    _chk(lib().pcr_decode_tensor(handle, k, crops_host_ptr, size, mean_host_ptr, std_host_ptr, dtype,
                                 rgb_dev_ptr, tensor_dev_ptr, stream), "pcr_decode_tensor")


def pcr_msssim_scratch_bytes(handle: int) -> int:
    return lib().pcr_msssim_scratch_bytes(handle)


def pcr_msssim(handle: int, rgb_a_dev_ptr: int, rgb_b_dev_ptr: int, scratch_dev_ptr: int, scores_dev_ptr: int,
               stream: int = 0) -> None:
    _chk(lib().pcr_msssim(handle, rgb_a_dev_ptr, rgb_b_dev_ptr, scratch_dev_ptr, scores_dev_ptr, stream), "pcr_msssim")


PCR_UPSAMPLE_REPLICATE, PCR_UPSAMPLE_TRIANGLE = 0, 1


def pcr_set_upsampling(handle: int, mode: int) -> None:
    _chk(lib().pcr_set_upsampling(handle, mode), "pcr_set_upsampling")


def pcr_evict(handle: int) -> None:
    _chk(lib().pcr_evict(handle), "pcr_evict")


def pcr_status(handle: int):
    bad, code = C.c_int(), C.c_int()
    _chk(lib().pcr_status(handle, C.byref(bad), C.byref(code)), "pcr_status")
    return bad.value, code.value


def pcr_coeffs(handle: int):
    p, n = C.c_void_p(), C.c_size_t()
    _chk(lib().pcr_coeffs(handle, C.byref(p), C.byref(n)), "pcr_coeffs")
    return p.value, n.value


def pcr_image_blocks(handle: int, i: int):
    a, b = C.c_uint64(), C.c_uint64()
    _chk(lib().pcr_image_blocks(handle, i, C.byref(a), C.byref(b)), "pcr_image_blocks")
    return a.value, b.value


def pcr_launch_count() -> int:
    return lib().pcr_launch_count()


def pcr_get_scan(handle: int, s: int) -> ScanInfo:
    info = ScanInfo()
    _chk(lib().pcr_get_scan(handle, s, C.byref(info)), "pcr_get_scan")
    return info


def pcr_set_profiling(handle: int, enable: bool) -> None:
    _chk(lib().pcr_set_profiling(handle, 1 if enable else 0), "pcr_set_profiling")


def pcr_get_profile(handle: int):
    """[(stage name, milliseconds, kernel launches)] of the last decode (after a synchronise)."""
    arr = (StageTime * 16)()
    n = C.c_int()
    _chk(lib().pcr_get_profile(handle, arr, 16, C.byref(n)), "pcr_get_profile")
    return [(arr[i].name.decode(), float(arr[i].ms), int(arr[i].launches)) for i in range(n.value)]


def pcr_pixels_noalloc(dev_coeffs_ptr: int, width: int, height: int, host_qtab_ptr: int, dev_rgb_ptr: int,
                       stream: int = 0) -> None:
    """Pixel stage of one image with no allocation inside the library (see include/pcr.h):
    device coefficients + host quantisers -> device RGB, enqueued on `stream`."""
    _chk(lib().pcr_pixels_noalloc(dev_coeffs_ptr, width, height, host_qtab_ptr, dev_rgb_ptr, stream),
         "pcr_pixels_noalloc")


def pcr_get_sampling(handle: int):
    """(hs, vs, components) of the record's images."""
    a, b, c = C.c_int(), C.c_int(), C.c_int()
    _chk(lib().pcr_get_sampling(handle, C.byref(a), C.byref(b), C.byref(c)), "pcr_get_sampling")
    return a.value, b.value, c.value


def pcr_selftest_bounded_wait() -> bool:
    """True if the decoder's bounded device-side wait, pointed at a flag nothing sets, gave up at its limit."""
    v = C.c_int(-1)
    _chk(lib().pcr_selftest_bounded_wait(C.byref(v)), "pcr_selftest_bounded_wait")
    return v.value == 1


def pcr_set_record_cache(max_device_bytes: int) -> None:
    """Park closed records (up to this much device memory) for later opens of the same bytes; 0 = off."""
    _chk(lib().pcr_set_record_cache(max_device_bytes), "pcr_set_record_cache")


def pcr_release_cached_memory() -> None:
    lib().pcr_release_cached_memory()
