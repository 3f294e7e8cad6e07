"""CPU-only checks of the boundary: the library loads and exports every declared symbol,
and the host-side validation paths that need no device work behave as documented."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1911_00472_b200 import build
    path = build.build()
    return C.CDLL(path)


def _declared():
    text = open(os.path.join(ROOT, "include", "pcr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pcr_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared()
    assert {"pcr_open", "pcr_decode", "pcr_close"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_names():
    from paper_1911_00472_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_argument_errors_need_no_device(lib):
    lib.pcr_open.argtypes = [C.c_void_p, C.c_size_t, C.POINTER(C.c_void_p)]
    h = C.c_void_p()
    assert lib.pcr_open(None, 10, C.byref(h)) == -1
    buf = (C.c_uint8 * 128)()
    assert lib.pcr_open(buf, 128, C.byref(h)) == -2 and not h.value       # bad magic
    assert lib.pcr_open(buf, 10, C.byref(h)) == -2                          # too short
    lib.pcr_num_images.argtypes = [C.c_void_p]
    assert lib.pcr_num_images(None) == -1
    lib.pcr_out_bytes.restype = C.c_size_t
    lib.pcr_out_bytes.argtypes = [C.c_void_p]
    assert lib.pcr_out_bytes(None) == 0
    lib.pcr_decode.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
    assert lib.pcr_decode(None, 1, None, None) == -1
    lib.pcr_close.argtypes = [C.c_void_p]
    lib.pcr_close(None)
    lib.pcr_strerror.restype = C.c_char_p
    assert lib.pcr_strerror(-3) == b"corrupt entropy-coded data"


def test_product_path_does_not_touch_the_oracle():
    """Neither the package nor the generator imports or mentions the oracle."""
    for folder in ("paper_1911_00472_b200", "pcr_synth"):
        for dirpath, _, files in os.walk(os.path.join(ROOT, folder)):
            for f in files:
                if f.endswith((".py", ".cu", ".cuh", ".h", ".c")):
                    text = open(os.path.join(dirpath, f)).read()
                    assert "import oracle" not in text and "from oracle" not in text and "pcr_oracle" not in text, f
