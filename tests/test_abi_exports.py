"""Host-only checks of the C ABI: the library builds, loads without a GPU and exports every
function that include/flexq.h declares; size helpers and error strings work without a device."""
import ctypes as C
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "flexq.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(fq_[a-z_0-9]+)\s*\(", src)))


def _lib():
    from paper_2501_07139_b200.build import build_library
    return C.CDLL(build_library())


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert {"fq_pack_layer", "fq_set_config", "fq_gemv", "fq_gemm"} <= set(names)
    lib = _lib()
    for n in names:
        assert hasattr(lib, n), n
    from paper_2501_07139_b200 import flexq
    assert set(flexq.EXPORTS) == set(names)


def test_size_helpers_and_error_strings_need_no_gpu():
    import paper_2501_07139_b200 as P
    assert P.fq_store_bytes(4096, 4096, 4, P.FQ_FMT_PACKED) == 8_388_608 + 524_288     # codes + scale/zero words
    assert P.fq_store_bytes(4096, 4096, 8, P.FQ_FMT_PLANES) == 16_777_216 + 524_288
    assert P.fq_store_bytes(17, 128, 3, P.FQ_FMT_PACKED) == 512 + 2048 * 3                # one blob: 32 rows x 512 cols
    assert P.fq_store_bytes(33, 1024, 5, P.FQ_FMT_PACKED) == 2 * 2 * (512 + 2048 * 5)
    assert P.fq_store_bytes(16, 100, 4, P.FQ_FMT_PACKED) == 0
    assert P.fq_store_bytes(16, 128, 9, P.FQ_FMT_PACKED) == 0
    assert P.fq_store_bytes(16, 128, 4, P.FQ_FMT_PLANES) == 0
    for code in range(0, -10, -1):
        assert P.fq_strerror(code) != "unknown error"
    assert P.fq_strerror(-99) == "unknown error"


def test_create_without_device_fails_cleanly():
    import torch
    if torch.cuda.is_available():
        return
    h = C.c_void_p()
    lib = _lib()
    lib.fq_create.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_int]
    assert lib.fq_create(C.byref(h), 0, 4) == -7 and not h
    assert lib.fq_create(None, 0, 4) == -1
