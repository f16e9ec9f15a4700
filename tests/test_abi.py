"""The C-ABI library loads without a GPU and exports every function include/nuq.h declares
(no compute call is made here)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "nuq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nuq_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_1908_06077_b200 import build
    lib = ctypes.CDLL(build.build())
    names = _declared()
    assert {"nuq_encode", "nuq_decode_accumulate", "nuq_encode_bound", "nuq_last_status"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_argument_only_calls_need_no_gpu():
    from paper_1908_06077_b200 import build
    lib = ctypes.CDLL(build.build())
    lib.nuq_encode_bound.restype = ctypes.c_uint64
    lib.nuq_encode_bound.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32]
    lib.nuq_version.restype = ctypes.c_char_p
    assert b"sm_100a" in lib.nuq_version()
    assert lib.nuq_encode_bound(65536, 1024, 3, 0) > 65536 // 8
    assert lib.nuq_encode_bound(65536, 1000, 3, 0) == 0          # bucket not a multiple of 256
    assert lib.nuq_encode_bound(65536, 1024, 0, 0) == 0
    # fixed mode: header + per bucket one norm word and B*w/32 field words, rounded up to 16 bytes
    assert lib.nuq_encode_bound(8192, 8192, 4, 1 << 16) == (4 * (16 + 1 + 8192 * 4 // 32) + 15) // 16 * 16
