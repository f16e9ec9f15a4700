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


def test_code_fitting_on_the_host_matches_the_oracle():
    """nuq_fit_level_code and nuq_set_level_code are host functions: the lengths equal those of the oracle's
    Huffman construction (same tie rule, different implementation) on counts with ties and zeros."""
    import numpy as np
    import oracle as O
    from paper_1908_06077_b200 import build
    lib = ctypes.CDLL(build.build())
    lib.nuq_fit_level_code.argtypes = [ctypes.POINTER(ctypes.c_uint64), ctypes.c_uint32, ctypes.POINTER(ctypes.c_uint8)]
    lib.nuq_set_level_code.argtypes = [ctypes.POINTER(ctypes.c_uint8), ctypes.c_uint32]
    lib.nuq_encode_bound.restype = ctypes.c_uint64
    lib.nuq_encode_bound.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32]
    rng = np.random.default_rng(4)
    for s in range(1, 8):
        for trial in range(40):
            hi = [3, 10, 1000, 1 << 40][trial % 4]
            hist = rng.integers(0, hi, s + 2).astype(np.uint64)
            arr = (ctypes.c_uint64 * (s + 2))(*[int(x) for x in hist])
            out = (ctypes.c_uint8 * (s + 1))()
            assert lib.nuq_fit_level_code(arr, s, out) == 0
            assert list(out) == list(O.huffman_lengths(hist[1:])), (s, hist)
            assert lib.nuq_set_level_code(out, s) == 0
    out8 = (ctypes.c_uint8 * 9)()
    assert lib.nuq_fit_level_code((ctypes.c_uint64 * 10)(), 8, out8) == -1
    assert lib.nuq_fit_level_code((ctypes.c_uint64 * 10)(), 0, out8) == -1
    for bad in ([1, 1, 2], [0, 1], [1, 8], [1, 2, 3, 3, 3]):
        assert lib.nuq_set_level_code((ctypes.c_uint8 * len(bad))(*bad), len(bad) - 1) == -1
    assert lib.nuq_set_level_code((ctypes.c_uint8 * 3)(2, 2, 2), 2) == 0           # an incomplete code is a code
    # coded mode: two more header words than the ERC mode, and up to 7 bits per level index
    # (header, two table entries, norm + 16 length words + padding, 2 + L bits per element; L = |ERC(5)| = 6 or 7)
    assert lib.nuq_encode_bound(8192, 8192, 4, 0) == (4 * (16 + 4 + 18 + 8192 * 8 // 32) + 15) // 16 * 16
    assert lib.nuq_encode_bound(8192, 8192, 4, 2 << 16) == (4 * (18 + 4 + 18 + 8192 * 9 // 32) + 15) // 16 * 16
    assert lib.nuq_encode_bound(8192, 8192, 8, 2 << 16) == 0 and lib.nuq_encode_bound(8192, 8192, 4, (2 << 16) | (1 << 8)) == 0
