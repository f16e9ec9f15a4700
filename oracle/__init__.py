"""ctypes binding of the CPU oracle (oracle/nuq_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The product package never imports this module
and this module never imports the product package.

All arrays are numpy arrays in host memory.  Names and arguments mirror the C
functions; see nuq_oracle.c for the passage of the paper each one follows.
"""
import ctypes as C

import numpy as np

from .build import build as _build

NORM_L2, NORM_LINF = 0, 1
LEVELS_EXP, LEVELS_UNIFORM, LEVELS_TABLE = 0, 1, 2
MODE_ERC, MODE_FIXED, MODE_CODED = 0, 1, 2
MAX_CODED_S = 7
SB = 256
BLK = 32 * SB
HEADER_WORDS = 16
MAGIC = 0x3151554E


def make_flags(norm=NORM_L2, levelset=LEVELS_EXP, mode=MODE_ERC):
    return norm | (levelset << 8) | (mode << 16)


_lib = C.CDLL(_build())
_u8p = np.ctypeslib.ndpointer(np.uint8, flags="C_CONTIGUOUS")
_u16p = np.ctypeslib.ndpointer(np.uint16, flags="C_CONTIGUOUS")
_u32p = np.ctypeslib.ndpointer(np.uint32, flags="C_CONTIGUOUS")
_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")


def _sig(name, res, *args):
    f = getattr(_lib, name)
    f.restype = res
    f.argtypes = list(args)
    return f


_philox = _sig("nuq_oracle_philox4x32_10", None, _u32p, _u32p, _u32p)
_draw_word = _sig("nuq_oracle_draw_word", C.c_uint32, C.c_uint64, C.c_uint64, C.c_uint64)
_draw_uniform = _sig("nuq_oracle_draw_uniform", C.c_float, C.c_uint64, C.c_uint64, C.c_uint64)
_set_levels = _sig("nuq_oracle_set_levels", C.c_int, _f32p, C.c_uint32)
_huff = _sig("nuq_oracle_huffman_lengths", C.c_int, np.ctypeslib.ndpointer(np.uint64, flags="C_CONTIGUOUS"),
             C.c_uint32, _u8p)
_set_code = _sig("nuq_oracle_set_level_code", C.c_int, _u8p, C.c_uint32)
_level_code = _sig("nuq_oracle_level_code", C.c_uint32, C.c_uint32, _u8p)
_num_levels = _sig("nuq_oracle_num_levels", C.c_uint32, C.c_uint32, C.c_uint32)
_level_value = _sig("nuq_oracle_level_value", C.c_double, C.c_uint32, C.c_uint32, C.c_uint32)
_fixed_width = _sig("nuq_oracle_fixed_width", C.c_uint32, C.c_uint32, C.c_uint32)
_norm = _sig("nuq_oracle_norm", C.c_float, _f32p, C.c_uint64, C.c_uint32)
_bucket_norms = _sig("nuq_oracle_bucket_norms", None, _f32p, C.c_uint64, C.c_uint32, C.c_uint32, _f32p)
_round_prob = _sig("nuq_oracle_round_probability", None, C.c_float, C.c_float, C.c_uint32, C.c_uint32,
                   C.POINTER(C.c_uint32), C.POINTER(C.c_float))
_quant_bucket = _sig("nuq_oracle_quantize_bucket", None, _f32p, C.c_uint64, C.c_float, C.c_uint32, C.c_uint32,
                     C.c_uint64, C.c_uint64, C.c_uint64, _u8p, _u16p)
_quant_draws = _sig("nuq_oracle_quantize_with_draws", None, _f32p, C.c_uint64, C.c_float, C.c_uint32,
                    C.c_uint32, _f32p, _u8p, _u16p)
_dequant = _sig("nuq_oracle_dequantize", C.c_float, C.c_float, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32)
_qdq = _sig("nuq_oracle_quantize_dequantize", None, _f32p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32,
            C.c_uint32, C.c_uint64, C.c_uint64, _f32p)
_var_cf = _sig("nuq_oracle_variance_closed_form", C.c_double, _f32p, C.c_uint64, C.c_float, C.c_uint32,
               C.c_uint32)
_erc_enc = _sig("nuq_oracle_erc_encode", C.c_uint32, C.c_uint64, _u8p)
_erc_dec = _sig("nuq_oracle_erc_decode", C.c_uint64, _u8p, C.c_uint64, C.POINTER(C.c_uint64))
_bound = _sig("nuq_oracle_encode_bound", C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32)
_encode = _sig("nuq_oracle_encode", C.c_int, _f32p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32,
               C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p, C.c_uint64, C.POINTER(C.c_uint64))
_decode_sym = _sig("nuq_oracle_decode_symbols", C.c_int, C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint32,
                   _u8p, _u16p, _f32p)
_decode_acc = _sig("nuq_oracle_decode_accumulate", C.c_int, C.POINTER(C.c_void_p), C.c_uint32, C.c_uint64,
                   C.c_uint32, C.c_uint32, _f32p)
_chain_bits = _sig("nuq_oracle_single_chain_bits", C.c_uint64, _u16p, C.c_uint64)
_f64p = np.ctypeslib.ndpointer(np.float64, flags="C_CONTIGUOUS")
_momentum = _sig("nuq_oracle_momentum_step", None, _f64p, _f64p, _f32p, C.c_uint64, C.c_double, C.c_uint32,
                 C.c_double, C.c_double)


def philox4x32_10(ctr, key):
    out = np.zeros(4, np.uint32)
    _philox(np.ascontiguousarray(ctr, np.uint32), np.ascontiguousarray(key, np.uint32), out)
    return out


def draw_word(seed, offset, i):
    return int(_draw_word(seed, offset, i))


def draw_uniform(seed, offset, i):
    return float(_draw_uniform(seed, offset, i))


def set_levels(interior):
    """the interior levels l_1 < ... < l_s of the level sequence (0, l_1, ..., l_s, 1) that LEVELS_TABLE calls use"""
    lv = np.ascontiguousarray(interior, np.float32)
    rc = _set_levels(lv, lv.size)
    if rc != 0:
        raise ValueError("not a level sequence")


def huffman_lengths(weights):
    """code lengths of a Huffman tree over the given weights (2 to 8 of them), ties as the C file states"""
    w = np.ascontiguousarray(weights, np.uint64)
    out = np.zeros(w.size, np.uint8)
    if _huff(w, w.size, out) != 0:
        raise ValueError("2 to 8 weights")
    return out


def set_level_code(lengths):
    """code lengths of the level indices 1..s+1 that MODE_CODED calls use (canonical code words)"""
    ln = np.ascontiguousarray(lengths, np.uint8)
    if _set_code(ln, ln.size - 1) != 0:
        raise ValueError("not the lengths of a prefix code of at most 7 bits")


def level_code(j):
    """bits of the code word of level index j under the code last set"""
    bits = np.zeros(8, np.uint8)
    n = _level_code(j, bits)
    return bits[:n].copy()


def level_histogram(sym, s):
    """how often each level index 0..s+1 occurs (the sample a code is fitted on)"""
    return np.bincount(np.asarray(sym).ravel(), minlength=s + 2).astype(np.uint64)


def num_levels(levelset, s):
    return int(_num_levels(levelset, s))


def level_value(levelset, s, sym):
    return float(_level_value(levelset, s, sym))


def fixed_width(levelset, s):
    return int(_fixed_width(levelset, s))


def norm(v, norm_kind=NORM_L2):
    v = np.ascontiguousarray(v, np.float32)
    return np.float32(_norm(v, v.size, norm_kind))


def bucket_norms(g, bucket, norm_kind=NORM_L2):
    g = np.ascontiguousarray(g, np.float32)
    out = np.zeros((g.size + bucket - 1) // bucket, np.float32)
    _bucket_norms(g, g.size, bucket, norm_kind, out)
    return out


def round_probability(v, nrm, s, levelset=LEVELS_EXP):
    low, p = C.c_uint32(), C.c_float()
    _round_prob(float(v), float(nrm), s, levelset, C.byref(low), C.byref(p))
    return low.value, np.float32(p.value)


def quantize_bucket(v, nrm, s, levelset, seed, offset, i0):
    v = np.ascontiguousarray(v, np.float32)
    sign, sym = np.zeros(v.size, np.uint8), np.zeros(v.size, np.uint16)
    _quant_bucket(v, v.size, float(nrm), s, levelset, seed, offset, i0, sign, sym)
    return sign, sym


def quantize_with_draws(v, nrm, s, levelset, u):
    v = np.ascontiguousarray(v, np.float32)
    u = np.ascontiguousarray(u, np.float32)
    sign, sym = np.zeros(v.size, np.uint8), np.zeros(v.size, np.uint16)
    _quant_draws(v, v.size, float(nrm), s, levelset, u, sign, sym)
    return sign, sym


def dequantize(nrm, s, levelset, sign, sym):
    return np.float32(_dequant(float(nrm), s, levelset, int(sign), int(sym)))


def quantize(g, bucket, s, norm_kind, levelset, seed, offset, norms=None):
    """signs and level indices of a whole vector, bucket by bucket"""
    g = np.ascontiguousarray(g, np.float32)
    if norms is None:
        norms = bucket_norms(g, bucket, norm_kind)
    sign, sym = np.zeros(g.size, np.uint8), np.zeros(g.size, np.uint16)
    for b, lo in enumerate(range(0, g.size, bucket)):
        hi = min(lo + bucket, g.size)
        sg, sy = quantize_bucket(g[lo:hi], norms[b], s, levelset, seed, offset, lo)
        sign[lo:hi], sym[lo:hi] = sg, sy
    return sign, sym, norms


def quantize_dequantize(g, bucket, s, norm_kind, levelset, seed, offset):
    g = np.ascontiguousarray(g, np.float32)
    out = np.zeros_like(g)
    _qdq(g, g.size, bucket, s, norm_kind, levelset, seed, offset, out)
    return out


def variance_closed_form(v, nrm, s, levelset=LEVELS_EXP):
    v = np.ascontiguousarray(v, np.float32)
    return float(_var_cf(v, v.size, float(nrm), s, levelset))


def erc_encode(n):
    """Elias recursive code word of n >= 1 as a '0'/'1' string"""
    buf = np.zeros(160, np.uint8)
    ln = _erc_enc(int(n), buf)
    return "".join(str(int(b)) for b in buf[:ln])


def erc_decode(bits, pos=0):
    """decode one integer from a '0'/'1' string; returns (value, new position), value 0 on overrun"""
    arr = np.frombuffer(bytes(int(c) for c in bits), np.uint8).copy() if len(bits) else np.zeros(1, np.uint8)
    p = C.c_uint64(pos)
    v = _erc_dec(arr, len(bits), C.byref(p))
    return int(v), int(p.value)


def encode_bound(d, bucket, s, flags):
    return int(_bound(d, bucket, s, flags))


def encode(g, bucket, s, flags, seed, offset, norms=None):
    """returns (container as uint32 array trimmed to its valid words, container_bits)"""
    g = np.ascontiguousarray(g, np.float32)
    cap = encode_bound(g.size, bucket, s, flags)
    if cap == 0:
        raise ValueError("invalid arguments")
    out = np.zeros(cap // 4 + 1, np.uint32)
    bits = C.c_uint64()
    nptr = None
    if norms is not None:
        norms = np.ascontiguousarray(norms, np.float32)
        nptr = norms.ctypes.data
    rc = _encode(g, g.size, bucket, s, flags, seed, offset, nptr, out.ctypes.data, out.nbytes, C.byref(bits))
    if rc != 0:
        raise RuntimeError(f"oracle encode failed: {rc}")
    return out[: (bits.value + 31) // 32].copy(), int(bits.value)


def decode_symbols(stream, d, bucket, s):
    stream = np.ascontiguousarray(stream, np.uint32)
    sign, sym = np.zeros(d, np.uint8), np.zeros(d, np.uint16)
    norms = np.zeros((d + bucket - 1) // bucket, np.float32)
    rc = _decode_sym(stream.ctypes.data, d, bucket, s, sign, sym, norms)
    return rc, sign, sym, norms


def decode_accumulate(streams, d, bucket, s):
    streams = [np.ascontiguousarray(x, np.uint32) for x in streams]
    ptrs = (C.c_void_p * len(streams))(*[x.ctypes.data for x in streams])
    acc = np.zeros(d, np.float32)
    rc = _decode_acc(ptrs, len(streams), d, bucket, s, acc)
    return rc, acc


def momentum_step(w, yl, total, alpha, K, mu=0.0, l=0.0):
    """(w_next, yl_next) of the aggregation step with momentum, in fp64; `total` = sum of the K decoded gradients"""
    w = np.array(w, np.float64)
    yl = np.array(yl, np.float64)
    total = np.ascontiguousarray(total, np.float32)
    _momentum(w, yl, total, total.size, float(alpha), int(K), float(mu), float(l))
    return w, yl


def single_chain_bits(sym):
    sym = np.ascontiguousarray(sym, np.uint16)
    return int(_chain_bits(sym, sym.size))


def header(stream):
    w = np.asarray(stream[:HEADER_WORDS], np.uint32).astype(np.uint64)
    u64 = lambda i: int(w[i]) | (int(w[i + 1]) << 32)
    return dict(magic=int(w[0]), version=int(w[1]), d=u64(2), bucket=int(w[4]), s=int(w[5]), flags=int(w[6]),
                sb=int(w[7]), nblk=u64(8), container_bits=u64(10), code_bits=u64(12), nnz=u64(14))
