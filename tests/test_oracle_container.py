"""The oracle's ENCODE / DECODE (App. A) and its container, against hand-built
streams, the round-trip identity and malformed input."""
import numpy as np
import pytest

import oracle as O

ERC, FIXED = O.make_flags(mode=O.MODE_ERC), O.make_flags(mode=O.MODE_FIXED)


def _hand_vector():
    # s = 2: levels 0, 1/4, 1/2, 1.  With norm 1 every entry sits on a level, so no draw matters.
    v = np.array([0.0, 0.5, 0.0, 0.0, -0.25, 1.0, 0.0], np.float32)
    return v, np.array([1.0], np.float32)


def test_erc_stream_built_by_hand():
    """App. A: norm in 32 bits, then per nonzero ERC(gap), sign bit, ERC(level index).
    Tokens: pos 2 -> 100|0|100, pos 5 -> 110|1|0, pos 6 -> 0|0|110  (17 bits)."""
    v, norms = _hand_vector()
    st, bits = O.encode(v, 7, 2, ERC, seed=3, offset=0, norms=norms)
    h = O.header(st)
    assert (h["magic"], h["version"], h["d"], h["bucket"], h["s"], h["flags"], h["sb"]) == \
        (O.MAGIC, 1, 7, 7, 2, 0, 256)
    assert (h["nblk"], h["code_bits"], h["nnz"]) == (1, 17, 3)
    table = st[16:20].view(np.uint64)
    assert list(table) == [0, 96]
    assert [hex(x) for x in st[20:23]] == ["0x3f800000", "0x11", "0x89a30000"]
    assert bits == h["container_bits"] == 32 * 23 and st.size == 23
    rc, sign, sym, nrm = O.decode_symbols(st, 7, 7, 2)
    assert rc == 0 and list(sym) == [0, 2, 0, 0, 1, 3, 0] and list(sign) == [0, 0, 0, 0, 1, 0, 0]
    rc, acc = O.decode_accumulate([st, st], 7, 7, 2)
    assert rc == 0 and list(acc) == [0.0, 1.0, 0.0, 0.0, -0.5, 2.0, 0.0]


def test_fixed_stream_built_by_hand():
    """w = 1 + ceil(log2(4)) = 3 bits: fields 000 010 000 000 101 011 000, MSB first."""
    v, norms = _hand_vector()
    st, bits = O.encode(v, 7, 2, FIXED, seed=3, offset=0, norms=norms)
    h = O.header(st)
    assert (h["nblk"], h["code_bits"], h["nnz"], h["flags"]) == (1, 21, 3, 1 << 16)
    assert [hex(x) for x in st[16:]] == ["0x3f800000", "0x80ac000"]
    assert bits == 32 * 18
    rc, sign, sym, _ = O.decode_symbols(st, 7, 7, 2)
    assert rc == 0 and list(sym) == [0, 2, 0, 0, 1, 3, 0] and list(sign) == [0, 0, 0, 0, 1, 0, 0]


def test_run_restarts_at_sub_block():
    """positions are counted from the start of each 256-element sub-block"""
    v = np.zeros(1024, np.float32)
    v[255], v[256], v[700] = 1.0, 1.0, -1.0
    st, _ = O.encode(v, 1024, 3, ERC, 0, 0, norms=np.array([1.0], np.float32))
    lens = st[21:23].view(np.uint16)
    tok = lambda gap, sg, lev: O.erc_encode(gap) + str(sg) + O.erc_encode(lev)
    want = [len(tok(256, 0, 4)), len(tok(1, 0, 4)), len(tok(700 - 512 + 1, 1, 4)), 0]
    assert list(lens) == want
    bits = "".join(f"{int(x):032b}" for x in st[23:])
    assert bits.startswith(tok(256, 0, 4) + tok(1, 0, 4) + tok(189, 1, 4))
    assert set(bits[sum(want):]) <= {"0"}


CASES = [
    (65536, 1024, 3, O.NORM_L2, O.LEVELS_EXP),
    (5000, 1024, 4, O.NORM_L2, O.LEVELS_EXP),       # ragged last bucket and sub-block
    (20000, 8192, 2, O.NORM_L2, O.LEVELS_EXP),
    (1, 512, 4, O.NORM_L2, O.LEVELS_EXP),
    (257, 256, 1, O.NORM_L2, O.LEVELS_EXP),
    (50000, 20000, 4, O.NORM_L2, O.LEVELS_EXP),     # bucket spans three coding blocks
    (9000, 512, 4, O.NORM_L2, O.LEVELS_UNIFORM),
    (9000, 512, 4, O.NORM_LINF, O.LEVELS_UNIFORM),
    (3000, 300, 8, O.NORM_L2, O.LEVELS_UNIFORM),
    (3000, 100, 14, O.NORM_L2, O.LEVELS_EXP),
]


@pytest.mark.parametrize("d,bucket,s,nk,ls", CASES)
@pytest.mark.parametrize("mode", [O.MODE_ERC, O.MODE_FIXED])
def test_round_trip_identity(d, bucket, s, nk, ls, mode):
    """DECODE(ENCODE(v)) reproduces (norm, signs, levels) exactly and the aggregate is the ordered sum."""
    rng = np.random.default_rng(d + s)
    flags = O.make_flags(nk, ls, mode)
    gs = [(rng.standard_normal(d) * 10.0 ** rng.uniform(-3, 0, d)).astype(np.float32) for _ in range(3)]
    streams, total = [], np.zeros(d, np.float32)
    for k, g in enumerate(gs):
        st, bits = O.encode(g, bucket, s, flags, seed=k + 1, offset=5)
        assert bits % 32 == 0 and bits <= 8 * O.encode_bound(d, bucket, s, flags)
        sign, sym, norms = O.quantize(g, bucket, s, nk, ls, seed=k + 1, offset=5)
        rc, dsign, dsym, dnorms = O.decode_symbols(st, d, bucket, s)
        assert rc == 0
        assert np.array_equal(dsym, sym) and np.array_equal(dsign, sign)
        assert np.array_equal(dnorms.view(np.uint32), norms.view(np.uint32))
        h = O.header(st)
        assert h["nnz"] == np.count_nonzero(sym) and h["container_bits"] == bits
        q = O.quantize_dequantize(g, bucket, s, nk, ls, seed=k + 1, offset=5)
        total = total + q
        streams.append(st)
    rc, acc = O.decode_accumulate(streams, d, bucket, s)
    assert rc == 0 and np.array_equal(acc, total)


def test_block_layout_of_a_wide_bucket():
    d, bucket = 50000, 20000
    g = np.random.default_rng(0).standard_normal(d).astype(np.float32)
    st, _ = O.encode(g, bucket, 4, ERC, 1, 0)
    h = O.header(st)
    assert h["nblk"] == 3 + 3 + 2            # 8192 + 8192 + 3616, twice; then 8192 + 1808
    table = st[16:16 + 2 * (h["nblk"] + 1)].view(np.uint64)
    payload = st[16 + 2 * (h["nblk"] + 1):]
    norms = O.bucket_norms(g, bucket)
    owner = [0, 0, 0, 1, 1, 1, 2, 2]
    for b in range(h["nblk"]):
        assert table[b] % 32 == 0 and table[b] < table[b + 1]
        assert payload[int(table[b]) // 32] == norms[owner[b]].view(np.uint32)
    assert 32 * payload.size == table[-1]


def test_sub_block_restart_only_shortens_the_code():
    g = np.random.default_rng(1).standard_normal(8192).astype(np.float32)
    st, _ = O.encode(g, 8192, 4, ERC, 1, 0)
    _, sym, _ = O.quantize(g, 8192, 4, 0, 0, 1, 0)
    assert O.header(st)["code_bits"] <= O.single_chain_bits(sym) - 32


def test_malformed_streams_are_rejected():
    g = np.random.default_rng(2).standard_normal(4096).astype(np.float32)
    st, _ = O.encode(g, 1024, 3, ERC, 1, 0)
    assert O.decode_symbols(st, 4096, 1024, 3)[0] == 0
    for word, value in ((0, 0), (1, 2), (2, 4095), (4, 512), (5, 4), (7, 128), (8, 5)):
        bad = st.copy(); bad[word] = value
        assert O.decode_symbols(bad, 4096, 1024, 3)[0] == -3
    bad = st.copy(); bad[16 + 2 * 5 + 1] = 0           # norm-only block: offset table shrinks block 0
    bad[18:20] = [64, 0]
    assert O.decode_symbols(bad, 4096, 1024, 3)[0] == -3
    payload0 = 16 + 2 * 5
    bad = st.copy(); bad[payload0 + 1] += 5             # sub-block 0 claims 5 more bits
    assert O.decode_symbols(bad, 4096, 1024, 3)[0] == -3
    bad = st.copy(); bad[payload0 + 3] |= 0xFFFFFFFF    # token soup: level index out of range or overrun
    assert O.decode_symbols(bad, 4096, 1024, 3)[0] == -3
    with pytest.raises(ValueError):
        O.encode(g, 1024, 0, ERC, 1, 0)
    with pytest.raises(ValueError):
        O.encode(g, 1024, 9, O.make_flags(levelset=O.LEVELS_UNIFORM), 1, 0)


def test_c1_reference_statistics():
    """Config C1 (d = 65 536 N(0,1), bucket 1024, s = 3): code density and error of the oracle."""
    from paper_1908_06077_b200 import inputs
    g = inputs.c1_input()
    st, bits = O.encode(g, 1024, 3, ERC, 0, 0)
    h = O.header(st)
    assert 0.15 < h["nnz"] / g.size < 0.25
    assert 1.0 < h["code_bits"] / g.size < 1.6
    rc, acc = O.decode_accumulate([st], g.size, 1024, 3)
    rel = float(((acc - g) ** 2).sum() / (g ** 2).sum())
    assert rc == 0 and 1.5 < rel < 3.125                # below Theorem 1's bound for (1024, 3)


# ---- coded level indices (Sec. 5, "efficient encoding") -------------------------------------------

CODED = O.make_flags(mode=O.MODE_CODED)


def _erc_len(n):
    return len(O.erc_encode(n))


def test_coded_stream_built_by_hand():
    """Lengths (2, 2, 1) for the indices 1, 2, 3 give the words 10, 11, 0.  Tokens ERC(gap) | sign | word:
    pos 2 -> 100|0|11, pos 5 -> 110|1|10, pos 6 -> 0|0|0  (15 bits: 1000 1111 0110 000)."""
    v, norms = _hand_vector()
    O.set_level_code([2, 2, 1])
    st, bits = O.encode(v, 7, 2, CODED, seed=3, offset=0, norms=norms)
    h = O.header(st)
    assert (h["nblk"], h["code_bits"], h["nnz"], h["flags"]) == (1, 15, 3, 2 << 16)
    assert [hex(x) for x in st[16:18]] == ["0x10202", "0x0"]           # the lengths, one byte each
    assert list(st[18:22].view(np.uint64)) == [0, 96]
    assert [hex(x) for x in st[22:25]] == ["0x3f800000", "0xf", "0x8f600000"]
    assert bits == h["container_bits"] == 32 * 25 and st.size == 25
    rc, sign, sym, nrm = O.decode_symbols(st, 7, 7, 2)
    assert rc == 0 and list(sym) == [0, 2, 0, 0, 1, 3, 0] and list(sign) == [0, 0, 0, 0, 1, 0, 0]
    O.set_level_code([1, 2, 2])                              # the decoder reads the code from the container
    rc, acc = O.decode_accumulate([st, st], 7, 7, 2)
    assert rc == 0 and list(acc) == [0.0, 1.0, 0.0, 0.0, -0.5, 2.0, 0.0]


@pytest.mark.parametrize("s, levelset", [(4, O.LEVELS_EXP), (2, O.LEVELS_EXP), (7, O.LEVELS_EXP), (3, O.LEVELS_TABLE)])
def test_coded_mode_sends_the_same_symbols_and_saves_what_the_histogram_says(s, levelset):
    rng = np.random.default_rng(s)
    d, bucket = 20_000, 2048
    g = (rng.standard_t(3, d) * 10.0 ** rng.uniform(-3, 0, d)).astype(np.float32)
    if levelset == O.LEVELS_TABLE:
        O.set_levels(np.array([0.3 ** 3, 0.3 ** 2, 0.3], np.float32))
    erc = O.make_flags(O.NORM_L2, levelset, O.MODE_ERC)
    coded = O.make_flags(O.NORM_L2, levelset, O.MODE_CODED)
    sign, sym, norms = O.quantize(g, bucket, s, O.NORM_L2, levelset, 9, 2)
    hist = O.level_histogram(sym, s)
    assert hist.sum() == d and hist.size == s + 2
    lengths = O.huffman_lengths(hist[1:])
    O.set_level_code(lengths)
    a, abits = O.encode(g, bucket, s, erc, 9, 2)
    b, bbits = O.encode(g, bucket, s, coded, 9, 2)
    rc, sign_b, sym_b, norms_b = O.decode_symbols(b, d, bucket, s)
    assert rc == 0 and np.array_equal(sign_b, sign) and np.array_equal(sym_b, sym) and np.array_equal(norms_b, norms)
    ha, hb = O.header(a), O.header(b)
    saved = sum(int(hist[j]) * (_erc_len(j) - int(lengths[j - 1])) for j in range(1, s + 2))
    assert ha["nnz"] == hb["nnz"] and ha["code_bits"] - hb["code_bits"] == saved
    assert saved >= 0                                        # ERC is a prefix code too, and Huffman's is the cheapest
    assert np.array_equal(O.decode_accumulate([a], d, bucket, s)[1], O.decode_accumulate([b], d, bucket, s)[1])
    assert np.array_equal(O.decode_accumulate([a, b], d, bucket, s)[1], O.decode_accumulate([b, a], d, bucket, s)[1])
    # any other code the lengths allow works as well: here every index gets a word of the same length
    worse = np.full(s + 1, int(np.ceil(np.log2(s + 1))), np.uint8)
    O.set_level_code(worse)
    c, _ = O.encode(g, bucket, s, coded, 9, 2)
    assert O.header(c)["code_bits"] - ha["code_bits"] == sum(int(hist[j]) * (int(worse[j - 1]) - _erc_len(j)) for j in range(1, s + 2))
    assert np.array_equal(O.decode_symbols(c, d, bucket, s)[2], sym)


def test_malformed_coded_streams_are_rejected():
    rng = np.random.default_rng(2)
    g = rng.standard_normal(3000).astype(np.float32)
    O.set_level_code([1, 2, 3, 3])
    st, _ = O.encode(g, 512, 3, CODED, 1, 0)
    assert O.decode_symbols(st, 3000, 512, 3)[0] == 0
    bad = st.copy(); bad[16] = 0x01010101                    # Kraft sum 2: no prefix code
    assert O.decode_symbols(bad, 3000, 512, 3)[0] == -3
    bad = st.copy(); bad[16] = 0x03030200                    # a zero length
    assert O.decode_symbols(bad, 3000, 512, 3)[0] == -3
    bad = st.copy(); bad[16] = 0x04040403                    # an incomplete code: chains that run into an unused word
    assert O.decode_symbols(bad, 3000, 512, 3)[0] == -3
    assert O.encode_bound(3000, 512, 8, CODED) == 0          # more than 8 level indices
    assert O.encode_bound(3000, 512, 4, O.make_flags(O.NORM_L2, O.LEVELS_UNIFORM, O.MODE_CODED)) == 0
    with pytest.raises(Exception):
        O.encode(g, 512, 4, CODED, 1, 0)                     # the code set has 4 words, s = 4 needs 5
