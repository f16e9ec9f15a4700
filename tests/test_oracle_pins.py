"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA path: they make sure that a plausible
mistake in the oracle (a dropped term, a wrong sign or index, a transposed
operand) fails somewhere before the oracle is used to judge the kernels.
"""
import ctypes
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle as O
from conftest import golden_rows


# ---------------------------------------------------------------- levels
def test_level_set_closed_form():
    """Sec. 3.1: L = (0, 2^-s, ..., 1/2, 1); Fig. 1 uses s = 3."""
    for row in golden_rows("levels.txt"):
        s, want = int(row[0]), [Fraction(x) for x in row[1:]]
        assert O.num_levels(O.LEVELS_EXP, s) == len(want) == s + 2
        got = [Fraction(O.level_value(O.LEVELS_EXP, s, j)) for j in range(s + 2)]
        assert got == want
    for s in range(1, 15):
        lv = [O.level_value(O.LEVELS_EXP, s, j) for j in range(s + 2)]
        assert lv[0] == 0.0 and lv[-1] == 1.0 and lv[1] == 2.0 ** -s
        assert all(lv[j + 1] == 2 * lv[j] for j in range(1, s + 1))


def test_uniform_level_set():
    for s in (1, 2, 4, 8):
        n = O.num_levels(O.LEVELS_UNIFORM, s)
        assert n == 2 ** s + 1
        assert [O.level_value(O.LEVELS_UNIFORM, s, k) for k in range(n)] == [k / 2 ** s for k in range(n)]


def test_fixed_width():
    # sign bit + ceil(log2(number of levels))
    assert [O.fixed_width(O.LEVELS_EXP, s) for s in (1, 2, 3, 4, 6, 7)] == [3, 3, 4, 4, 4, 5]
    assert [O.fixed_width(O.LEVELS_UNIFORM, s) for s in (1, 2, 4, 8)] == [3, 4, 6, 10]


# ---------------------------------------------------------------- ERC
def _erc_len(n):
    return 1 if n == 1 else n.bit_length() + _erc_len(n.bit_length() - 1)


def test_erc_codewords_by_hand():
    """Algorithm 2 executed by hand (tests/golden/erc_codewords.txt)."""
    for n, word in golden_rows("erc_codewords.txt"):
        assert O.erc_encode(int(n)) == word
        assert O.erc_decode(word) == (int(n), len(word))


def test_erc_lengths_and_round_trip():
    # |ERC(N)| = floor(log2 N)+1 + |ERC(floor(log2 N))|, |ERC(1)| = 1  (App. A, property 1)
    ns = list(range(1, 1 << 13)) + [2 ** k + j for k in range(13, 40) for j in (-1, 0, 1)]
    for n in ns:
        w = O.erc_encode(n)
        assert len(w) == _erc_len(n)
        assert O.erc_decode(w) == (n, len(w))
        assert w[-1] == "0" and (n == 1 or w[0] == "1")
    assert [_erc_len(n) for n in (32, 64, 128, 256, 65536)] == [12, 13, 14, 16, 28]


def test_erc_prefix_free_concatenation():
    # decoding without knowing an upper bound on N (App. A, property 3)
    rng = np.random.default_rng(5)
    vals = [int(v) for v in rng.integers(1, 5000, 400)] + [1, 1, 2, 1, 3]
    s = "".join(O.erc_encode(v) for v in vals)
    pos, out = 0, []
    while pos < len(s):
        v, pos = O.erc_decode(s, pos)
        out.append(v)
    assert out == vals
    # a truncated string is reported, not misread
    assert O.erc_decode(O.erc_encode(100)[:-3])[0] == 0


def test_erc_is_prefix_code_small():
    words = [O.erc_encode(n) for n in range(1, 600)]
    assert len(set(words)) == len(words)
    wl = sorted(words)
    for a, b in zip(wl, wl[1:]):
        assert not b.startswith(a)


# ---------------------------------------------------------------- Philox
def _curand_host(seed, n_words, offset=0):
    try:
        lib = ctypes.CDLL("libcurand.so.10")
    except OSError:
        try:
            lib = ctypes.CDLL("/usr/local/cuda/lib64/libcurand.so.10")
        except OSError:
            pytest.skip("libcurand not available")
    gen = ctypes.c_void_p()
    if lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) != 0:  # CURAND_RNG_PSEUDO_PHILOX4_32_10
        pytest.skip("cuRAND host generator not available")
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
    assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(offset)) == 0
    out = np.zeros(n_words, np.uint32)
    assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(n_words)) == 0
    lib.curandDestroyGenerator(gen)
    return out


def test_philox_against_curand_host_generator():
    """An independent Philox4x32-10: cuRAND's host generator emits, as words 4n..4n+3 of its
    sequence, the Philox output for the counter (m_lo, m_hi, n mod 2^16, 0), m = n div 2^16,
    under key = seed (65536 interleaved subsequences)."""
    def block(n, key):
        m = n >> 16
        return O.philox4x32_10([m & 0xFFFFFFFF, m >> 32, n & 0xFFFF, 0], key)

    for seed in (0, 1, 0x0123456789ABCDEF, 0xFFFFFFFFFFFFFFFF):
        key = [seed & 0xFFFFFFFF, seed >> 32]
        ref = _curand_host(seed, 4 * 300)
        assert np.array_equal(ref, np.concatenate([block(n, key) for n in range(300)]))
        for first in (1, 7, 65534, 123456, (1 << 48) + 5, (0x2BCD << 48) + 0xFFFFFFFFFFFE):
            ref = _curand_host(seed, 4 * 8, offset=4 * first)
            assert np.array_equal(ref, np.concatenate([block(first + n, key) for n in range(8)])), (seed, first)


def test_draw_mapping_and_uniformity():
    seed, offset = 0xDEADBEEF12345678, 0x1_0000_0007
    for i in (0, 1, 2, 3, 4, 5, 1023, (1 << 34) + 6):
        q = i >> 2
        blk = O.philox4x32_10([q & 0xFFFFFFFF, q >> 32, offset & 0xFFFFFFFF, offset >> 32],
                              [seed & 0xFFFFFFFF, seed >> 32])
        assert O.draw_word(seed, offset, i) == int(blk[i & 3])
        assert O.draw_uniform(seed, offset, i) == (int(blk[i & 3]) >> 8) / 2.0 ** 24
    # every counter and key word matters
    base = O.philox4x32_10([1, 2, 3, 4], [5, 6])
    for w in range(4):
        c = [1, 2, 3, 4]; c[w] ^= 1
        assert not np.array_equal(base, O.philox4x32_10(c, [5, 6]))
    assert not np.array_equal(base, O.philox4x32_10([1, 2, 3, 4], [4, 6]))
    assert not np.array_equal(base, O.philox4x32_10([1, 2, 3, 4], [5, 7]))
    # u in [0,1), mean 1/2, variance 1/12, flat histogram
    u = np.array([O.draw_uniform(7, 0, i) for i in range(200000)])
    assert 0.0 <= u.min() and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 4 * math.sqrt(1 / 12 / u.size)
    assert abs(u.var() - 1 / 12) < 2e-3
    hist = np.histogram(u, bins=64, range=(0, 1))[0]
    chi2 = ((hist - u.size / 64) ** 2 / (u.size / 64)).sum()
    assert chi2 < 63 + 5 * math.sqrt(2 * 63)


# ---------------------------------------------------------------- norm
def test_norms():
    rng = np.random.default_rng(1)
    g = (rng.standard_normal(5000) * 10.0 ** rng.uniform(-6, 2, 5000)).astype(np.float32)
    n = O.bucket_norms(g, 1024)
    assert n.size == 5
    for b in range(5):
        seg = g[b * 1024:(b + 1) * 1024].astype(np.float64)
        assert n[b] == np.float32(math.sqrt(float((seg * seg).sum()))) or \
            abs(float(n[b]) - math.sqrt(float((seg * seg).sum()))) <= 1.2e-7 * float(n[b])
    ninf = O.bucket_norms(g, 1024, O.NORM_LINF)
    assert [float(x) for x in ninf] == [float(np.abs(g[b * 1024:(b + 1) * 1024]).max()) for b in range(5)]
    assert O.norm(np.array([3.0, -4.0], np.float32)) == 5.0
    assert O.norm(np.zeros(7, np.float32)) == 0.0


# ---------------------------------------------------------------- Definition 1
def _exact_split(v, nrm, s):
    """lower level index and exact probability from the real-number definition:
    r = |v|/||v||, l_j <= r <= l_{j+1}, p = (r - l_j)/(l_{j+1} - l_j)."""
    r = Fraction(abs(float(v))) / Fraction(float(nrm))
    lv = [Fraction(0)] + [Fraction(1, 2 ** (s + 1 - j)) for j in range(1, s + 2)]
    j = max(k for k in range(s + 1) if lv[k] <= r)
    return j, (r - lv[j]) / (lv[j + 1] - lv[j])


def test_rounding_probability_matches_definition():
    """App. B: p_1 = 2^s r on [0, 2^-s], p_2 = 2^(s-j) r - 1 on [2^(j-s), 2^(j+1-s)]."""
    rng = np.random.default_rng(2)
    for s in (1, 3, 4, 7):
        for _ in range(300):
            nrm = np.float32(10.0 ** rng.uniform(-3, 3))
            v = np.float32(nrm * rng.uniform(0, 1) ** 3 * rng.choice([-1, 1]))
            low, p = O.round_probability(v, nrm, s)
            j, pe = _exact_split(v, nrm, s)
            # fp32: one rounding in 2^s/norm and one in the product; the affine map is exact
            assert abs(Fraction(float(p)) + low - (pe + j)) <= Fraction(3, 2 ** 24) * max(1, 2 ** j)
            assert 0 <= p <= 1
    # exact cases: r on a level and midway between levels
    assert O.round_probability(0.25, 1.0, 3) in ((2, 0.0), (1, 1.0))
    assert O.round_probability(0.1875, 1.0, 3) == (1, 0.5)     # midway between 1/8 and 1/4 (Fig. 1)
    assert O.round_probability(-0.0625, 1.0, 3) == (0, 0.5)
    assert O.round_probability(0.75, 1.0, 3) == (3, 0.5)
    assert O.round_probability(1.0, 1.0, 3) == (3, 1.0)
    assert O.round_probability(0.0, 1.0, 3) == (0, 0.0)


def test_rounding_frequency_over_all_draws():
    """Enumerate every 24-bit draw: #(u < p) = ceil(p 2^24); equal to p 2^24 when r >= 2^-s."""
    u = (np.arange(1 << 24, dtype=np.float64) / 2.0 ** 24).astype(np.float32)
    for s, v, nrm in ((3, 0.3, 1.0), (4, 0.01, 1.0), (3, 0.7, 2.0), (2, 1e-5, 0.003)):
        v32, n32 = np.float32(v), np.float32(nrm)
        low, p = O.round_probability(v32, n32, s)
        sign, sym = O.quantize_with_draws(np.full(u.size, v32, np.float32), n32, s, O.LEVELS_EXP, u)
        ups = int((sym == low + 1).sum())
        assert int((sym == low).sum()) + ups == u.size
        assert ups == math.ceil(Fraction(float(p)) * 2 ** 24)
        if low >= 1:
            assert Fraction(ups, 2 ** 24) == Fraction(float(p))
        assert not sign.any()


def test_unbiased_by_full_enumeration():
    """Theorem 1, first claim: E[Q_s(v)] = v.  Enumerate all 2^d outcomes of a tiny vector."""
    rng = np.random.default_rng(3)
    for s, d in ((3, 8), (2, 10), (4, 6)):
        v = (rng.standard_normal(d) * 10.0 ** rng.uniform(-2, 0, d)).astype(np.float32)
        nrm = O.norm(v)
        split = [O.round_probability(x, nrm, s) for x in v]
        mean = [Fraction(0)] * d
        total = Fraction(0)
        for ups in itertools.product((0, 1), repeat=d):
            u = np.array([0.0 if b else 0.99999994 for b in ups], np.float32)
            pr = Fraction(1)
            for b, (_, p) in zip(ups, split):
                pr *= Fraction(float(p)) if b else 1 - Fraction(float(p))
            if pr == 0:
                continue
            sign, sym = O.quantize_with_draws(v, nrm, s, O.LEVELS_EXP, u)
            for i in range(d):
                assert sym[i] == split[i][0] + (1 if (ups[i] and split[i][1] > 0) else 0)
                q = O.dequantize(nrm, s, O.LEVELS_EXP, sign[i], sym[i])
                mean[i] += pr * Fraction(float(q))
            total += pr
        assert total == 1
        for i in range(d):
            assert abs(float(mean[i]) - float(v[i])) <= 4e-7 * float(nrm)


def test_unbiased_and_variance_monte_carlo():
    """E[Q] = v and Lemma 7's closed form, on one N(0,1) bucket of 1024 with s = 3."""
    v = np.random.default_rng(4).standard_normal(1024).astype(np.float32)
    s, reps = 3, 4000
    nrm = O.norm(v)
    acc = np.zeros(1024)
    err2 = np.zeros(reps)
    for t in range(reps):
        q = O.quantize_dequantize(v, 1024, s, O.NORM_L2, O.LEVELS_EXP, seed=1000 + t, offset=0).astype(np.float64)
        acc += q
        err2[t] = ((q - v) ** 2).sum()
    var_cf = O.variance_closed_form(v, nrm, s)
    # mean of err2 against the closed form, 4 standard errors
    assert abs(err2.mean() - var_cf) < 4 * err2.std() / math.sqrt(reps)
    # ||mean Q - v||^2 has expectation var_cf / reps
    bias2 = ((acc / reps - v) ** 2).sum()
    assert bias2 < 1.5 * var_cf / reps
    assert bias2 > 0.5 * var_cf / reps          # and it is not suspiciously deterministic
    # different offsets give different draws
    a = O.quantize_dequantize(v, 1024, s, 0, 0, seed=1, offset=0)
    b = O.quantize_dequantize(v, 1024, s, 0, 0, seed=1, offset=1)
    assert not np.array_equal(a, b)


def test_variance_closed_form_worked_examples():
    """Lemma 7 on the all-equal vectors of Theorem 4 and Theorem 12."""
    for d, s, frac in golden_rows("worked_examples.txt"):
        d, s = int(d), int(s)
        v = np.full(d, 0.37, np.float32)
        nrm = O.norm(v)
        got = O.variance_closed_form(v, nrm, s) / float(nrm) ** 2
        assert abs(got - float(Fraction(frac))) < 2e-6 * max(1.0, float(Fraction(frac)))


def _eps_q(d, s):
    """Theorem 1's bound with the switch placed where its derivation puts it
    (delta = sqrt(d)/2^s >= 2); never below the printed bound's first branch."""
    delta = math.sqrt(d) / 2 ** s
    return 1 / 8 + delta * delta / 4 if delta < 2 else delta - 7 / 8


def test_variance_bound_theorem_1():
    rng = np.random.default_rng(6)
    for d, s in ((1024, 3), (8192, 4), (8192, 2), (512, 4), (64, 3)):
        for kind in range(4):
            if kind == 0:
                v = rng.standard_normal(d)
            elif kind == 1:
                v = rng.standard_t(3, d)
            elif kind == 2:
                v = np.full(d, 1.0)
            else:
                v = rng.laplace(0, 1, d) * (rng.random(d) < 0.1)
                v[0] = 1.0
            v = v.astype(np.float32)
            nrm = O.norm(v)
            assert O.variance_closed_form(v, nrm, s) <= _eps_q(d, s) * float(nrm) ** 2 * (1 + 1e-6)
    assert [round(_eps_q(b, s), 3) for b, s in ((1024, 3), (8192, 4), (8192, 3), (8192, 2), (65536, 4))] == \
        [3.125, 4.782, 10.439, 21.752, 15.125]


def test_sparsity_lemma_10():
    """#{r_i > 2^-s} <= 2^(2s), and E||Q||_0 <= 2^(2s) + 2^s sqrt(d)."""
    rng = np.random.default_rng(8)
    for d, s in ((1024, 3), (8192, 4), (8192, 2)):
        v = rng.standard_t(3, d).astype(np.float32)
        nrm = float(O.norm(v))
        r = np.abs(v.astype(np.float64)) / nrm
        assert (r > 2.0 ** -s).sum() <= 2 ** (2 * s)
        e_nnz = (r >= 2.0 ** -s).sum() + (2.0 ** s * r[r < 2.0 ** -s]).sum()
        assert e_nnz <= 2 ** (2 * s) + 2 ** s * math.sqrt(d)
        cnt = [np.count_nonzero(O.quantize(v, d, s, 0, 0, seed=t, offset=0)[1]) for t in range(200)]
        assert abs(np.mean(cnt) - e_nnz) < 5 * math.sqrt(e_nnz / 200)


def test_uniform_quantizer_definition():
    """QSGD-style levels k/2^s: p = 2^s r - floor(2^s r); QSGD's variance bound min(d/s'^2, sqrt(d)/s')."""
    assert O.round_probability(0.40625, 1.0, 4, O.LEVELS_UNIFORM) == (6, 0.5)
    assert O.round_probability(1.0, 1.0, 4, O.LEVELS_UNIFORM) == (15, 1.0)
    assert O.round_probability(0.01, 1.0, 4, O.LEVELS_UNIFORM)[0] == 0
    v = np.random.default_rng(9).standard_normal(8192).astype(np.float32)
    nrm = O.norm(v)
    var = O.variance_closed_form(v, nrm, 4, O.LEVELS_UNIFORM) / float(nrm) ** 2
    assert var <= min(8192 / 16 ** 2, math.sqrt(8192) / 16)
    # L-infinity normalisation: r <= 1 exactly, the largest coordinate maps to the top level
    ninf = O.norm(v, O.NORM_LINF)
    sign, sym = O.quantize_bucket(v, ninf, 4, O.LEVELS_UNIFORM, 1, 0, 0)
    assert sym.max() == 16 and sym[np.argmax(np.abs(v))] == 16
    q = np.array([O.dequantize(ninf, 4, O.LEVELS_UNIFORM, a, b) for a, b in zip(sign, sym)])
    assert np.abs(q - v).max() <= float(ninf) / 16 * (1 + 1e-6)


def test_degenerate_buckets():
    z = np.zeros(300, np.float32)
    sign, sym, norms = O.quantize(z, 128, 3, 0, 0, 1, 0)
    assert not sym.any() and not sign.any() and not norms.any()
    v = np.ones(256, np.float32); v[7] = np.nan
    assert not O.quantize(v, 256, 3, 0, 0, 1, 0)[1].any()
    v[7] = np.inf
    assert not O.quantize(v, 256, 3, 0, 0, 1, 0)[1].any()
    v = np.full(256, 1e-42, np.float32)            # 2^s / norm overflows
    assert not O.quantize(v, 256, 4, 0, 0, 1, 0)[1].any()
    v = np.array([-0.0, 0.0, 1.0, -1.0], np.float32)
    sign, sym, _ = O.quantize(v, 4, 3, 0, 0, 1, 0)
    assert list(sym[:2]) == [0, 0] and list(sign[:2]) == [0, 0] and sign[3] == 1 and sign[2] == 0


# ---------------------------------------------------------------- general level sequences (Sec. 3.3)
def _lp_levels(p, s):
    """interior levels of L_p = (0, p^s, ..., p^2, p, 1) as exact fractions"""
    return [Fraction(p) ** (s + 1 - j) for j in range(1, s + 1)]


def test_level_table_is_the_sequence_it_was_given():
    for p, s in ((Fraction(1, 3), 3), (Fraction(3, 10), 5), (Fraction(1, 2), 4)):
        want = _lp_levels(p, s)
        lv32 = np.array([float(x) for x in want], np.float32)
        O.set_levels(lv32)
        assert O.num_levels(O.LEVELS_TABLE, s) == s + 2
        got = [O.level_value(O.LEVELS_TABLE, s, j) for j in range(s + 2)]
        assert got[0] == 0.0 and got[-1] == 1.0
        assert [np.float32(x) for x in got[1:-1]] == list(lv32)
        assert all(abs(Fraction(float(g)) - w) <= w * Fraction(1, 2 ** 23) for g, w in zip(got[1:-1], want))
    # p = 1/2 is the paper's own level set
    O.set_levels(np.array([2.0 ** -(4 - j) for j in range(4)], np.float32))
    assert [O.level_value(O.LEVELS_TABLE, 4, j) for j in range(6)] == [O.level_value(O.LEVELS_EXP, 4, j) for j in range(6)]
    for bad in ([0.5, 0.25], [0.0, 0.5], [0.5, 1.0], [0.3, 0.3], [float("nan")]):
        with pytest.raises(ValueError):
            O.set_levels(np.array(bad, np.float32))


def test_level_table_rounding_probability_against_exact_arithmetic():
    """p = (r - l_j) / (l_{j+1} - l_j) (Definition 1 for a general sequence, Sec. 3.3) in exact rational
    arithmetic on the fp32 inputs; the oracle's fp32 value may differ by its few roundings only, and of
    all 2^24 draws exactly ceil(p 2^24) move the coordinate up."""
    lv = np.array([0.027, 0.09, 0.3], np.float32)
    O.set_levels(lv)
    levels = [Fraction(0)] + [Fraction(float(x)) for x in lv] + [Fraction(1)]
    norm = np.float32(3.7)
    draws = (np.arange(1 << 24, dtype=np.float64) / (1 << 24)).astype(np.float32)
    for v in (0.01, -0.2, 0.5, 1.0, -2.9, 3.6999):
        v32 = np.float32(v)
        low, p = O.round_probability(v32, norm, 3, O.LEVELS_TABLE)
        r = abs(Fraction(float(v32))) / Fraction(float(norm))
        j = max(k for k in range(5) if levels[k] <= r)
        assert low == j
        exact = (r - levels[j]) / (levels[j + 1] - levels[j])
        assert abs(Fraction(float(p)) - exact) <= Fraction(1, 10 ** 6)
        sign, sym = O.quantize_with_draws(np.full(1 << 24, v32, np.float32), norm, 3, O.LEVELS_TABLE, draws)
        ups = int((sym == j + 1).sum())
        assert ups + int((sym == j).sum()) == 1 << 24
        assert ups == math.ceil(Fraction(float(p)) * (1 << 24))
        assert (sign == (1 if v < 0 else 0)).all() or j == 0
    # r = 1 exactly, and r > 1 from a norm that is too small: the top level, never above it
    assert O.round_probability(np.float32(4.0), np.float32(4.0), 3, O.LEVELS_TABLE) == (4, np.float32(0.0))
    assert O.round_probability(np.float32(5.0), norm, 3, O.LEVELS_TABLE) == (4, np.float32(0.0))
    low, p = O.round_probability(norm, norm, 3, O.LEVELS_TABLE)        # |v| * fl(1 / norm) may fall one place short of 1
    assert (low, p) == (4, np.float32(0.0)) or (low == 3 and p >= 1.0 - 2.0 ** -22)


def test_level_table_unbiased_by_enumeration():
    """E[Q(v)] = v for any level sequence (Sec. 3.3): all 2^d up/down outcomes of a tiny vector with the
    oracle's own probabilities."""
    O.set_levels(np.array([0.05, 0.2, 0.6], np.float32))
    v = np.array([0.3, -1.1, 0.02, 0.7, -0.45, 2.0], np.float32)
    norm = O.norm(v)
    lows, ps = zip(*[O.round_probability(x, norm, 3, O.LEVELS_TABLE) for x in v])
    mean = np.zeros(v.size)
    for ups in itertools.product((0, 1), repeat=v.size):
        prob = np.prod([float(p) if u else 1.0 - float(p) for u, p in zip(ups, ps)])
        q = [float(O.dequantize(norm, 3, O.LEVELS_TABLE, x < 0, low + u)) for x, low, u in zip(v, lows, ups)]
        mean += prob * np.array(q)
    assert np.abs(mean - v).max() <= 1e-6 * float(norm)


def test_level_table_variance_closed_form_by_hand_and_by_monte_carlo():
    """Lemma 7 for sequences other than the paper's (tests/golden/general_levels.txt), then the same
    closed form against the sample variance of the quantizer itself."""
    for p, s, d, want in golden_rows("general_levels.txt"):
        p, s, d, want = Fraction(p), int(s), int(d), Fraction(want)
        O.set_levels(np.array([float(x) for x in _lp_levels(p, s)], np.float32))
        v = np.full(d, 0.75, np.float32)
        norm = O.norm(v)
        got = O.variance_closed_form(v, norm, s, O.LEVELS_TABLE) / float(norm) ** 2
        assert abs(got - float(want)) <= 1e-6, (p, s, d, got)
    O.set_levels(np.array([0.3 ** 3, 0.3 ** 2, 0.3], np.float32))
    rng = np.random.default_rng(7)
    v = (rng.standard_normal(512) * 10.0 ** rng.uniform(-2, 0, 512)).astype(np.float32)
    norm = O.norm(v)
    cf = O.variance_closed_form(v, norm, 3, O.LEVELS_TABLE)
    errs = []
    for seed in range(400):
        sign, sym = O.quantize_bucket(v, norm, 3, O.LEVELS_TABLE, seed, 0, 0)
        q = np.array([float(O.dequantize(norm, 3, O.LEVELS_TABLE, a, b)) for a, b in zip(sign, sym)])
        errs.append(float(((q - v.astype(np.float64)) ** 2).sum()))
    assert abs(np.mean(errs) - cf) <= 4 * np.std(errs) / math.sqrt(len(errs))


def test_level_table_container():
    """The container of a level-table stream carries the s interior levels behind the header (padded to an
    even number of words); everything else is laid out as for the paper's levels."""
    lv = np.array([0.3 ** 3, 0.3 ** 2, 0.3], np.float32)
    O.set_levels(lv)
    rng = np.random.default_rng(3)
    g = (rng.standard_normal(3000) * 10.0 ** rng.uniform(-3, 0, 3000)).astype(np.float32)
    for mode in (O.MODE_ERC, O.MODE_FIXED):
        flags = O.make_flags(O.NORM_L2, O.LEVELS_TABLE, mode)
        st, bits = O.encode(g, 512, 3, flags, 5, 1)
        assert bits == 32 * st.size and O.header(st)["flags"] == flags
        assert np.array_equal(st[16:19].view(np.float32), lv) and st[19] == 0           # 3 levels + a pad word
        rc, sign, sym, norms = O.decode_symbols(st, g.size, 512, 3)
        assert rc == 0
        s2, y2, n2 = O.quantize(g, 512, 3, O.NORM_L2, O.LEVELS_TABLE, 5, 1)
        assert np.array_equal(sign, s2) and np.array_equal(sym, y2) and np.array_equal(norms, n2)
        rc, acc = O.decode_accumulate([st], g.size, 512, 3)
        assert rc == 0 and np.array_equal(acc, O.quantize_dequantize(g, 512, 3, O.NORM_L2, O.LEVELS_TABLE, 5, 1))
        # the decoder takes the levels from the container, not from the table that happens to be set
        O.set_levels(np.array([0.1, 0.2, 0.4], np.float32))
        assert np.array_equal(O.decode_accumulate([st], g.size, 512, 3)[1], acc)
        O.set_levels(lv)
        bad = st.copy()
        bad[17] = bad[16]                                                                # not increasing
        assert O.decode_symbols(bad, g.size, 512, 3)[0] == -3
    # with the paper's levels in the table every symbol stands for the same value as in the paper's level set
    O.set_levels(np.array([2.0 ** -3, 2.0 ** -2, 2.0 ** -1], np.float32))
    for sym in range(5):
        assert O.dequantize(np.float32(1.7), 3, O.LEVELS_TABLE, 1, sym) == O.dequantize(np.float32(1.7), 3, O.LEVELS_EXP, 1, sym)


# ---- coded level indices (Sec. 5, "efficient encoding") -------------------------------------------

def test_huffman_lengths_and_code_words_of_hand_worked_trees():
    for row in golden_rows("level_codes.txt"):
        n = int(row[0])
        weights = [int(x) for x in row[1:1 + n]]
        lengths = [int(x) for x in row[1 + n:1 + 2 * n]]
        words = row[1 + 2 * n:1 + 3 * n]
        assert list(O.huffman_lengths(weights)) == lengths, weights
        O.set_level_code(lengths)
        assert ["".join(str(b) for b in O.level_code(j)) for j in range(1, n + 1)] == words, weights
        assert len(O.level_code(0)) == 0 and len(O.level_code(n + 1)) == 0


def test_huffman_cost_is_the_least_of_any_prefix_code():
    """A prefix code with lengths l_i exists iff sum 2^-l_i <= 1 (Kraft); the Huffman lengths reach the
    least sum w_i l_i over all of them, and fill the Kraft sum exactly."""
    rng = np.random.default_rng(11)
    for n in (2, 3, 4, 5, 6):
        grids = np.stack(np.meshgrid(*[np.arange(1, 8)] * n, indexing="ij"), -1).reshape(-1, n)
        feasible = grids[(2.0 ** -grids).sum(1) <= 1.0]
        for trial in range(6):
            w = rng.integers(0, 5 if trial % 2 else 1000, n).astype(np.uint64)
            ln = O.huffman_lengths(w).astype(np.int64)
            assert sum(Fraction(1, 2 ** int(l)) for l in ln) == 1
            assert int((w.astype(np.int64) * ln).sum()) == int((feasible * w.astype(np.int64)).sum(1).min()), (w, ln)


def test_level_code_words_are_prefix_free_and_bad_lengths_are_refused():
    for lengths in ([1, 2, 3, 3], [2, 2, 2, 3, 4, 4], [3, 3, 3, 3, 3, 3, 3, 3], [1, 7], [2, 3, 1]):
        O.set_level_code(lengths)                            # Kraft sum <= 1: incomplete codes are codes too
        words = ["".join(str(b) for b in O.level_code(j)) for j in range(1, len(lengths) + 1)]
        assert [len(w) for w in words] == lengths
        for a in range(len(words)):
            for b in range(len(words)):
                assert a == b or not words[b].startswith(words[a])
    for lengths in ([1, 1, 2], [0, 1], [1, 8], [2], [1] * 9, [1, 2, 3, 3, 3]):
        with pytest.raises(ValueError):
            O.set_level_code(lengths)


def test_momentum_step_worked_by_hand():
    """The aggregation step of Algorithm 1 and its momentum form (tests/golden/momentum_steps.txt)."""
    for w, yl, total, alpha, K, mu, l, w_next, yl_next in golden_rows("momentum_steps.txt"):
        got_w, got_yl = O.momentum_step([float(w)], [float(yl)], [float(total)], float(alpha), int(K), float(mu), float(l))
        assert got_w[0] == float(w_next) and got_yl[0] == float(yl_next), (w, yl, total)


def test_momentum_step_is_heavy_ball_and_nesterov_in_their_velocity_forms():
    """Sec. 4: l = 0 gives the heavy-ball method, l = 1 Nesterov's.  Both are iterated here in their
    velocity forms (v <- mu v - alpha grad, w <- w + v; for Nesterov the gradient at the look-ahead point
    theta + mu v, whose sequence is the rule's w) on a quadratic, K workers sending the same gradient."""
    rng = np.random.default_rng(5)
    n, K, alpha, mu = 6, 4, 0.05, 0.8                     # (K a power of two: K times a gradient is exact in fp32)
    m = rng.standard_normal((n, n))
    a = m @ m.T / n + 0.5 * np.eye(n)                       # gradient of w' A w / 2 is A w
    w0 = rng.standard_normal(n)
    for l in (0.0, 1.0):
        w, yl = w0.copy(), w0.copy()                        # the rule starts from y^l_0 = w_0, i.e. from rest
        theta, v = w0.copy(), np.zeros(n)
        for step in range(60):
            grad = (a @ w).astype(np.float32)               # what the K workers send, exactly representable sums
            w, yl = O.momentum_step(w, yl, K * grad.astype(np.float64), alpha, K, mu, l)
            if l == 0.0:
                v = mu * v - alpha * grad.astype(np.float64)
                theta = theta + v
                want = theta
            else:
                v = mu * v - alpha * grad.astype(np.float64)    # grad was taken at theta + mu v (= w, see below)
                theta = theta + v
                want = theta + mu * v
            assert np.allclose(w, want, rtol=0, atol=1e-12 * (1 + np.abs(want).max())), (l, step)
        assert np.linalg.norm(w) < 0.5 * np.linalg.norm(w0)        # and it does descend


def test_momentum_step_fixed_point_and_plain_sgd():
    w = np.array([1.5, -2.0, 0.0]); zero = np.zeros(3, np.float32)
    for mu, l in ((0.0, 0.0), (0.9, 0.0), (0.9, 1.0), (0.5, 0.3)):
        got_w, got_yl = O.momentum_step(w, w, zero, 0.1, 4, mu, l)
        assert np.array_equal(got_w, w) and np.array_equal(got_yl, w)     # no gradient, at rest: nothing moves
    total = np.array([8.0, -4.0, 2.0], np.float32)
    got_w, _ = O.momentum_step(w, w, total, 0.25, 8, 0.0, 0.0)
    assert np.array_equal(got_w, np.array([1.5 - 0.25, -2.0 + 0.125, -0.0625]))   # w - (alpha / K) sum
