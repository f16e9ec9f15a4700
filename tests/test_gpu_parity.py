"""Element-by-element parity of the CUDA path (through the C ABI) with the CPU
oracle on seeded inputs: sizes span several tiles and ragged tails."""
import numpy as np
import pytest

import oracle as O
from gpu_util import compare_symbols, gpu_decode, gpu_encode, require_cuda

pytestmark = pytest.mark.gpu

L2, LINF = O.NORM_L2, O.NORM_LINF
EXP, UNI = O.LEVELS_EXP, O.LEVELS_UNIFORM

# (d, bucket, s, norm, levels)
CASES = [
    (65536, 1024, 3, L2, EXP),
    (100037, 8192, 4, L2, EXP),
    (20000, 512, 4, L2, EXP),
    (3 * 8192 + 5, 256, 2, L2, EXP),
    (70000, 768, 3, L2, EXP),
    (200000, 65536, 4, L2, EXP),
    (150001, 16384, 4, L2, EXP),
    (40000, 8192, 14, L2, EXP),
    (40000, 2048, 1, L2, EXP),
    (50000, 8192, 4, L2, UNI),
    (50000, 8192, 4, LINF, UNI),
    (30000, 4096, 8, L2, UNI),
    (90000, 32768, 3, LINF, EXP),
    (1, 512, 4, L2, EXP),
    (255, 256, 3, L2, EXP),
    (256, 256, 3, L2, EXP),
    (257, 256, 3, L2, EXP),
    (8193, 8192, 4, L2, EXP),
]


def _input(d, seed):
    rng = np.random.default_rng(seed)
    g = rng.standard_normal(d) * 10.0 ** rng.uniform(-4, 0, d)
    g[rng.random(d) < 0.02] = 0.0
    return g.astype(np.float32)


@pytest.mark.parametrize("d,bucket,s,nk,ls", CASES)
@pytest.mark.parametrize("mode", [O.MODE_ERC, O.MODE_FIXED])
def test_bitstream_exact_with_oracle_norms(d, bucket, s, nk, ls, mode):
    """Fed the oracle's bucket norms, the GPU container equals the oracle's bit for bit."""
    flags = O.make_flags(nk, ls, mode)
    g = _input(d, d + s)
    norms = O.bucket_norms(g, bucket, nk)
    want, want_bits = O.encode(g, bucket, s, flags, seed=11, offset=3, norms=norms)
    got, got_bits = gpu_encode(g, bucket, s, flags, seed=11, offset=3, norms=norms)
    assert got_bits == want_bits
    assert np.array_equal(got[:16], want[:16]), "header"
    assert np.array_equal(got, want)


@pytest.mark.parametrize("d,bucket,s,nk,ls", CASES)
def test_free_running_encode_matches_oracle(d, bucket, s, nk, ls):
    """The GPU's own norms agree to 1e-6; signs and levels are equal except within 1e-6 of a threshold."""
    flags = O.make_flags(nk, ls, O.MODE_ERC)
    g = _input(d, 7 * d + s)
    got, _ = gpu_encode(g, bucket, s, flags, seed=5, offset=0)
    compare_symbols(g, bucket, s, flags, 5, 0, got)
    got_fixed, _ = gpu_encode(g, bucket, s, O.make_flags(nk, ls, O.MODE_FIXED), seed=5, offset=0)
    compare_symbols(g, bucket, s, flags, 5, 0, got_fixed)


@pytest.mark.parametrize("d,bucket,s,nk,ls", CASES)
@pytest.mark.parametrize("K", [1, 3])
def test_decode_accumulate_matches_oracle(d, bucket, s, nk, ls, K):
    """GPU decode of oracle-written containers equals the oracle's ordered sum bit for bit."""
    streams = []
    for k in range(K):
        mode = O.MODE_FIXED if (k == 1) else O.MODE_ERC          # mixed modes in one call
        g = _input(d, 1000 * k + d)
        streams.append(O.encode(g, bucket, s, O.make_flags(nk, ls, mode), seed=k + 1, offset=0)[0])
    rc, want = O.decode_accumulate(streams, d, bucket, s)
    assert rc == 0
    got = gpu_decode(streams, d, bucket, s)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_c1_end_to_end():
    """Config C1: encode on the GPU, decode on the GPU, against the oracle end to end."""
    from paper_1908_06077_b200 import inputs
    g = inputs.c1_input()
    got, bits = gpu_encode(g, 1024, 3, 0, seed=0, offset=0)
    nbad, nrel = compare_symbols(g, 1024, 3, 0, 0, 0, got)
    want, _ = O.encode(g, 1024, 3, 0, 0, 0)
    if nbad == 0 and nrel == 0.0:
        assert np.array_equal(got, want)
    acc = gpu_decode([got], g.size, 1024, 3)
    rc, ref = O.decode_accumulate([want], g.size, 1024, 3)
    err = np.linalg.norm(acc.astype(np.float64) - ref) / np.linalg.norm(ref)
    assert err <= 1e-5


def test_encode_is_deterministic_and_ignores_stale_output():
    g = _input(300000, 1)
    a, _ = gpu_encode(g, 8192, 4, 0, 9, 2)
    b, _ = gpu_encode(g, 8192, 4, 0, 9, 2, prefill=0x7FFFFFFF)
    c, _ = gpu_encode(g, 8192, 4, 0, 9, 3)
    assert np.array_equal(a, b)
    assert not np.array_equal(a, c)


def test_scan_state_is_clean_after_a_call_with_wide_buckets():
    """A call with buckets wider than a tile keeps its bucket norms behind its scan state in the stream's
    workspace.  A later call with more tiles keeps scan state at that place and must find it cleared."""
    gpu_encode(_input(2_000_000, 5), 8192, 4, 0, 1, 0)       # the workspace grows once, here
    for (d_wide, b_wide, d_next) in ((100_000, 16384, 300_001), (40_000, 32768, 8192 * 12 + 7), (200_000, 65536, 8192 * 40),
                                     # the next call's group word (a sum that is added to) lies where the norms were
                                     (200_000, 65536, 8192 * 25 + 100), (100_000, 16384, 8192 * 13 + 50), (40_000, 32768, 8192 * 5 + 9)):
        for rep in range(3):
            # (4-bit fixed-width calls take their norms from the workspace; ERC calls add them up in clusters)
            gpu_encode(_input(d_wide, d_wide + rep), b_wide, 4, O.make_flags(mode=O.MODE_FIXED) if rep % 2 == 0 else 0, 3, rep)
            if rep == 1:                                      # a short call in between clears only what it uses itself
                gpu_encode(_input(1000, 1), 256, 3, 0, 1, 0)
            if rep == 2:                                      # the histogram's norms lie at the front of the workspace
                from gpu_util import gpu_level_histogram
                gpu_level_histogram(_input(d_wide, 9), 512, 4, 0, 1, 0)
                gpu_encode(_input(1000, 1), 256, 3, 0, 1, 0)
            g = _input(d_next, d_next + rep)
            norms = O.bucket_norms(g, 8192, L2)
            want, want_bits = O.encode(g, 8192, 4, 0, seed=5, offset=rep, norms=norms)
            got, got_bits = gpu_encode(g, 8192, 4, 0, seed=5, offset=rep, norms=norms)
            assert got_bits == want_bits and np.array_equal(got, want)


@pytest.mark.parametrize("d,bucket,nk,ls", [(6_000_001, 16384, L2, EXP), (6_000_001, 32768, LINF, EXP),
                                            (5_000_000 + 8192 * 3 + 11, 65536, L2, UNI), (65536 * 3 + 8192 * 2 + 1, 65536, L2, EXP)])
def test_wide_buckets_encoded_by_clusters(d, bucket, nk, ls):
    """Buckets wider than a tile: a cluster of 2, 4 or 8 CTAs encodes a bucket and adds up its norm among
    themselves.  More buckets than resident clusters (so that buckets are handed out by ticket), a last
    bucket with fewer tiles than the cluster has CTAs, both norms; the decoded sum of two such streams."""
    flags = O.make_flags(nk, ls, O.MODE_ERC)
    gs = [_input(d, 31 * d + k) for k in range(2)]
    streams = []
    for k, g in enumerate(gs):
        got, _ = gpu_encode(g, bucket, 4, flags, seed=7 + k, offset=k)
        compare_symbols(g, bucket, 4, flags, 7 + k, k, got)
        # given the norms the clusters agreed on, the whole container is the oracle's
        rc, _, _, gnorms = O.decode_symbols(got, d, bucket, 4)
        assert rc == 0
        want, _ = O.encode(g, bucket, 4, flags, 7 + k, k, norms=gnorms)
        assert np.array_equal(got, want)
        streams.append(got)
    acc = gpu_decode(streams, d, bucket, 4)
    assert np.array_equal(acc.view(np.uint32), O.decode_accumulate(streams, d, bucket, 4)[1].view(np.uint32))


def test_stream_info_and_status():
    torch, nuq = require_cuda()
    g = torch.from_numpy(_input(50000, 2)).cuda()
    out, bits = nuq.encode(g, 1024, 3, 0, 1, 0)
    info = nuq.stream_info(out)
    assert info["d"] == 50000 and info["bucket"] == 1024 and info["s"] == 3 and info["sub_block"] == 256
    assert info["container_bits"] == int(bits.item()) and info["nblk"] == 49
    assert nuq.last_status() == 0


def test_invalid_arguments_are_refused():
    torch, nuq = require_cuda()
    g = torch.zeros(4096, device="cuda")
    for bucket, s, flags in ((100, 3, 0), (0, 3, 0), (1024, 0, 0), (1024, 15, 0), (1024, 9, nuq.LEVELS_UNIFORM),
                             (1024, 3, 2), (1024, 3, 1 << 26), (131072, 3, 0), (1024, 3, nuq.TEST_NORMS)):
        assert nuq.encode_bound(4096, bucket, s, flags & ~nuq.TEST_NORMS) == 0 or flags & nuq.TEST_NORMS
        with pytest.raises(nuq.NuqError) as e:
            nuq.encode(g, bucket, s, flags, out=torch.empty(65536, dtype=torch.int32, device="cuda"))
        assert e.value.code == nuq.ERR_INVALID_ARG
    out, _ = nuq.encode(g, 1024, 3)
    with pytest.raises(nuq.NuqError):
        nuq.decode_accumulate([out] * 65, 4096, 1024, 3)
    with pytest.raises(nuq.NuqError):
        nuq.decode_accumulate([out], 4096, 1000, 3)
    with pytest.raises(nuq.NuqError):                      # misaligned input
        nuq.encode(torch.zeros(4097, device="cuda")[1:], 1024, 3)
    assert nuq.last_status() == 0


def test_malformed_containers_are_reported_not_trusted():
    """Corrupt headers, offsets, lengths and tokens: the decoder latches BAD_STREAM and stays in bounds."""
    d, bucket, s = 40000, 1024, 3
    g = _input(d, 3)
    good, _ = O.encode(g, bucket, s, 0, 1, 0)
    nblk = 40
    payload0 = 16 + 2 * (nblk + 1)
    gpu_decode([good], d, bucket, s)
    edits = [
        (0, 0), (1, 9), (2, d - 1), (4, 2048), (5, 4), (7, 128), (8, nblk - 1), (10, 31),
        (16 + 2 * 3, 5),                       # block 3 offset not a multiple of 32
        (16 + 2 * 3, 0xFFFFFF00),              # block 3 offset beyond the payload
        (payload0 + 1, 0xFFFFFFFF),            # sub-block lengths of block 0 beyond the block
        (payload0 + 4, 0xFFFFFFFF),            # token soup
    ]
    for word, value in edits:
        bad = good.copy()
        bad[word] = value
        assert O.decode_symbols(bad, d, bucket, s)[0] == -3, (word, value)
        gpu_decode([bad], d, bucket, s, expect_status=-3)
        gpu_decode([good, bad, good], d, bucket, s, expect_status=-3)
    fx, _ = O.encode(g, bucket, s, O.make_flags(mode=O.MODE_FIXED), 1, 0)
    bad = fx.copy(); bad[20] = 0xFFFFFFFF      # level index 7 does not exist for s = 3
    gpu_decode([bad], d, bucket, s, expect_status=-3)
    assert np.array_equal(gpu_decode([good], d, bucket, s), O.decode_accumulate([good], d, bucket, s)[1])


def test_degenerate_buckets():
    d, bucket = 5 * 1024, 1024
    g = _input(d, 4)
    g[0:1024] = 0.0                            # all-zero bucket
    g[1024 + 5] = np.nan                       # NaN poisons bucket 1
    g[2048 + 9] = np.inf                       # infinite norm
    g[3072:4096] = 1e-42                       # 2^s / norm overflows
    for flags in (0, O.make_flags(mode=O.MODE_FIXED), O.make_flags(L2, UNI), O.make_flags(LINF, UNI)):
        # buckets 1 to 3 cannot be quantized: the encoder says so (bucket 0 is all zero, which is no warning)
        got, _ = gpu_encode(g, bucket, 4, flags, 1, 0, expect_status=1)
        # the degenerate buckets' norm words are the oracle's bit for bit, the ordinary bucket's norm agrees
        # to 1e-6; given the norms the GPU used, the whole container is the oracle's
        rc, _, _, gnorms = O.decode_symbols(got, d, bucket, 4)
        assert rc == 0
        onorms = O.bucket_norms(g, bucket, flags & 0xff)
        assert np.array_equal(gnorms[:4].view(np.uint32), onorms[:4].view(np.uint32))
        assert abs(float(gnorms[4]) - float(onorms[4])) <= 1e-6 * float(onorms[4])
        want, _ = O.encode(g, bucket, 4, flags, 1, 0, norms=gnorms)
        assert np.array_equal(got, want)
        acc = gpu_decode([got], d, bucket, 4)
        assert np.array_equal(acc.view(np.uint32), O.decode_accumulate([want], d, bucket, 4)[1].view(np.uint32))
        assert not acc[:4096].any()


@pytest.mark.parametrize("d,bucket,s", [(40000, 256, 4), (70000, 1024, 5), (50000, 4096, 6), (33000, 256, 2),
                                        (100000, 8192, 4)])
def test_dense_inputs_stay_inside_the_staging_buffers(d, bucket, s):
    """Vectors whose coordinates all have r = 2^-s (every coordinate becomes a token) or are as
    dense as the norm allows: the encoder sizes its shared-memory staging by the sparsity bound of
    the paper (at most 4^s coordinates of a bucket above the lowest level, Lemma 10), so the
    free-running path must still equal the oracle here."""
    rng = np.random.default_rng(d + s)
    flat = np.where(rng.random(d) < 0.5, -1.0, 1.0).astype(np.float32)         # r = 1/sqrt(bucket) everywhere
    spiky = flat.copy()
    spiky[:: max(1, bucket // (4 ** s))] *= 3.0                                # about 4^s larger coordinates per bucket
    noisy = (rng.standard_normal(d) * 1.0).astype(np.float32)
    for g in (flat, spiky, noisy):
        got, bits = gpu_encode(g, bucket, s, 0, seed=3, offset=1)
        nbad, rel = compare_symbols(g, bucket, s, 0, 3, 1, got)
        if nbad == 0 and rel == 0.0:
            want, want_bits = O.encode(g, bucket, s, 0, 3, 1)
            assert bits == want_bits and np.array_equal(got, want)
        acc = gpu_decode([got], d, bucket, s)
        assert np.array_equal(acc.view(np.uint32), O.decode_accumulate([got], d, bucket, s)[1].view(np.uint32))


@pytest.mark.parametrize("d,bucket,s,ls", [(70001, 1024, 4, O.LEVELS_EXP), (8192 * 3 + 17, 8192, 2, O.LEVELS_EXP),
                                           (200000, 65536, 4, O.LEVELS_EXP), (50000, 512, 7, O.LEVELS_EXP),
                                           (33333, 256, 3, O.LEVELS_UNIFORM), (40000, 2048, 8, O.LEVELS_UNIFORM)])
def test_fixed_width_streams_decoded_where_they_were_encoded(d, bucket, s, ls):
    """Containers that stay on the device where the library wrote them: the decoder then knows (and
    checks) that all of them are in the fixed-width mode and takes its simple path.  The sums must
    equal the oracle's bit for bit, also when a buffer's content no longer is what the library wrote
    there (an ERC container copied over a fixed-width one)."""
    torch, nuq = require_cuda()
    K = 3
    flags_fixed = O.make_flags(O.NORM_L2, ls, O.MODE_FIXED)
    flags_erc = O.make_flags(O.NORM_L2, ls, O.MODE_ERC)
    gs = [_input(d, 100 + k) for k in range(K)]
    nbytes = max(nuq.encode_bound(d, bucket, s, flags_fixed), nuq.encode_bound(d, bucket, s, flags_erc))
    outs, host = [], []
    for k in range(K):
        out = torch.zeros(nbytes // 4, dtype=torch.int32, device="cuda")
        _, bits = nuq.encode(torch.from_numpy(gs[k]).cuda(), bucket, s, flags_fixed, 11 + k, 0, out=out)
        outs.append(out)
        host.append(out.cpu().numpy().view(np.uint32)[: int(bits.item()) // 32].copy())
    acc = nuq.decode_accumulate(outs, d, bucket, s)
    assert nuq.last_status() == 0
    want = O.decode_accumulate(host, d, bucket, s)[1]
    assert np.array_equal(acc.cpu().numpy().view(np.uint32), want.view(np.uint32))
    # same buffers, but the middle one now holds an ERC container of the same vector
    erc, _ = gpu_encode(gs[1], bucket, s, flags_erc, seed=12, offset=0)
    outs[1].zero_()
    outs[1][: erc.size] = torch.from_numpy(erc.view(np.int32)).cuda()
    host[1] = erc
    acc = nuq.decode_accumulate(outs, d, bucket, s)
    assert nuq.last_status() == 0
    want = O.decode_accumulate(host, d, bucket, s)[1]
    assert np.array_equal(acc.cpu().numpy().view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("modes", [(O.MODE_ERC, O.MODE_FIXED, O.MODE_ERC), (O.MODE_FIXED, O.MODE_ERC, O.MODE_FIXED)])
@pytest.mark.parametrize("d,bucket,s", [(20000, 256, 4), (50000, 1024, 5)])
def test_mixed_modes_keep_the_stream_order_when_chains_take_several_rounds(modes, d, bucket, s):
    """Dense ERC streams (every coordinate a token) are decoded in several rounds of positions; the
    fixed-width streams of the same call must add their terms round by round too, or an element
    would receive its terms out of stream order and the fp32 sum would differ."""
    rng = np.random.default_rng(d)
    streams = []
    for k, mode in enumerate(modes):
        g = np.where(rng.random(d) < 0.5, -1.0, 1.0).astype(np.float32) * (1.0 + 0.25 * rng.random(d).astype(np.float32))
        streams.append(O.encode(g, bucket, s, O.make_flags(O.NORM_L2, O.LEVELS_EXP, mode), seed=k + 1, offset=0)[0])
    rc, want = O.decode_accumulate(streams, d, bucket, s)
    assert rc == 0
    got = gpu_decode(streams, d, bucket, s)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("K", [9, 17])
def test_more_streams_than_one_group(K):
    """More than 8 streams are decoded in groups of 8, one group after the other, the last one
    partly filled; the order of the adds is still the stream order across groups."""
    d, bucket, s = 30000, 1024, 4
    streams = []
    for k in range(K):
        mode = O.MODE_FIXED if k == 10 else O.MODE_ERC
        streams.append(O.encode(_input(d, 7000 + k), bucket, s, O.make_flags(O.NORM_L2, O.LEVELS_EXP, mode),
                                seed=k + 1, offset=0)[0])
    rc, want = O.decode_accumulate(streams, d, bucket, s)
    assert rc == 0
    got = gpu_decode(streams, d, bucket, s)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_a_scan_wait_that_runs_out_is_reported_and_does_no_harm():
    """The look-back over tile sizes waits with a limit.  A test flag shortens that limit to two polls, so
    that on a vector of several thousand tiles some writer warp does give up: the call must come back at
    once with NUQ_ERR_TIMEOUT latched, write nothing outside its buffer, and leave the library in a state
    in which the next ordinary call is bit-exact again.  Nothing is withheld and nothing can hang: the
    flag only makes the wait shorter."""
    import time
    torch, nuq = require_cuda()
    from paper_1908_06077_b200 import inputs
    g = inputs.c3_input(1)
    ref, ref_bits = gpu_encode(g, 8192, 4, 0, seed=1, offset=0)
    seen = []
    for attempt in range(4):
        gd = torch.from_numpy(g).cuda()
        nbytes = nuq.encode_bound(gd.numel(), 8192, 4, 0)
        out = torch.full((nbytes // 4 + 64,), -1515870811, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        nuq.encode(gd, 8192, 4, nuq.TEST_SHORT_PATIENCE, 1, 0, out=out)
        status = nuq.last_status()
        dt = time.perf_counter() - t0
        assert dt < 0.5, dt
        assert status in (0, nuq.ERR_TIMEOUT), status
        host = out.cpu().numpy().view(np.uint32)
        assert (host[nbytes // 4:] == np.uint32(0xA5A5A5A5)).all()
        seen.append(status)
        if status == nuq.ERR_TIMEOUT:
            break
    assert nuq.ERR_TIMEOUT in seen, seen
    again, again_bits = gpu_encode(g, 8192, 4, 0, seed=1, offset=0)
    assert again_bits == ref_bits and np.array_equal(again, ref)


def test_nonfinite_norms_raise_a_warning_only():
    torch, nuq = require_cuda()
    g = _input(8192, 5)
    gpu_encode(g, 1024, 3, 0, 1, 0)                                  # ordinary data: no warning
    g[100] = np.inf
    got, _ = gpu_encode(g, 1024, 3, 0, 1, 0, expect_status=nuq.WARN_NONFINITE)
    want, _ = O.encode(g, 1024, 3, 0, 1, 0, norms=O.decode_symbols(got, g.size, 1024, 3)[3])
    assert np.array_equal(got, want)
    gpu_encode(np.zeros(4096, np.float32), 1024, 3, 0, 1, 0)         # an all-zero vector is not a warning


@pytest.mark.parametrize("d,bucket,s", [(70001, 1024, 4), (8192 * 3 + 17, 8192, 2), (200000, 65536, 4), (50000, 512, 7),
                                        (33000, 256, 3), (255, 256, 3)])
@pytest.mark.parametrize("K", [5, 8, 11])
def test_five_to_eleven_erc_streams(d, bucket, s, K):
    """One partly filled group of streams, one full group, and a full group followed by a partly filled one."""
    streams = [O.encode(_input(d, 500 * k + d + s), bucket, s, 0, seed=k + 1, offset=k)[0] for k in range(K)]
    rc, want = O.decode_accumulate(streams, d, bucket, s)
    assert rc == 0
    got = gpu_decode(streams, d, bucket, s)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("d,bucket,s", [(20000, 256, 4), (50000, 1024, 5), (100000, 8192, 4)])
def test_eight_streams_of_mixed_density_and_lists_that_run_over(d, bucket, s):
    """Every coordinate a token in some streams, ordinary density in others: rounds of positions, and
    rounds that have to be taken again because a list ran over."""
    rng = np.random.default_rng(d + 1)
    streams = []
    for k in range(8):
        if k % 3 == 0:
            g = np.where(rng.random(d) < 0.5, -1.0, 1.0).astype(np.float32) * (1.0 + 0.25 * rng.random(d).astype(np.float32))
        elif k % 3 == 1:
            g = _input(d, 9000 + k)
            g[: d // 2] = np.where(rng.random(d // 2) < 0.5, -1.0, 1.0)      # dense front half, sparse back half
        else:
            g = _input(d, 9100 + k)
        streams.append(O.encode(g, bucket, s, 0, seed=k + 1, offset=0)[0])
    rc, want = O.decode_accumulate(streams, d, bucket, s)
    assert rc == 0
    got = gpu_decode(streams, d, bucket, s)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_malformed_container_among_six_streams():
    d, bucket, s = 40000, 1024, 3
    good = [O.encode(_input(d, 40 + k), bucket, s, 0, k + 1, 0)[0] for k in range(6)]
    nblk = 40
    payload0 = 16 + 2 * (nblk + 1)
    for word, value in [(0, 0), (5, 4), (16 + 2 * 3, 5), (16 + 2 * 3, 0xFFFFFF00), (payload0 + 1, 0xFFFFFFFF),
                        (payload0 + 4, 0xFFFFFFFF)]:
        bad = good[2].copy()
        bad[word] = value
        gpu_decode(good[:2] + [bad] + good[3:], d, bucket, s, expect_status=-3)
    want = O.decode_accumulate(good, d, bucket, s)[1]
    assert np.array_equal(gpu_decode(good, d, bucket, s).view(np.uint32), want.view(np.uint32))


# ---------------------------------------------------------------- general level sequences (Sec. 3.3)
def _lp(p, s):
    return np.array([p ** (s + 1 - j) for j in range(1, s + 1)], np.float32)


TABLE_CASES = [
    (70001, 1024, _lp(0.3, 3)),
    (3 * 8192 + 5, 8192, _lp(0.5, 4)),                     # the paper's own levels, as a table
    (20000, 512, _lp(0.7, 6)),
    (150001, 16384, _lp(0.25, 2)),
    (40000, 2048, np.array([0.01, 0.02, 0.05, 0.1, 0.15, 0.2, 0.3, 0.4, 0.5, 0.6, 0.7, 0.8, 0.9, 0.95], np.float32)),
    (257, 256, np.array([0.5], np.float32)),
]


@pytest.mark.parametrize("d,bucket,levels", TABLE_CASES)
@pytest.mark.parametrize("mode", [O.MODE_ERC, O.MODE_FIXED])
def test_level_table_streams_match_the_oracle(d, bucket, levels, mode):
    """Level sequences given as a table: with the oracle's norms the container is the oracle's bit for bit
    (level words behind the header included); free running, norms and symbols agree by the usual rule;
    the decoded vector is the oracle's."""
    torch, nuq = require_cuda()
    s = levels.size
    O.set_levels(levels)
    nuq.set_level_table(levels)
    flags = O.make_flags(O.NORM_L2, O.LEVELS_TABLE, mode)
    g = _input(d, 31 * d + s)
    norms = O.bucket_norms(g, bucket, O.NORM_L2)
    want, want_bits = O.encode(g, bucket, s, flags, seed=11, offset=3, norms=norms)
    got, got_bits = gpu_encode(g, bucket, s, flags, seed=11, offset=3, norms=norms)
    assert got_bits == want_bits and np.array_equal(got, want)
    free, _ = gpu_encode(g, bucket, s, flags, seed=5, offset=0)
    compare_symbols(g, bucket, s, flags, 5, 0, free)
    acc = gpu_decode([free], d, bucket, s)
    assert np.array_equal(acc.view(np.uint32), O.decode_accumulate([free], d, bucket, s)[1].view(np.uint32))


def test_level_table_streams_sum_with_others_and_bad_tables_are_refused():
    torch, nuq = require_cuda()
    d, bucket, s = 50000, 1024, 4
    O.set_levels(_lp(0.35, s))
    streams = []
    for k in range(6):                                       # tables of two kinds, the paper's levels, fixed width
        ls = O.LEVELS_TABLE if k % 2 == 0 else O.LEVELS_EXP
        if k == 4:
            O.set_levels(_lp(0.6, s))
        mode = O.MODE_FIXED if k in (2, 3) else O.MODE_ERC
        streams.append(O.encode(_input(d, 77 + k), bucket, s, O.make_flags(O.NORM_L2, ls, mode), k + 1, 0)[0])
    rc, want = O.decode_accumulate(streams, d, bucket, s)
    assert rc == 0
    got = gpu_decode(streams, d, bucket, s)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    bad = streams[0].copy()
    bad[17] = bad[16]                                        # levels that do not increase
    gpu_decode([bad], d, bucket, s, expect_status=-3)
    for levels in ([0.5, 0.25], [0.0, 0.5], [0.5, 1.0], [float("nan")], [0.1] * 15):
        with pytest.raises(nuq.NuqError):
            nuq.set_level_table(levels)
    nuq.set_level_table([0.25, 0.5])
    g = torch.zeros(4096, device="cuda")
    with pytest.raises(nuq.NuqError):                        # the table has two levels, the call asks for three
        nuq.encode(g, 1024, 3, nuq.LEVELS_TABLE)


# ---- coded level indices (Sec. 5, "efficient encoding") -------------------------------------------

CODED_CASES = [
    (100037, 8192, 4, O.LEVELS_EXP),
    (70000, 768, 3, O.LEVELS_EXP),
    (3 * 8192 + 5, 256, 2, O.LEVELS_EXP),
    (200000, 65536, 7, O.LEVELS_EXP),
    (40000, 2048, 1, O.LEVELS_EXP),
    (60000, 4096, 5, O.LEVELS_TABLE),
    (257, 256, 3, O.LEVELS_EXP),
]


@pytest.mark.parametrize("d,bucket,s,ls", CODED_CASES)
def test_coded_streams_match_the_oracle(d, bucket, s, ls):
    """The whole of the coded variant: the level histogram equals the oracle's (given its norms; free running
    it moves by a few counts), the lengths fitted on it are the oracle's, the container written with that
    code is the oracle's bit for bit, and the decoded vector is the oracle's."""
    from gpu_util import gpu_level_histogram
    torch, nuq = require_cuda()
    if ls == O.LEVELS_TABLE:
        levels = _lp(0.4, s)
        O.set_levels(levels)
        nuq.set_level_table(levels)
    g = _input(d, 17 * d + s)
    norms = O.bucket_norms(g, bucket, O.NORM_L2)
    sign, sym, _ = O.quantize(g, bucket, s, O.NORM_L2, ls, 11, 3, norms=norms)
    want_hist = O.level_histogram(sym, s)
    hist = gpu_level_histogram(g, bucket, s, O.make_flags(O.NORM_L2, ls, 0), 11, 3, norms=norms)
    assert np.array_equal(hist, want_hist)
    free_hist = gpu_level_histogram(g, bucket, s, O.make_flags(O.NORM_L2, ls, 0), 11, 3)
    assert free_hist.sum() == d and np.abs(free_hist.astype(np.int64) - want_hist.astype(np.int64)).sum() <= 2 + 2e-5 * d
    lengths = nuq.fit_level_code(hist, s)
    assert lengths == list(O.huffman_lengths(want_hist[1:]))
    O.set_level_code(lengths)
    nuq.set_level_code(lengths)
    flags = O.make_flags(O.NORM_L2, ls, O.MODE_CODED)
    want, want_bits = O.encode(g, bucket, s, flags, seed=11, offset=3, norms=norms)
    got, got_bits = gpu_encode(g, bucket, s, flags, seed=11, offset=3, norms=norms)
    assert got_bits == want_bits and np.array_equal(got, want)
    free, _ = gpu_encode(g, bucket, s, flags, seed=5, offset=0)
    compare_symbols(g, bucket, s, flags, 5, 0, free)
    acc = gpu_decode([free], d, bucket, s)
    assert np.array_equal(acc.view(np.uint32), O.decode_accumulate([free], d, bucket, s)[1].view(np.uint32))
    # the code is kept: another vector, the same words
    g2 = _input(d, 17 * d + s + 1)
    norms2 = O.bucket_norms(g2, bucket, O.NORM_L2)
    want2, _ = O.encode(g2, bucket, s, flags, seed=12, offset=4, norms=norms2)
    got2, _ = gpu_encode(g2, bucket, s, flags, seed=12, offset=4, norms=norms2)
    assert np.array_equal(got2, want2)


@pytest.mark.parametrize("K", [1, 2, 4, 8, 11])
def test_coded_streams_sum_with_streams_of_the_other_modes(K):
    """Each stream brings its own code; streams of all three modes are summed in stream order."""
    torch, nuq = require_cuda()
    d, bucket, s = 90000, 2048, 4
    codes = ([1, 2, 3, 4, 4], [3, 3, 2, 2, 2], [2, 2, 2, 3, 3], [4, 4, 3, 2, 1], [3, 3, 3, 3, 3])
    streams = []
    for k in range(K):
        O.set_level_code(codes[k % len(codes)])
        mode = (O.MODE_CODED, O.MODE_CODED, O.MODE_ERC, O.MODE_CODED, O.MODE_FIXED)[k % 5] if K > 1 else O.MODE_CODED
        g = _input(d, 5 + k) * (30.0 if k % 3 == 1 else 1.0)
        streams.append(O.encode(g, bucket, s, O.make_flags(O.NORM_L2, O.LEVELS_EXP, mode), k + 1, k)[0])
    rc, want = O.decode_accumulate(streams, d, bucket, s)
    assert rc == 0
    got = gpu_decode(streams, d, bucket, s)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_coded_streams_with_dense_symbols_and_long_words_stay_inside_the_staging_buffers():
    """A code that gives the commonest level index the longest word, on inputs where most coordinates are
    nonzero: the token strings are as long as they can get."""
    torch, nuq = require_cuda()
    for (d, bucket, s, lengths, scale) in ((50000, 256, 7, [7, 7, 6, 5, 4, 3, 2, 1], 1.0),
                                           (50000, 8192, 2, [2, 2, 2], 1.0),
                                           (30000, 512, 3, [3, 3, 3, 3], 1.0)):
        rng = np.random.default_rng(d + s)
        g = (rng.uniform(0.5, 1.0, d) * rng.choice([-1.0, 1.0], d)).astype(np.float32)      # every coordinate large
        O.set_level_code(lengths)
        nuq.set_level_code(lengths)
        flags = O.make_flags(O.NORM_L2, O.LEVELS_EXP, O.MODE_CODED)
        norms = O.bucket_norms(g, bucket, O.NORM_L2)
        want, want_bits = O.encode(g, bucket, s, flags, seed=2, offset=1, norms=norms)
        got, got_bits = gpu_encode(g, bucket, s, flags, seed=2, offset=1, norms=norms)
        assert got_bits == want_bits and np.array_equal(got, want)
        free, _ = gpu_encode(g, bucket, s, flags, seed=2, offset=1)
        compare_symbols(g, bucket, s, flags, 2, 1, free)
        got_acc = gpu_decode([free, want], d, bucket, s)
        assert np.array_equal(got_acc.view(np.uint32), O.decode_accumulate([free, want], d, bucket, s)[1].view(np.uint32))


def test_malformed_coded_containers_and_bad_codes_are_refused():
    torch, nuq = require_cuda()
    d, bucket, s = 30000, 1024, 3
    O.set_level_code([1, 2, 3, 3])
    st, _ = O.encode(_input(d, 3), bucket, s, O.make_flags(O.NORM_L2, O.LEVELS_EXP, O.MODE_CODED), 1, 0)
    gpu_decode([st], d, bucket, s)
    for word in (0x01010101, 0x03030200, 0x08030201):        # Kraft sum above one, a zero length, a length above 7
        bad = st.copy()
        bad[16] = word
        gpu_decode([bad], d, bucket, s, expect_status=-3)
    bad = st.copy()
    bad[16] = 0x04040403                                     # an incomplete code: chains run into bits that spell no word
    gpu_decode([bad], d, bucket, s, expect_status=-3)
    other = O.encode(_input(d, 4), bucket, s, 0, 2, 0)[0]
    gpu_decode([other, bad, other], d, bucket, s, expect_status=-3)
    for lengths in ([1, 1, 2], [0, 1], [1, 8], [1, 2, 3, 3, 3]):
        with pytest.raises(nuq.NuqError):
            nuq.set_level_code(lengths)
    nuq.set_level_code([1, 2, 2])
    g = torch.zeros(4096, device="cuda")
    with pytest.raises(nuq.NuqError):                        # the code has three words, s = 3 needs four
        nuq.encode(g, 1024, 3, nuq.MODE_CODED)
    with pytest.raises(nuq.NuqError):                        # no coded level indices with uniform levels
        nuq.encode(g, 1024, 2, nuq.MODE_CODED | nuq.LEVELS_UNIFORM)
    with pytest.raises(nuq.NuqError):
        nuq.level_histogram(g, 1024, 2, nuq.LEVELS_UNIFORM)


def test_a_long_sequence_of_calls_of_many_shapes_on_one_stream():
    """Every call on a stream uses the same workspace (scan state, tickets, bucket norms of wide buckets,
    histogram norms, the decoder's ticket).  A seeded sequence of encode, histogram and decode calls of
    unrelated shapes and modes must give, call after call, the container the oracle writes when it is
    given the norms the GPU took (bit for bit), and the oracle's sums."""
    from gpu_util import gpu_level_histogram
    torch, nuq = require_cuda()
    rng = np.random.default_rng(2024)
    buckets = [256, 512, 768, 1024, 2048, 4096, 8192, 16384, 32768, 65536]
    O.set_level_code([1, 2, 3, 4, 4])
    nuq.set_level_code([1, 2, 3, 4, 4])
    checked = 0
    for it in range(160):
        d = int(rng.choice([rng.integers(1, 3000), rng.integers(3000, 120_000), rng.integers(120_000, 600_000)]))
        bucket = int(rng.choice(buckets))
        mode = int(rng.choice([O.MODE_ERC, O.MODE_ERC, O.MODE_FIXED, O.MODE_CODED]))
        ls = O.LEVELS_EXP if mode == O.MODE_CODED or rng.random() < 0.7 else O.LEVELS_UNIFORM
        s = 4 if mode == O.MODE_CODED else int(rng.integers(1, 8))
        nk = int(rng.integers(0, 2)) if ls == O.LEVELS_UNIFORM else O.NORM_L2
        flags = O.make_flags(nk, ls, mode)
        g = _input(d, 1000 + it)
        seed, offset = int(rng.integers(0, 2 ** 40)), int(rng.integers(0, 2 ** 20))
        got, bits = gpu_encode(g, bucket, s, flags, seed, offset)
        rc, sign, sym, norms = O.decode_symbols(got, d, bucket, s)
        assert rc == 0, (it, d, bucket, s, flags)
        want, want_bits = O.encode(g, bucket, s, flags, seed, offset, norms=norms)
        assert bits == want_bits and np.array_equal(got, want), (it, d, bucket, s, flags)
        ref_norms = O.bucket_norms(g, bucket, nk)
        live = np.isfinite(ref_norms) & (ref_norms > 0)
        assert np.all(np.abs(norms[live].astype(np.float64) - ref_norms[live]) <= 1e-6 * ref_norms[live])
        if it % 5 == 2:                                      # a histogram call leaves its norms in the workspace
            hist = gpu_level_histogram(g, min(bucket, 8192), 4, 0, seed, offset)
            assert hist.sum() == d
        if it % 4 == 1:                                      # the decoder uses the same workspace
            acc = gpu_decode([got, got], d, bucket, s)
            assert np.array_equal(acc.view(np.uint32), O.decode_accumulate([got, got], d, bucket, s)[1].view(np.uint32))
        checked += 1
    assert checked == 160


def test_two_streams_work_side_by_side_and_the_library_starts_over_after_shutdown():
    """Every (device, stream) pair has a workspace of its own: calls enqueued alternately on two streams,
    whose kernels may overlap, give the oracle's containers and sums; after nuq_shutdown the next call
    allocates again and is bit-exact as before; a status is reported on the stream that latched it."""
    torch, nuq = require_cuda()
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    shapes = [(300_001, 8192, 4, 0), (200_000, 65536, 3, 0), (150_000, 1024, 4, O.make_flags(mode=O.MODE_FIXED)),
              (90_000, 512, 2, O.make_flags(O.NORM_LINF, O.LEVELS_UNIFORM))]
    for round_ in range(2):
        jobs = []
        for i, (d, bucket, s, flags) in enumerate(shapes * 2):
            st = sa if i % 2 == 0 else sb
            g = _input(d, 500 + i)
            with torch.cuda.stream(st):
                gd = torch.from_numpy(g).cuda()
                out, bits = nuq.encode(gd, bucket, s, flags, seed=i + 1, offset=round_, stream=st)
                acc = nuq.decode_accumulate([out, out], d, bucket, s, stream=st)
            jobs.append((g, d, bucket, s, flags, i, gd, out, bits, acc))
        torch.cuda.synchronize()
        assert nuq.last_status(sa) == 0 and nuq.last_status(sb) == 0
        for (g, d, bucket, s, flags, i, gd, out, bits, acc) in jobs:
            got = out.cpu().numpy().view(np.uint32)[: int(bits.item()) // 32].copy()
            rc, sign, sym, norms = O.decode_symbols(got, d, bucket, s)
            assert rc == 0
            want, _ = O.encode(g, bucket, s, flags, i + 1, round_, norms=norms)
            assert np.array_equal(got, want), (round_, i)
            ref = O.decode_accumulate([got, got], d, bucket, s)[1]
            assert np.array_equal(acc.cpu().numpy().view(np.uint32), ref.view(np.uint32)), (round_, i)
        nuq.shutdown()                                       # the second round starts from nothing
    # a malformed container on one stream is reported there and not on the other
    bad = torch.zeros(4096, dtype=torch.int32, device="cuda")
    with torch.cuda.stream(sa):
        nuq.decode_accumulate([bad], 1000, 256, 3, stream=sa)
    torch.cuda.synchronize()
    assert nuq.last_status(sb) == 0 and nuq.last_status(sa) == nuq.ERR_BAD_STREAM and nuq.last_status(sa) == 0
