"""Parity at the benchmark's sizes, in the launch configuration bench.py times: the
ResNet-50-sized workload (d = 25 557 032, bucket 8192, K streams) in full, and the flat Laplace
workload at d = 2^24 with the three bucket sizes of the large configuration."""
import numpy as np
import pytest

import oracle as O
from gpu_util import compare_symbols, gpu_decode, gpu_encode

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def c3_inputs():
    from paper_1908_06077_b200 import inputs
    return [inputs.c3_input(k) for k in (1, 2, 3)]


@pytest.mark.parametrize("s", [4, 2])
def test_c3_encode_matches_oracle(c3_inputs, s):
    g = c3_inputs[0]
    got, bits = gpu_encode(g, 8192, s, 0, seed=1, offset=0)
    nbad, rel = compare_symbols(g, 8192, s, 0, 1, 0, got)
    assert nbad <= 1e-5 * g.size and rel <= 1e-6
    if nbad == 0 and rel == 0.0:                            # same norms, same symbols: same bits
        want, want_bits = O.encode(g, 8192, s, 0, 1, 0)
        assert bits == want_bits and np.array_equal(got, want)


def test_c3_fixed_width_and_uniform_levels(c3_inputs):
    g = c3_inputs[1]
    for flags in (O.make_flags(mode=O.MODE_FIXED), O.make_flags(O.NORM_L2, O.LEVELS_UNIFORM),
                  O.make_flags(O.NORM_LINF, O.LEVELS_UNIFORM)):
        got, _ = gpu_encode(g, 8192, 4, flags, seed=2, offset=0)
        compare_symbols(g, 8192, 4, flags & 0xFFFF, 2, 0, got)


def test_c3_decode_accumulate_matches_oracle(c3_inputs):
    d = c3_inputs[0].size
    streams = [gpu_encode(g, 8192, 4, 0, seed=k + 1, offset=0)[0] for k, g in enumerate(c3_inputs)]
    rc, want = O.decode_accumulate(streams, d, 8192, 4)
    assert rc == 0
    got = gpu_decode(streams, d, 8192, 4)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # the criterion of the problem statement, for the record
    err = np.linalg.norm(got.astype(np.float64) - want) / np.linalg.norm(want)
    assert err <= 1e-5


@pytest.mark.parametrize("bucket", [512, 8192, 65536])
def test_c4_sized_down(bucket):
    from paper_1908_06077_b200 import inputs
    d = 1 << 24
    gs = [inputs.c4_input(k, d) for k in (1, 2)]
    streams = []
    for k, g in enumerate(gs):
        got, _ = gpu_encode(g, bucket, 4, 0, seed=k + 1, offset=0)
        compare_symbols(g, bucket, 4, 0, k + 1, 0, got)
        streams.append(got)
    rc, want = O.decode_accumulate(streams, d, bucket, 4)
    assert rc == 0
    got = gpu_decode(streams, d, bucket, 4)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_c3_decode_of_eight_workers_as_benchmarked():
    """The benchmark's decode call: eight distinct ResNet-50-sized gradients, eight streams side by
    side (the instance of the kernel with the sums in shared memory, 25 warps per SM)."""
    from paper_1908_06077_b200 import inputs
    gs = [inputs.c3_input(k) for k in range(1, 9)]
    d = gs[0].size
    streams = [gpu_encode(g, 8192, 4, 0, seed=k + 1, offset=0)[0] for k, g in enumerate(gs)]
    rc, want = O.decode_accumulate(streams, d, 8192, 4)
    assert rc == 0
    got = gpu_decode(streams, d, 8192, 4)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_c2_in_full():
    """Config C2: the ResNet-18-sized layout with outliers at 50 sigma, four workers: every worker's
    symbols against the oracle's, then the decode call of the benchmark (four streams side by side)."""
    from paper_1908_06077_b200 import inputs
    gs = [inputs.c2_input(k) for k in (1, 2, 3, 4)]
    d = gs[0].size
    streams = []
    for k, g in enumerate(gs):
        got, _ = gpu_encode(g, 8192, 4, 0, seed=k + 1, offset=0)
        nbad, rel = compare_symbols(g, 8192, 4, 0, k + 1, 0, got)
        assert nbad <= 1e-5 * d and rel <= 1e-6
        streams.append(got)
    rc, want = O.decode_accumulate(streams, d, 8192, 4)
    assert rc == 0
    got = gpu_decode(streams, d, 8192, 4)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_c3_s3_encode_matches_oracle(c3_inputs):
    g = c3_inputs[2]
    got, _ = gpu_encode(g, 8192, 3, 0, seed=3, offset=0)
    nbad, rel = compare_symbols(g, 8192, 3, 0, 3, 0, got)
    assert nbad <= 1e-5 * g.size and rel <= 1e-6
    # given the norms the GPU took, the whole container is the oracle's
    rc, _, _, gnorms = O.decode_symbols(got, g.size, 8192, 3)
    assert rc == 0
    want, _ = O.encode(g, 8192, 3, 0, 3, 0, norms=gnorms)
    if nbad == 0:
        assert np.array_equal(got, want)


@pytest.mark.parametrize("norm", [O.NORM_L2, O.NORM_LINF])
def test_c5_decode_of_uniform_level_streams(c3_inputs, norm):
    """Config C5: the comparison quantizers (uniform levels k/16 with the Euclidean and with the max
    norm) at the ResNet-50 size: GPU-written containers decoded and summed by the GPU, against the oracle."""
    flags = O.make_flags(norm, O.LEVELS_UNIFORM)
    d = c3_inputs[0].size
    streams = [gpu_encode(g, 8192, 4, flags, seed=k + 1, offset=0)[0] for k, g in enumerate(c3_inputs)]
    rc, want = O.decode_accumulate(streams, d, 8192, 4)
    assert rc == 0
    got = gpu_decode(streams, d, 8192, 4)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


@pytest.fixture(scope="module")
def c4_inputs():
    from paper_1908_06077_b200 import inputs
    return [inputs.c4_input(k) for k in (1, 2)]


@pytest.mark.parametrize("bucket", [8192, 512, 65536])
def test_c4_at_its_stated_length(c4_inputs, bucket):
    """Config C4 at d = 2^30: table offsets beyond 2^32 bits, 131072 tiles and thousands of look-back
    groups, two million buckets at bucket 512, the separate norm pass of the wide buckets, and the
    decoder's instance for two streams.  Worker 1: the norms of all buckets against the oracle's, and
    the whole container against the oracle's encode given those norms (bit-exact streams for equal
    norms).  Then the GPU's sum of both workers' containers against the oracle's sum of them."""
    d = c4_inputs[0].size
    assert d == 1 << 30
    streams = [gpu_encode(g, bucket, 4, 0, seed=k + 1, offset=0)[0] for k, g in enumerate(c4_inputs)]
    g, st = c4_inputs[0], streams[0]
    assert O.header(st)["container_bits"] == 32 * st.size
    table_words = 2 * (O.header(st)["nblk"] + 1)
    gnorms = np.empty((d + bucket - 1) // bucket, np.float32)
    # the norm word of a bucket is the first word of its first coding block
    offs = st[16:16 + table_words].view(np.uint64)[:-1]
    step = max(1, bucket // 8192)
    gnorms[:] = st[16 + table_words + (offs[::step] >> np.uint64(5)).astype(np.int64)].view(np.float32)
    norms = O.bucket_norms(g, bucket, O.NORM_L2)
    rel = np.abs(gnorms.astype(np.float64) - norms) / norms
    print(f"C4 bucket {bucket}: largest relative norm difference {rel.max():.3g}, "
          f"{int((gnorms != norms).sum())} of {norms.size} norms differ in the last place")
    assert rel.max() <= 1e-6
    want, _ = O.encode(g, bucket, 4, 0, 1, 0, norms=gnorms)
    assert want.size == st.size and np.array_equal(st, want)
    del want
    rc, want = O.decode_accumulate(streams, d, bucket, 4)
    assert rc == 0
    got = gpu_decode(streams, d, bucket, 4)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_c3_coded_level_indices_as_benchmarked(c3_inputs):
    """The coded workload of the benchmark: the code is fitted on worker 1's gradient from the GPU's own
    histogram and kept; the histogram, the lengths, the symbols of two workers and the decoded sum of two
    coded streams and one ERC stream are the oracle's."""
    from gpu_util import gpu_level_histogram, require_cuda
    torch, nuq = require_cuda()
    d = c3_inputs[0].size
    hist = gpu_level_histogram(c3_inputs[0], 8192, 4, 0, 1, 0)
    _, sym, _ = O.quantize(c3_inputs[0], 8192, 4, O.NORM_L2, O.LEVELS_EXP, 1, 0)
    want_hist = O.level_histogram(sym, 4)
    assert hist.sum() == d and np.abs(hist.astype(np.int64) - want_hist.astype(np.int64)).sum() <= 2e-5 * d
    lengths = nuq.fit_level_code(hist, 4)
    assert lengths == list(O.huffman_lengths(want_hist[1:]))
    nuq.set_level_code(lengths)
    O.set_level_code(lengths)
    coded = O.make_flags(mode=O.MODE_CODED)
    streams = []
    for k in (0, 1):
        got, _ = gpu_encode(c3_inputs[k], 8192, 4, coded, seed=k + 1, offset=0)
        nbad, rel = compare_symbols(c3_inputs[k], 8192, 4, coded, k + 1, 0, got)
        assert nbad <= 1e-5 * d and rel <= 1e-6
        streams.append(got)
    streams.append(gpu_encode(c3_inputs[2], 8192, 4, 0, seed=3, offset=0)[0])
    rc, want = O.decode_accumulate(streams, d, 8192, 4)
    assert rc == 0
    got = gpu_decode(streams, d, 8192, 4)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_c3_with_a_level_table(c3_inputs):
    """General level sequences at the benchmark's size: L_p with p = 0.4, s = 4, in both modes."""
    from gpu_util import require_cuda
    torch, nuq = require_cuda()
    levels = np.array([0.4 ** 4, 0.4 ** 3, 0.4 ** 2, 0.4], np.float32)
    O.set_levels(levels)
    nuq.set_level_table(levels)
    g, d = c3_inputs[1], c3_inputs[1].size
    streams = []
    for mode in (O.MODE_ERC, O.MODE_FIXED):
        flags = O.make_flags(O.NORM_L2, O.LEVELS_TABLE, mode)
        got, _ = gpu_encode(g, 8192, 4, flags, seed=2, offset=0)
        nbad, rel = compare_symbols(g, 8192, 4, flags, 2, 0, got)
        assert nbad <= 1e-5 * d and rel <= 1e-6
        streams.append(got)
    rc, want = O.decode_accumulate(streams, d, 8192, 4)
    assert rc == 0
    got = gpu_decode(streams, d, 8192, 4)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("bucket,mode", [(8192, O.MODE_ERC), (65536, O.MODE_ERC), (32768, O.MODE_ERC), (8192, O.MODE_FIXED),
                                         (65536, O.MODE_FIXED)])
def test_two_streams_encode_at_the_same_time(c3_inputs, bucket, mode):
    """Two streams, each with several ResNet-50-sized encode calls in flight: neither call has all its CTAs
    resident, so a tile may only ever belong to a CTA that is running (every tile is handed out by ticket),
    and a CTA that starts when no tile is left still takes tickets, so the call's counters may be zeroed
    only when every CTA has finished (else the next call on the stream starts counting above zero and never
    encodes its first tiles).  Buckets wider than a tile are encoded by clusters, which take a ticket per
    bucket.  The containers are those of the same calls made alone, and no wait runs out."""
    import torch
    from gpu_util import require_cuda
    torch, nuq = require_cuda()
    flags = O.make_flags(mode=mode)
    gs = [torch.from_numpy(g).cuda() for g in c3_inputs[:2]]
    d = gs[0].numel()
    nbytes = nuq.encode_bound(d, bucket, 4, flags)
    alone = []
    for k, g in enumerate(gs):
        out = torch.zeros(nbytes // 4, dtype=torch.int32, device="cuda")
        _, bits = nuq.encode(g, bucket, 4, flags, seed=k + 1, offset=0, out=out)
        assert nuq.last_status() == 0
        alone.append(out.cpu().numpy().view(np.uint32)[: int(bits.item()) // 32].copy())
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [[torch.zeros(nbytes // 4, dtype=torch.int32, device="cuda") for _ in range(4)] for _ in range(2)]
    bits = [[torch.zeros(1, dtype=torch.int64, device="cuda") for _ in range(4)] for _ in range(2)]
    for attempt in range(3):
        for k in range(2):
            for rep in range(4):
                outs[k][rep].zero_()
                bits[k][rep].zero_()
        torch.cuda.synchronize()
        for rep in range(4):
            for k in range(2):
                with torch.cuda.stream(streams[k]):
                    nuq.encode(gs[k], bucket, 4, flags, seed=k + 1, offset=0, out=outs[k][rep], out_bits=bits[k][rep],
                               stream=streams[k])
            if attempt == 1 and rep == 0:
                torch.cuda.synchronize()                     # the later calls start at another moment of the other stream's
        torch.cuda.synchronize()
        for k in range(2):
            assert nuq.last_status(streams[k]) == 0
            for rep in range(4):
                n = int(bits[k][rep].item())
                assert n == 32 * alone[k].size
                assert np.array_equal(outs[k][rep].cpu().numpy().view(np.uint32)[: n // 32], alone[k])


@pytest.mark.parametrize("bucket,mode", [(8192, O.MODE_ERC), (8192, O.MODE_FIXED), (65536, O.MODE_ERC), (65536, O.MODE_FIXED)])
def test_encode_calls_keep_the_order_of_their_stream(c3_inputs, bucket, mode):
    """An encode kernel is set up while the kernel before it in the stream ends, but touches memory only when
    that kernel has ended: a gradient written by the kernel just before the call is the one that is encoded, a
    kernel that overwrites the gradient after the call does not reach into it, and of two calls into the same
    buffer the second one's container stays."""
    from gpu_util import require_cuda
    torch, nuq = require_cuda()
    flags = O.make_flags(mode=mode)
    src = [torch.from_numpy(g).cuda() for g in c3_inputs]
    d = src[0].numel()
    nbytes = nuq.encode_bound(d, bucket, 4, flags)
    alone = []
    for k, g in enumerate(src):
        out = torch.zeros(nbytes // 4, dtype=torch.int32, device="cuda")
        _, bits = nuq.encode(g, bucket, 4, flags, seed=7, offset=k, out=out)
        assert nuq.last_status() == 0
        alone.append(out.cpu().numpy().view(np.uint32)[: int(bits.item()) // 32].copy())
    g = torch.zeros(d, dtype=torch.float32, device="cuda")
    outs = [torch.zeros(nbytes // 4, dtype=torch.int32, device="cuda") for _ in range(6)]
    bits = [torch.zeros(1, dtype=torch.int64, device="cuda") for _ in range(6)]
    same = torch.zeros(nbytes // 4, dtype=torch.int32, device="cuda")
    same_bits = torch.zeros(1, dtype=torch.int64, device="cuda")
    torch.cuda.synchronize()
    for i in range(6):                                       # copy kernel, encode, copy kernel, encode, ... nothing waits
        g.copy_(src[i % 3])
        nuq.encode(g, bucket, 4, flags, seed=7, offset=i % 3, out=outs[i], out_bits=bits[i])
    for i in range(3):                                       # three calls in a row into one buffer
        nuq.encode(src[i], bucket, 4, flags, seed=7, offset=i, out=same, out_bits=same_bits)
    torch.cuda.synchronize()
    assert nuq.last_status() == 0
    for i in range(6):
        n = int(bits[i].item())
        assert n == 32 * alone[i % 3].size
        assert np.array_equal(outs[i].cpu().numpy().view(np.uint32)[: n // 32], alone[i % 3])
    n = int(same_bits.item())
    assert n == 32 * alone[2].size
    assert np.array_equal(same.cpu().numpy().view(np.uint32)[: n // 32], alone[2])


def test_encode_calls_replayed_from_a_cuda_graph(c3_inputs):
    """The eight encode calls of a step, captured once into a CUDA graph and replayed: an encode kernel leaves
    its workspace as it found it and takes nothing from the host but its arguments, so every replay writes the
    containers of the gradients that are in the input buffers at that time."""
    from gpu_util import require_cuda
    torch, nuq = require_cuda()
    src = [torch.from_numpy(g).cuda() for g in c3_inputs]
    d = src[0].numel()
    cases = [(8192, 0), (8192, O.make_flags(mode=O.MODE_FIXED)), (65536, 0)]
    side = torch.cuda.Stream()
    gs = [torch.zeros(d, dtype=torch.float32, device="cuda") for _ in range(3)]
    outs = [torch.zeros(nuq.encode_bound(d, b, 4, f) // 4, dtype=torch.int32, device="cuda") for b, f in cases]
    bits = [torch.zeros(1, dtype=torch.int64, device="cuda") for _ in cases]

    def enqueue():
        for i, (b, f) in enumerate(cases):
            nuq.encode(gs[i], b, 4, f, seed=11 + i, offset=5, out=outs[i], out_bits=bits[i], stream=side)

    with torch.cuda.stream(side):                            # first use of the stream: the workspace is allocated here
        enqueue()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        enqueue()
    for rnd in range(3):
        for i in range(3):
            gs[i].copy_(src[(i + rnd) % 3])
            outs[i].zero_()
            bits[i].zero_()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert nuq.last_status(side) == 0
        for i, (b, f) in enumerate(cases):
            want = torch.zeros_like(outs[i])
            _, wbits = nuq.encode(src[(i + rnd) % 3], b, 4, f, seed=11 + i, offset=5, out=want)
            n = int(wbits.item())
            assert int(bits[i].item()) == n
            assert torch.equal(outs[i][: n // 32], want[: n // 32])
