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
