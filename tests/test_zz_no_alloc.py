"""nuq_encode_static, the encoder entry point that allocates nothing.

Some callers cannot call cudaMalloc: a training framework whose caching allocator
already owns the whole GPU, a loop that cannot afford the device-wide
synchronisation an allocation implies, a process with a memory budget fixed at
start-up.  For them the library offers a second encoder whose cross-tile scan
state sits in a fixed array inside the library's device image.  This test calls
it through the C ABI twice in a row (the second call finds the first call's
leftovers in the shared array) and requires the containers to equal those of
nuq_encode word for word -- the same tolerance the bit-stream tests use: none.

The file name sorts last on purpose: a run that stops at the first failure has
then already run every other test.
"""
import numpy as np
import pytest

from gpu_util import require_cuda

pytestmark = pytest.mark.gpu


def _input(d, seed):
    rng = np.random.default_rng(seed)
    g = rng.standard_normal(d) * 10.0 ** rng.uniform(-4, 0, d)
    g[rng.random(d) < 0.02] = 0.0
    return g.astype(np.float32)


def _container(torch, out, bits):
    n = int(bits.item())
    assert n % 32 == 0
    return out.cpu().numpy().view(np.uint32)[: n // 32].copy()


@pytest.mark.parametrize("d,bucket,s,flags", [
    (300001, 8192, 4, 0),                 # ERC, several tiles and a ragged tail
    (70000, 512, 3, 0),                   # many buckets per tile
    (200000, 65536, 4, 0),                # wide bucket: encoded by clusters of eight CTAs
    (200000, 65536, 4, 1 << 16),          # wide bucket, fixed-width: norms also live in the static scratch
    (100000, 8192, 4, 1 << 16),           # fixed-width mode
])
def test_static_scratch_encode_equals_allocating_encode_twice(d, bucket, s, flags):
    torch, nuq = require_cuda()
    nbytes = nuq.encode_bound(d, bucket, s, flags)
    for call in range(2):                 # two calls in a row share the static array
        g = torch.from_numpy(_input(d, 31 * d + call)).cuda()
        ref_out, ref_bits = nuq.encode(g, bucket, s, flags, seed=7 + call, offset=call)
        out = torch.full((nbytes // 4,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
        bits = torch.zeros(1, dtype=torch.int64, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        nuq.encode_static(g, bucket, s, flags, seed=7 + call, offset=call, out=out, out_bits=bits)
        torch.cuda.synchronize()
        if call == 1:                     # the driver's free-memory figure: nothing was taken from the device
            assert torch.cuda.mem_get_info()[0] == free_before
        assert nuq.last_status() == 0
        assert int(bits.item()) == int(ref_bits.item())
        assert np.array_equal(_container(torch, out, bits), _container(torch, ref_out, ref_bits))


def test_static_scratch_rejects_vectors_beyond_its_capacity():
    torch, nuq = require_cuda()
    g = torch.zeros(1024, device="cuda")
    out = torch.empty(1024, dtype=torch.int32, device="cuda")
    bits = torch.zeros(1, dtype=torch.int64, device="cuda")
    # only the arguments are inspected: d = 2^30 with bucket 8192 needs 1 MiB of scan state
    import ctypes as C
    rc = nuq._lib.nuq_encode_static(C.c_void_p(g.data_ptr()), 1 << 30, 8192, 4, 0, 0, 0, C.c_void_p(out.data_ptr()),
                                    C.c_void_p(bits.data_ptr()), None)
    assert rc == nuq.ERR_CAPACITY
    assert nuq.last_status() == 0
