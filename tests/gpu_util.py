"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI
binding and bring results back as numpy arrays for comparison with the oracle."""
import numpy as np
import pytest

import oracle as O


def require_cuda():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_1908_06077_b200 import nuq
    return torch, nuq


def gpu_encode(g, bucket, s, flags, seed, offset, norms=None, prefill=None, expect_status=0):
    """container (uint32 numpy, trimmed to container_bits) produced by nuq_encode"""
    torch, nuq = require_cuda()
    gd = torch.from_numpy(np.ascontiguousarray(g, np.float32)).cuda()
    nbytes = nuq.encode_bound(gd.numel(), bucket, s, flags)
    assert nbytes > 0
    guard = 64
    out = torch.full((nbytes // 4 + guard,), -1515870811 if prefill is None else prefill, dtype=torch.int32,
                     device="cuda")                                   # 0xA5A5A5A5
    if norms is not None:
        nd = torch.from_numpy(np.ascontiguousarray(norms, np.float32)).cuda()
        nuq.set_test_norms(nd)
        flags |= nuq.TEST_NORMS
    _, bits = nuq.encode(gd, bucket, s, flags, seed, offset, out=out)
    status = nuq.last_status()
    if norms is not None:
        nuq.set_test_norms(None)
    assert status == expect_status, status
    nbits = int(bits.item())
    host = out.cpu().numpy().view(np.uint32)
    assert nbits % 32 == 0 and nbits // 8 <= nbytes
    assert (host[nbytes // 4:] == np.uint32(0xA5A5A5A5 if prefill is None else prefill & 0xFFFFFFFF)).all(), \
        "encoder wrote past nuq_encode_bound"
    return host[: nbits // 32].copy(), nbits


def gpu_decode(streams, d, bucket, s, expect_status=0):
    torch, nuq = require_cuda()
    dev = []
    for st in streams:
        t = torch.from_numpy(np.ascontiguousarray(st, np.uint32).view(np.int32)).cuda()
        dev.append(t)
    guard = 64
    buf = torch.full((d + 2 * guard,), float("nan"), dtype=torch.float32, device="cuda")
    acc = buf[guard:guard + d]
    nuq.decode_accumulate(dev, d, bucket, s, acc=acc)
    status = nuq.last_status()
    assert status == expect_status, status
    host = buf.cpu().numpy()
    assert np.isnan(host[:guard]).all() and np.isnan(host[guard + d:]).all(), "decoder wrote outside acc"
    return host[guard:guard + d].copy()


def near_threshold_mask(g, bucket, s, levelset, seed, offset, norms, window=1e-6):
    """elements whose uniform draw lies within `window` of the rounding probability (oracle arithmetic)"""
    d = g.size
    mask = np.zeros(d, bool)
    return mask, lambda idx: _near(g, bucket, s, levelset, seed, offset, norms, idx, window)


def _near(g, bucket, s, levelset, seed, offset, norms, idx, window):
    out = []
    for i in idx:
        _, p = O.round_probability(g[i], norms[i // bucket], s, levelset)
        u = O.draw_uniform(seed, offset, int(i))
        out.append(abs(u - float(p)) < window)
    return np.array(out, bool)


def compare_symbols(g, bucket, s, flags, seed, offset, gpu_stream):
    """spec criterion for a free-running encode: norms within 1e-6 relative; signs and level
    indices equal except where the draw is within 1e-6 of the threshold.  Returns the mismatch count."""
    nk, ls = flags & 0xff, (flags >> 8) & 0xff
    d = g.size
    rc, gsign, gsym, gnorms = O.decode_symbols(gpu_stream, d, bucket, s)
    assert rc == 0
    sign, sym, norms = O.quantize(g, bucket, s, nk, ls, seed, offset)
    live = np.isfinite(norms) & (norms > 0)
    rel = np.abs(gnorms[live].astype(np.float64) - norms[live]) / norms[live]
    assert rel.size == 0 or rel.max() <= 1e-6, rel.max()
    assert np.array_equal(gnorms[~live].view(np.uint32), norms[~live].view(np.uint32))
    bad = np.nonzero((gsym != sym) | (gsign != sign))[0]
    if bad.size:
        near = _near(g, bucket, s, ls, seed, offset, norms, bad, 1e-6)
        assert near.all(), f"{(~near).sum()} mismatches away from the rounding threshold, first at {bad[~near][:5]}"
        assert (np.abs(gsym[bad].astype(int) - sym[bad].astype(int)) <= 1).all()
    assert bad.size <= max(1e-5 * d, 0) or bad.size <= int(np.ceil(1e-5 * d)), bad.size
    worst = float(rel.max()) if rel.size else 0.0
    print(f"symbol mismatches={int(bad.size)} of d={d} (all within 1e-6 of the rounding threshold), "
          f"largest relative norm difference {worst:.3g}")
    return int(bad.size), worst


def gpu_level_histogram(g, bucket, s, flags, seed, offset, norms=None):
    """counts of the level indices 0..s+1 from nuq_level_histogram (uint64 numpy)"""
    torch, nuq = require_cuda()
    gd = torch.from_numpy(np.ascontiguousarray(g, np.float32)).cuda()
    buf = torch.full((s + 2 + 2,), -1, dtype=torch.int64, device="cuda")     # a guard word on either side
    if norms is not None:
        nd = torch.from_numpy(np.ascontiguousarray(norms, np.float32)).cuda()
        nuq.set_test_norms(nd)
        flags |= nuq.TEST_NORMS
    nuq.level_histogram(gd, bucket, s, flags, seed, offset, hist=buf[1:s + 3])
    status = nuq.last_status()
    if norms is not None:
        nuq.set_test_norms(None)
    assert status == 0, status
    host = buf.cpu().numpy()
    assert host[0] == -1 and host[-1] == -1, "histogram wrote outside its counters"
    return host[1:-1].astype(np.uint64)
