"""The aggregation step of Algorithm 1 fused into the decoder (nuq_decode_update), against the oracle:
the sum of the decoded streams is the oracle's bit for bit, and the step applied to it (plain SGD, heavy
ball, Nesterov, a general l) agrees with the oracle's fp64 step to fp32 rounding."""
import numpy as np
import pytest

import oracle as O
from gpu_util import gpu_encode, require_cuda

pytestmark = pytest.mark.gpu

GUARD = 64


def _input(d, seed):
    rng = np.random.default_rng(seed)
    g = rng.standard_normal(d) * 10.0 ** rng.uniform(-4, 0, d)
    g[rng.random(d) < 0.02] = 0.0
    return g.astype(np.float32)


def _guarded(torch, host):
    buf = torch.full((host.size + 2 * GUARD,), float("nan"), dtype=torch.float32, device="cuda")
    buf[GUARD:GUARD + host.size] = torch.from_numpy(host).cuda()
    return buf, buf[GUARD:GUARD + host.size]


def _check_guard(buf, d, what):
    host = buf.cpu().numpy()
    assert np.isnan(host[:GUARD]).all() and np.isnan(host[GUARD + d:]).all(), f"the decoder wrote outside {what}"
    return host[GUARD:GUARD + d].copy()


def _tolerance(w0, yl0, total, alpha, K, mu, l):
    """a few fp32 roundings of the magnitudes the three lines of the step handle"""
    c = abs(alpha) / K
    y = np.abs(w0) + c * np.abs(total)
    yl = np.abs(w0) + l * c * np.abs(total)
    return 2.0 ** -21 * (y + mu * (yl + np.abs(yl0))) + 1e-30


def _step_and_compare(torch, nuq, dev_streams, host_streams, d, bucket, s, w0, yl0, alpha, mu, l, with_acc, with_yl=True):
    K = len(host_streams)
    rc, total = O.decode_accumulate(host_streams, d, bucket, s)
    assert rc == 0
    wbuf, w = _guarded(torch, w0)
    ylbuf, yl = _guarded(torch, yl0)
    accbuf, acc = _guarded(torch, np.zeros(d, np.float32))
    nuq.decode_update(dev_streams, d, bucket, s, w, yl if with_yl else None, alpha, mu, l, acc=acc if with_acc else None)
    assert nuq.last_status() == 0
    got_w, got_yl = _check_guard(wbuf, d, "w"), _check_guard(ylbuf, d, "yl")
    got_acc = _check_guard(accbuf, d, "acc")
    if with_acc:
        assert np.array_equal(got_acc.view(np.uint32), total.view(np.uint32))
    else:
        assert not got_acc.any()
    want_w, want_yl = O.momentum_step(w0, yl0, total, alpha, K, mu, l)
    tol = _tolerance(w0.astype(np.float64), yl0.astype(np.float64), total.astype(np.float64), alpha, K, mu, l)
    assert (np.abs(got_w - want_w) <= tol).all(), np.abs(got_w - want_w).max()
    if mu != 0.0:
        assert (np.abs(got_yl - want_yl) <= tol).all()
    else:
        assert np.array_equal(got_yl.view(np.uint32), yl0.view(np.uint32))      # not touched
    assert np.abs(got_w - w0).max() > 0
    return got_w, got_yl


@pytest.mark.parametrize("K,d,bucket,s,mode", [
    (1, 70001, 1024, 4, O.MODE_ERC),          # the sums are added up in acc itself (K <= 2)
    (2, 8192 * 3 + 17, 8192, 3, O.MODE_ERC),
    (4, 100037, 8192, 4, O.MODE_ERC),         # four streams side by side, sums in shared memory
    (8, 200000, 8192, 4, O.MODE_ERC),
    (9, 50000, 512, 4, O.MODE_ERC),           # two groups of streams
    (8, 100000, 8192, 4, O.MODE_FIXED),       # the fixed-width kernel, 4-bit fields
    (3, 70001, 768, 2, O.MODE_FIXED),         # the fixed-width kernel, other widths
    (3, 200000, 65536, 4, O.MODE_ERC),        # buckets wider than a tile
])
@pytest.mark.parametrize("alpha,mu,l", [(0.1, 0.0, 0.0), (0.05, 0.9, 0.0), (0.05, 0.9, 1.0), (0.3, 0.5, 0.25)])
def test_decode_update_matches_the_oracle(K, d, bucket, s, mode, alpha, mu, l):
    torch, nuq = require_cuda()
    flags = O.make_flags(mode=mode)
    rng = np.random.default_rng(d + K)
    outs, hosts = [], []
    nbytes = nuq.encode_bound(d, bucket, s, flags)
    for k in range(K):                                       # containers stay where the library wrote them
        out = torch.zeros(nbytes // 4, dtype=torch.int32, device="cuda")
        _, bits = nuq.encode(torch.from_numpy(_input(d, 17 * d + k)).cuda(), bucket, s, flags, 3 + k, 0, out=out)
        outs.append(out)
        hosts.append(out.cpu().numpy().view(np.uint32)[: int(bits.item()) // 32].copy())
    w0 = rng.standard_normal(d).astype(np.float32)
    yl0 = (w0 + 0.01 * rng.standard_normal(d)).astype(np.float32)
    with_acc = K < 3 or (d + K) % 2 == 0
    _step_and_compare(torch, nuq, outs, hosts, d, bucket, s, w0, yl0, alpha, mu, l, with_acc, with_yl=mu != 0.0 or K % 2 == 0)


def test_three_steps_carry_the_momentum_state():
    """w and y^l stay on the device from step to step; every step is checked against the oracle's step from
    the state the device held, and the whole trajectory against the oracle's own in fp64."""
    torch, nuq = require_cuda()
    d, bucket, s, K, alpha, mu, l = 60000, 4096, 4, 4, 0.2, 0.8, 1.0
    rng = np.random.default_rng(9)
    w = rng.standard_normal(d).astype(np.float32)
    yl = w.copy()                                            # at rest: y^l_0 = w_0
    fw, fyl = w.astype(np.float64), yl.astype(np.float64)    # the oracle's own trajectory
    for step in range(3):
        hosts = [gpu_encode(_input(d, 100 * step + k), bucket, s, 0, seed=k + 1, offset=step)[0] for k in range(K)]
        devs = [torch.from_numpy(h.view(np.int32)).cuda() for h in hosts]
        w, yl = _step_and_compare(torch, nuq, devs, hosts, d, bucket, s, w, yl, alpha, mu, l, with_acc=step == 1)
        fw, fyl = O.momentum_step(fw, fyl, O.decode_accumulate(hosts, d, bucket, s)[1], alpha, K, mu, l)
    assert np.abs(w - fw).max() <= 1e-5 * (1 + np.abs(fw).max())


def test_decode_update_refuses_what_it_cannot_do():
    torch, nuq = require_cuda()
    d, bucket, s = 5000, 256, 3
    host = gpu_encode(_input(d, 1), bucket, s, 0, 1, 0)[0]
    dev = torch.from_numpy(host.view(np.int32)).cuda()
    w = torch.zeros(d, device="cuda")
    yl = torch.zeros(d, device="cuda")
    acc = torch.zeros(d, device="cuda")
    for kwargs in (dict(streams=[dev, dev], acc=None),                      # K <= 2 needs acc
                   dict(streams=[dev] * 3, acc=None, mu=0.5, yl=None),      # momentum needs y^l
                   dict(streams=[dev] * 3, acc=acc, mu=1.0, yl=yl),         # mu in [0, 1)
                   dict(streams=[dev] * 3, acc=acc, mu=0.5, yl=yl, l=1.5),  # l in [0, 1]
                   dict(streams=[dev] * 3, acc=acc, alpha=float("nan"))):
        args = dict(yl=None, alpha=0.1, mu=0.0, l=0.0)
        args.update(kwargs)
        with pytest.raises(nuq.NuqError):
            nuq.decode_update(args["streams"], d, bucket, s, w, args["yl"], args["alpha"], args["mu"], args["l"],
                              acc=args["acc"])
    assert nuq.last_status() == 0 and not w.any().item()
