"""Seeded synthetic gradient generators for the five benchmark workloads.

This module holds no arithmetic of the method (no norms, levels, codes): it
only draws inputs.  It is the one module that both the tests' CPU oracle and
the CUDA path are fed from.

The paper trains ResNets on ImageNet / CIFAR-10 (Sec. 5); those datasets and
trajectories are not available offline, so each workload is a stand-in with the
same length, bucket / level settings and a per-layer scale structure (tensor
fusion mixes layers of very different scale inside one bucket, Sec. 5 "Horovod
tensor fusion").  Everything is drawn with numpy's PCG64 in fp64 and cast to
fp32 on the host.

    C1  d = 65 536            N(0,1), seed 0
    C2  ResNet-18 layout      per layer N(0, sigma_l^2), sigma_l log-uniform
                              [1e-4, 1e-1], 0.1 % entries replaced by +-50 sigma_l
    C3  ResNet-50 layout      Student-t(3) * scale_l, scale_l log-uniform [1e-5, 1e-1]
    C4  d = 2^30 flat         Laplace(0, 1e-3), 1 % of entries exactly zero,
                              generated in independent 2^22-element chunks
    C5  = C3 inputs (other quantizers)
"""
from __future__ import annotations

import numpy as np

RESNET18_NUMEL = 11_689_512
RESNET50_NUMEL = 25_557_032
C4_NUMEL = 1 << 30
C4_CHUNK = 1 << 22


def _conv(cin, cout, k):
    return [("conv", cout * cin * k * k)]


def _bn(c):
    return [("bn_w", c), ("bn_b", c)]


def resnet18_layer_sizes():
    """Parameter tensor sizes of ResNet-18 (BasicBlock, [2,2,2,2]) in module order."""
    t = _conv(3, 64, 7) + _bn(64)
    cin = 64
    for stage, width in enumerate((64, 128, 256, 512)):
        for block in range(2):
            stride = 2 if (stage > 0 and block == 0) else 1
            t += _conv(cin, width, 3) + _bn(width) + _conv(width, width, 3) + _bn(width)
            if stride != 1 or cin != width:
                t += _conv(cin, width, 1) + _bn(width)
            cin = width
    t += [("fc_w", 512 * 1000), ("fc_b", 1000)]
    sizes = [n for _, n in t]
    assert sum(sizes) == RESNET18_NUMEL, sum(sizes)
    return sizes


def resnet50_layer_sizes():
    """Parameter tensor sizes of ResNet-50 (Bottleneck, [3,4,6,3], expansion 4)."""
    t = _conv(3, 64, 7) + _bn(64)
    cin = 64
    for stage, (width, blocks) in enumerate(((64, 3), (128, 4), (256, 6), (512, 3))):
        for block in range(blocks):
            out = width * 4
            t += _conv(cin, width, 1) + _bn(width) + _conv(width, width, 3) + _bn(width)
            t += _conv(width, out, 1) + _bn(out)
            if block == 0:
                t += _conv(cin, out, 1) + _bn(out)
            cin = out
    t += [("fc_w", 2048 * 1000), ("fc_b", 1000)]
    sizes = [n for _, n in t]
    assert sum(sizes) == RESNET50_NUMEL, sum(sizes)
    return sizes


def _rng(*key):
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence(list(key))))


def c1_input():
    """C1: d = 65 536 i.i.d. N(0,1), data seed 0."""
    return np.random.Generator(np.random.PCG64(0)).standard_normal(65536).astype(np.float32)


def c2_input(worker: int):
    """C2: ResNet-18-shaped gradient of simulated worker `worker` (1..4)."""
    sizes = resnet18_layer_sizes()
    sigma = 10.0 ** _rng(100).uniform(-4.0, -1.0, len(sizes))      # layout seed 100, shared by workers
    out = np.empty(RESNET18_NUMEL, np.float32)
    pos = 0
    for l, n in enumerate(sizes):
        r = _rng(100 + worker, l)
        x = r.standard_normal(n) * sigma[l]
        hit = r.random(n) < 1e-3
        x[hit] = 50.0 * sigma[l] * np.where(r.random(int(hit.sum())) < 0.5, -1.0, 1.0)
        out[pos:pos + n] = x
        pos += n
    return out


def c3_input(worker: int):
    """C3 / C5: ResNet-50-shaped heavy-tailed gradient of simulated worker `worker` (1..8)."""
    sizes = resnet50_layer_sizes()
    scale = 10.0 ** _rng(200).uniform(-5.0, -1.0, len(sizes))      # layout seed 200
    out = np.empty(RESNET50_NUMEL, np.float32)
    pos = 0
    for l, n in enumerate(sizes):
        out[pos:pos + n] = _rng(200 + worker, l).standard_t(3.0, n) * scale[l]
        pos += n
    return out


def c4_chunk(worker: int, chunk: int, n: int = C4_CHUNK):
    """C4: chunk `chunk` (n elements) of worker `worker`'s (1..2) flat Laplace gradient."""
    r = _rng(300 + worker, chunk)
    x = r.laplace(0.0, 1e-3, n)
    x[r.random(n) < 0.01] = 0.0
    return x.astype(np.float32)


def c4_input(worker: int, d: int = C4_NUMEL):
    """C4 whole vector (d a multiple of the chunk size, or smaller than one chunk)."""
    if d <= C4_CHUNK:
        return c4_chunk(worker, 0, d)
    assert d % C4_CHUNK == 0
    out = np.empty(d, np.float32)
    for c in range(d // C4_CHUNK):
        out[c * C4_CHUNK:(c + 1) * C4_CHUNK] = c4_chunk(worker, c)
    return out
