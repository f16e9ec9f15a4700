#!/usr/bin/env python
"""Benchmark of the NUQ encode / decode+accumulate hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic gradients:
K simulated workers are encoded (K calls of nuq_encode on K distinct inputs that
are resident in HBM) and their K containers are decoded and summed by one call of
nuq_decode_accumulate.  The metric is GB/s of fp32 gradient data moved through
the path ("fp32 in": 4*d bytes per encode call, 4*d bytes per decode call).

    python bench.py --gpus N --steps K --warmup W [--workload c3|c2|c4-8192|...]
    python bench.py --impl reference          # the CPU oracle on the same workload

Prints ONE JSON line.  The headline workload (default: C3, ERC) is timed for
exactly K steps; with the default workload the line also carries, under
"workloads", short timings of the other ResNet-sized configurations (fixed-width
mode, s = 2 and 3, the two uniform comparison quantizers, C2, C1) with their code
lengths and quantization variance.  With N > 1 (under torchrun) every rank runs an
independent replica of the workload (the path has no exchange step); the value is
the sum.
"""
import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "NUQ encode and decode+accumulate GB/s (fp32 in) and % of B200 HBM peak"
FALLBACK_HBM_GBS = 6650.0

# workload name -> (description, d, bucket, s, flags, K)
WORKLOADS = {
    "c1": ("C1 tiny: N(0,1) d=65536, bucket 1024, s=3, ERC, K=1", 65536, 1024, 3, 0, 1),
    "c2": ("C2 ResNet-18-sized gradient d=11689512, bucket 8192, s=4, ERC, K=4", 11_689_512, 8192, 4, 0, 4),
    "c3": ("C3 ResNet-50-sized gradient d=25557032, bucket 8192, s=4, ERC, K=8", 25_557_032, 8192, 4, 0, 8),
    "c3-s2": ("C3 ResNet-50-sized, s=2, ERC, K=8", 25_557_032, 8192, 2, 0, 8),
    "c3-s3": ("C3 ResNet-50-sized, s=3, ERC, K=8", 25_557_032, 8192, 3, 0, 8),
    "c3-fixed": ("C3 ResNet-50-sized, s=4, fixed 4-bit, K=8", 25_557_032, 8192, 4, 1 << 16, 8),
    "c3-coded": ("C3 ResNet-50-sized, s=4, level indices in a Huffman code fitted on worker 1's gradient, K=8",
                 25_557_032, 8192, 4, 2 << 16, 8),
    "c4-512": ("C4 flat Laplace d=2^30, bucket 512, s=4, ERC, K=2", 1 << 30, 512, 4, 0, 2),
    "c4-8192": ("C4 flat Laplace d=2^30, bucket 8192, s=4, ERC, K=2", 1 << 30, 8192, 4, 0, 2),
    "c4-65536": ("C4 flat Laplace d=2^30, bucket 65536, s=4, ERC, K=2", 1 << 30, 65536, 4, 0, 2),
    "c5-qsgd": ("C5 ResNet-50-sized, uniform levels k/16, L2 norm, ERC, K=8", 25_557_032, 8192, 4, 1 << 8, 8),
    "c5-qsgdinf": ("C5 ResNet-50-sized, uniform levels k/16, Linf norm, ERC, K=8", 25_557_032, 8192, 4, (1 << 8) | 1, 8),
}
# timed briefly behind the headline workload when that is the default one
SIDE_WORKLOADS = ["c3-fixed", "c3-coded", "c3-s2", "c3-s3", "c5-qsgd", "c5-qsgdinf", "c2", "c1"]

_input_cache = {}


def worker_input(workload, k, d):
    """gradient of simulated worker k (1-based) as a float32 numpy array"""
    from paper_1908_06077_b200 import inputs
    if workload == "c1":
        key = ("c1", 1)
    elif workload == "c2":
        key = ("c2", k)
    elif workload.startswith("c3") or workload.startswith("c5"):
        key = ("c3", k)
    else:
        return inputs.c4_input(k, d)
    if key not in _input_cache:
        _input_cache[key] = {"c1": lambda: inputs.c1_input(), "c2": lambda: inputs.c2_input(k),
                             "c3": lambda: inputs.c3_input(k)}[key[0]]()
    return _input_cache[key]


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def variance_bounds(bucket, s, flags):
    """what the paper proves about E||Q(v) - v||^2 / ||v||^2 for a bucket of this size (context for the
    measured figures): Theorem 1 for the exponential levels, in the form its proof supports (switch at
    sqrt(B) / 2^s = 2), and QSGD's bound min(B / s'^2, sqrt(B) / s') for s' = 2^s uniform levels"""
    if (flags >> 8) & 0xff == 0:
        delta = math.sqrt(bucket) / 2 ** s
        return {"theorem_1": 0.125 + delta * delta / 4 if delta < 2 else delta - 0.875}
    sp = 2 ** s
    return {"qsgd_bound": min(bucket / sp ** 2, math.sqrt(bucket) / sp)}


class ClockSampler:
    """samples nvidia-smi clocks and throttle reasons while the timed region runs"""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except Exception:
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons)}


def max_over_ranks(values, device):
    """element-wise maximum of a list of floats over all ranks (the timing of a multi-rank run is the
    slowest rank's); a no-op without a process group.  The only collective in this benchmark: the path
    itself has no exchange step, every rank runs an independent replica."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(values, device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def aggregate_value(world, K, d, t_step_ms):
    """whole-job GB/s (fp32 in): every rank moves (K + 1) * 4 * d bytes per step"""
    return world * (K + 1) * 4.0 * d / (t_step_ms / 1e3) / 1e9


# ---------------------------------------------------------------------------------------------
# CPU legs: the oracle, as it stands, on the host cores
# ---------------------------------------------------------------------------------------------
def _oracle_encode_job(job):
    import oracle as O
    workload, k, n, bucket, s, flags = job
    g = worker_input(workload, k + 1, n)[:n]
    return O.encode(g, bucket, s, flags, k + 1, 0)[0]


def _oracle_fit_code(workload, n, bucket, s, flags):
    """coded level indices: the oracle fits its own code on worker 1's gradient (as the GPU leg does with its own)"""
    import oracle as O
    if (flags >> 16) & 0xff != O.MODE_CODED:
        return None
    g = worker_input(workload, 1, n)[:n]
    _, sym, _ = O.quantize(g, bucket, s, flags & 0xff, (flags >> 8) & 0xff, 1, 0)
    lengths = O.huffman_lengths(O.level_histogram(sym, s)[1:])
    O.set_level_code(lengths)
    return [int(x) for x in lengths]


def oracle_step(workload, steps, warmup, all_cores=False):
    """the CPU oracle on the same workload: K encodes + one decode_accumulate per step; on one core, or
    with the K encodes spread over a process pool (the oracle's C code itself is single threaded)"""
    import oracle as O
    desc, d, bucket, s, flags, K = WORKLOADS[workload]
    n = min(d, 1 << 22) if workload.startswith("c4") else d          # bounded sample for the 2^30 case
    gs = [worker_input(workload, k + 1, n)[:n] for k in range(K)]
    _oracle_fit_code(workload, n, bucket, s, flags)         # before the pool forks: its processes inherit the code
    pool, cores = None, 1
    if all_cores and K > 1:
        import multiprocessing as mp
        cores = min(K, os.cpu_count() or 1)
        pool = mp.get_context("fork").Pool(cores)
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        if pool is not None:
            streams = pool.map(_oracle_encode_job, [(workload, k, n, bucket, s, flags) for k in range(K)])
        else:
            streams = [O.encode(gs[k], bucket, s, flags, k + 1, 0)[0] for k in range(K)]
        rc, _ = O.decode_accumulate(streams, n, bucket, s)
        assert rc == 0
        if it >= warmup:
            times.append(time.perf_counter() - t0)
    if pool is not None:
        pool.close()
    t = sum(times) / len(times)
    sample = f"{K} encodes + 1 decode_accumulate of the first {n} elements of each worker's gradient"
    return (K + 1) * 4.0 * n / t / 1e9, t * 1e3, sample, cores


def cpu_leg(args):
    """Runs in a process of its own (no CUDA context, so that it may fork a pool): times the oracle on one
    core and on all cores, evaluates Lemma 7's closed form of the quantization variance on worker 1's
    gradient, and counts where the GPU's symbols of worker 1 (container passed in a file) differ from the
    oracle's.  Prints one JSON object."""
    import oracle as O
    desc, d, bucket, s, flags, K = WORKLOADS[args.workload]
    out = {}
    v, ms, sample, _ = oracle_step(args.workload, 1, 0)
    out["cpu_baseline"] = {"value": v, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample, "ms_per_step": ms}
    va, msa, _, cores = oracle_step(args.workload, 1, 0, all_cores=True)
    out["cpu_baseline"]["all_cores"] = {"value": va, "unit": "GB/s", "cores": cores, "nproc": os.cpu_count(),
                                        "ms_per_step": msa,
                                        "how": "the K encodes in a process pool, the decode on one core"}
    n = min(d, 1 << 22) if args.workload.startswith("c4") else d
    g = worker_input(args.workload, 1, n)[:n]
    nk, ls = flags & 0xff, (flags >> 8) & 0xff
    norms = O.bucket_norms(g, bucket, nk)
    num = 0.0
    for b, lo in enumerate(range(0, n, bucket)):
        if np.isfinite(norms[b]) and norms[b] > 0:
            num += O.variance_closed_form(g[lo:lo + bucket], norms[b], s, ls)
    out["variance_closed_form"] = num / float(np.sum(g.astype(np.float64) ** 2))
    if args.container and n == d:
        st = np.load(args.container)
        rc, gsign, gsym, gnorms = O.decode_symbols(st, d, bucket, s)
        sign, sym, _ = O.quantize(g, bucket, s, nk, ls, 1, 0, norms=norms)
        live = np.isfinite(norms) & (norms > 0)
        rel = np.abs(gnorms[live].astype(np.float64) - norms[live]) / norms[live]
        out["symbol_check"] = {"worker": 1, "status": rc, "symbol_mismatches": int(((gsym != sym) | (gsign != sign)).sum()),
                               "d": d, "allowed": int(math.ceil(1e-5 * d)),
                               "norm_max_relative_difference": float(rel.max()) if rel.size else 0.0}
    print(json.dumps(out))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    desc, d, bucket, s, flags, K = WORKLOADS[args.workload]
    steps, warmup = max(1, min(args.steps, 2)), min(args.warmup, 1)
    value, ms, sample, _ = oracle_step(args.workload, steps, warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": desc, "d": d, "bucket": bucket, "s": s, "K": K},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
# GPU legs
# ---------------------------------------------------------------------------------------------
class Workload:
    """the device buffers of one workload and its timed step"""

    def __init__(self, name, d_override=None, pin=False):
        import torch
        from paper_1908_06077_b200 import nuq
        self.torch, self.nuq, self.name = torch, nuq, name
        self.desc, self.d, self.bucket, self.s, self.flags, self.K = WORKLOADS[name]
        if d_override is not None:
            self.d = d_override
            self.desc += f" (shortened to d={self.d})"
        self.host = []
        for k in range(self.K):
            t = torch.from_numpy(worker_input(name, k + 1, self.d))
            self.host.append(t.pin_memory() if pin else t)
        self.gs = [h.cuda() for h in self.host]
        nbytes = nuq.encode_bound(self.d, self.bucket, self.s, self.flags)
        self.outs = [torch.empty(nbytes // 4, dtype=torch.int32, device="cuda") for _ in range(self.K)]
        self.bits = [torch.zeros(1, dtype=torch.int64, device="cuda") for _ in range(self.K)]
        self.acc = torch.empty(self.d, dtype=torch.float32, device="cuda")
        self.level_code = None
        if (self.flags >> 16) & 0xff == 2:
            # coded level indices: the code is fitted once on worker 1's gradient (the paper's "initial
            # sample"), outside the timed region, and kept for every step and every worker
            hist = nuq.level_histogram(self.gs[0], self.bucket, self.s, self.flags & 0xffff, seed=1, offset=0)
            self.level_histogram = [int(x) for x in hist.cpu().tolist()]
            self.level_code = nuq.fit_level_code(self.level_histogram, self.s)
            nuq.set_level_code(self.level_code)

    def step(self, flush):
        torch, nuq = self.torch, self.nuq
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        if flush is not None:
            flush.fill_(1)
        ev[0].record()
        for k in range(self.K):
            nuq.encode(self.gs[k], self.bucket, self.s, self.flags, seed=k + 1, offset=0, out=self.outs[k],
                       out_bits=self.bits[k])
        ev[1].record()
        if flush is not None:
            flush.fill_(2)                                                 # containers leave L2 too
        ev[2].record()
        nuq.decode_accumulate(self.outs, self.d, self.bucket, self.s, acc=self.acc)
        ev[3].record()
        return ev

    def timed(self, steps, warmup, flush, before=None, after=None):
        """(per-step encode ms, per-step decode ms) over `steps` steps after `warmup` untimed ones"""
        for _ in range(warmup):
            self.step(flush)
        self.torch.cuda.synchronize()
        assert self.nuq.last_status() == 0
        if before:
            before()
        events = [self.step(flush) for _ in range(steps)]
        self.torch.cuda.synchronize()
        if after:
            after()
        assert self.nuq.last_status() == 0
        return [e[0].elapsed_time(e[1]) for e in events], [e[2].elapsed_time(e[3]) for e in events]

    def stream_stats(self):
        """code lengths of the containers as the paper counts them and as they are sent"""
        infos = [self.nuq.stream_info(o) for o in self.outs]
        d, K = self.d, self.K
        nb = (d + self.bucket - 1) // self.bucket
        code = sum(i["code_bits"] for i in infos) / K
        cont = sum(i["container_bits"] for i in infos) / K
        return {"bits_per_element": {"tokens": code / d, "tokens_plus_norms": (code + 32.0 * nb) / d,
                                     "container": cont / d},
                "nnz_fraction": sum(i["nnz"] for i in infos) / K / d,
                "container_bytes": [i["container_bits"] // 8 for i in infos]}

    def single_draw_variance(self):
        """||Q(v) - v||^2 / ||v||^2 of worker 1's draw, from the GPU's own decode of its container"""
        self.nuq.decode_accumulate(self.outs[:1], self.d, self.bucket, self.s, acc=self.acc)
        g = self.gs[0].double()
        finite = self.torch.isfinite(g)
        num = ((self.acc.double() - g)[finite] ** 2).sum()
        return float(num / (g[finite] ** 2).sum())

    def fused_update(self, flush, reps=5):
        """The aggregation step of Algorithm 1 fused into the decoder (nuq_decode_update, Nesterov momentum):
        time per call beside the unfused pair it replaces (the decode call, then an optimizer step made
        of torch's elementwise kernels, for context)."""
        torch, nuq = self.torch, self.nuq
        w = torch.zeros(self.d, device="cuda")
        yl = torch.zeros(self.d, device="cuda")
        alpha, mu, l = 0.1, 0.9, 1.0
        acc = self.acc if self.K < 3 else None              # with one or two streams the library adds up in acc
        fused, pair = [], []
        for it in range(reps + 2):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            flush.fill_(3)
            ev[0].record()
            nuq.decode_update(self.outs, self.d, self.bucket, self.s, w, yl, alpha, mu, l, acc=acc)
            ev[1].record()
            flush.fill_(4)
            ev[2].record()
            nuq.decode_accumulate(self.outs, self.d, self.bucket, self.s, acc=self.acc)
            c = alpha / self.K                              # y = w - c G; y^l = w - l c G; w = y + mu (y^l - y^l_prev)
            yl_next = torch.add(w, self.acc, alpha=-l * c)
            w.add_(self.acc, alpha=-c).add_(yl_next - yl, alpha=mu)
            yl.copy_(yl_next)
            ev[3].record()
            torch.cuda.synchronize()
            if it >= 2:
                fused.append(ev[0].elapsed_time(ev[1]))
                pair.append(ev[2].elapsed_time(ev[3]))
        assert nuq.last_status() == 0
        d4 = 4.0 * self.d
        containers = sum(self.stream_stats()["container_bytes"])
        ms = statistics.median(fused)
        return {"what": "w, y^l <- momentum step (mu 0.9, l 1) on the decoded sum, one call",
                "decode_update_us_per_call": 1e3 * ms,
                "decode_then_torch_step_us": 1e3 * statistics.median(pair),
                "algorithmic_bytes": containers + 4 * d4 + (d4 if acc is not None else 0.0),
                "achieved_gbs": (containers + 4 * d4 + (d4 if acc is not None else 0.0)) / (ms / 1e3) / 1e9}

    def launches_per_step(self):
        # my kernels only: one encode kernel per worker (two for buckets wider than a tile in the 4-bit
        # fixed-width mode: the norms come first; otherwise a cluster adds the norm up inside the encode
        # kernel), one decode kernel (two when all streams are fixed-width: that path's own kernel, then
        # the general one, which returns at once)
        fixed = (self.flags >> 16) & 0xff == 1
        wide = self.bucket > 8192
        return self.K * (2 if wide and fixed else 1) + (2 if fixed else 1)


def summarize(ms):
    return {"mean": sum(ms) / len(ms), "median": statistics.median(ms), "best": min(ms)}


def roofline_entry(kernel, algorithmic_bytes, ms, peak, peak_kind, traffic):
    achieved = algorithmic_bytes / (ms / 1e3) / 1e9
    return {"kernel": kernel, "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "frac_of_nominal_8000": achieved / 8000.0,
            "traffic": traffic}


def side_report(w, steps, flush, peak):
    """short timing and code statistics of one of the other configurations"""
    enc, dec = w.timed(steps, 3, flush)
    stats = w.stream_stats()
    cb = stats.pop("container_bytes")
    enc_call = [e / w.K for e in enc]
    rep = {"workload": w.desc, "encode_us_per_call": {k: 1e3 * v for k, v in summarize(enc_call).items()},
           "decode_us_per_call": {k: 1e3 * v for k, v in summarize(dec).items()},
           "encode_frac": (4.0 * w.d + sum(cb) / w.K) / (statistics.median(enc_call) / 1e3) / 1e9 / peak,
           "decode_frac": (sum(cb) + 4.0 * w.d) / (statistics.median(dec) / 1e3) / 1e9 / peak}
    rep.update(stats)
    if w.level_code is not None:
        rep["level_code_lengths"] = w.level_code
        rep["level_histogram"] = w.level_histogram
    rep["variance_single_draw"] = w.single_draw_variance()
    rep["variance_bound"] = variance_bounds(w.bucket, w.s, w.flags)
    if w.d <= 30_000_000:                                   # the ResNet-sized and tiny configurations: L2 left warm
        enc_w, dec_w = w.timed(steps, 1, None)
        rep["l2_warm"] = {"encode_us_per_call": 1e3 * statistics.median(enc_w) / w.K,
                          "decode_us_per_call": 1e3 * statistics.median(dec_w)}
    return rep


def run_gpu(args):
    import torch
    import torch.distributed as dist

    from paper_1908_06077_b200 import nuq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    if args.d is not None:
        dmax = WORKLOADS[args.workload][1]
        if not args.workload.startswith("c4") or args.d < 1 or args.d > dmax:
            raise SystemExit("--d shortens the C4 workloads only")
    steps, warmup = args.steps, max(args.warmup, 3)

    # ---- inputs: K distinct worker gradients, generated on the host, resident in HBM ----
    w = Workload(args.workload, args.d, pin=args.e2e_steps > 0)
    d, bucket, s, flags, K = w.d, w.bucket, w.s, w.flags, w.K
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")        # > L2 (126 MB)

    sampler = ClockSampler(local)

    def before():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        sampler.start()

    clocks = {}

    def after():
        if world > 1:
            dist.barrier()
        clocks.update(sampler.stop())

    enc_ms, dec_ms = w.timed(steps, warmup, flush, before, after)
    t_enc, t_dec = sum(enc_ms) / steps, sum(dec_ms) / steps                # ms per step: K encodes, one decode
    t_step = t_enc + t_dec
    stats = w.stream_stats()
    container_bytes = stats.pop("container_bytes")
    fused_update = w.fused_update(flush) if rank == 0 else None

    # ---- end to end: pinned host gradients in, summed gradient out ------------------------
    e2e = None
    if args.e2e_steps > 0:
        acc_host = torch.empty(d, dtype=torch.float32).pin_memory()
        tl = []
        for it in range(args.e2e_steps + 1):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for k in range(K):
                w.gs[k].copy_(w.host[k], non_blocking=True)
                nuq.encode(w.gs[k], bucket, s, flags, seed=k + 1, offset=0, out=w.outs[k], out_bits=w.bits[k])
            nuq.decode_accumulate(w.outs, d, bucket, s, acc=w.acc)
            acc_host.copy_(w.acc, non_blocking=True)
            torch.cuda.synchronize()
            if it > 0:
                tl.append(time.perf_counter() - t0)
        t_e2e = sum(tl) / len(tl)
        e2e = {"value": (K + 1) * 4.0 * d / t_e2e / 1e9, "unit": "GB/s", "h2d_bytes_per_step": K * 4 * d,
               "d2h_bytes_per_step": 4 * d, "ms_per_step": t_e2e * 1e3}

    # ---- max over ranks ---------------------------------------------------------------------
    t_step, t_enc, t_dec = max_over_ranks([t_step, t_enc, t_dec], "cuda")
    if e2e is not None:
        e2e["ms_per_step"] = max_over_ranks([e2e["ms_per_step"]], "cuda")[0]
        e2e["value"] = aggregate_value(world, K, d, e2e["ms_per_step"])

    if rank == 0:
        peak, peak_kind = measured_peak()
        mean_container = sum(container_bytes) / K
        enc_launch_ms = t_enc / K
        enc_bytes = 4.0 * d + mean_container                               # read g once, write the container
        dec_bytes = sum(container_bytes) + 4.0 * d                         # read K containers, write acc once
        full = args.d is None
        line = {
            "metric": METRIC,
            "value": aggregate_value(world, K, d, t_step),
            "unit": "GB/s", "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": t_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.desc, "d": d, "bucket": bucket, "s": s, "K": K,
                       "container_bits_per_element": 8.0 * mean_container / d,
                       "l2": "256 MB written before the encode phase and before the decode phase of every step",
                       "parallelism": "replicas only" if world > 1 else "1 GPU"},
            "encode_gbs_fp32_in": K * 4.0 * d / (t_enc / 1e3) / 1e9,
            "decode_gbs_fp32_in": 4.0 * d / (t_dec / 1e3) / 1e9,
            "encode_ms_per_call": enc_launch_ms, "decode_ms_per_call": t_dec,
            "encode_us_per_call": {k: 1e3 * v for k, v in summarize([e / K for e in enc_ms]).items()},
            "decode_us_per_call": {k: 1e3 * v for k, v in summarize(dec_ms).items()},
            "roofline": roofline_entry(ENCODE_KERNEL.get(args.workload, "encode_kernel"), enc_bytes, enc_launch_ms, peak, peak_kind,
                                       ENCODE_TRAFFIC_BYTES.get(args.workload) if full else None),
            "roofline_decode": roofline_entry(DECODE_KERNEL.get(args.workload, "decode_kernel"), dec_bytes, t_dec, peak, peak_kind,
                                              DECODE_TRAFFIC_BYTES.get(args.workload) if full else None),
            "gpu_launches": steps * w.launches_per_step(),
            "clocks": clocks,
        }
        line.update(stats)
        line["fused_update"] = fused_update
        if w.level_code is not None:
            line["level_code_lengths"] = w.level_code
            line["level_histogram"] = w.level_histogram
        line["variance_single_draw"] = w.single_draw_variance()
        line["variance_bound"] = variance_bounds(bucket, s, flags)
        if e2e is not None:
            line["e2e"] = e2e
        if world == 1 and d <= 30_000_000:
            enc_w, dec_w = w.timed(min(steps, 10), 1, None)
            line["l2_warm"] = {"encode_us_per_call": 1e3 * statistics.median(enc_w) / K,
                               "decode_us_per_call": 1e3 * statistics.median(dec_w)}
        if world == 1 and not args.no_cpu_baseline:
            # the oracle legs run in a process of their own, which never creates a CUDA context
            with tempfile.TemporaryDirectory() as tmp:
                path = os.path.join(tmp, "worker1.npy")
                nwords = container_bytes[0] // 4
                np.save(path, w.outs[0][:nwords].cpu().numpy().view(np.uint32))
                cmd = [sys.executable, os.path.abspath(__file__), "--cpu-leg", "--workload", args.workload,
                       "--container", path]
                res = subprocess.run(cmd, capture_output=True, text=True)
            if res.returncode == 0:
                leg = json.loads(res.stdout.strip().splitlines()[-1])
                line["cpu_baseline"] = leg["cpu_baseline"]
                line["variance_closed_form"] = leg.get("variance_closed_form")
                if "symbol_check" in leg:
                    line["symbol_check"] = leg["symbol_check"]
            else:
                line["cpu_baseline"] = {"error": res.stderr.strip()[-300:]}
        if world == 1 and args.workload == "c3" and full and not args.no_side_workloads:
            del w
            side = {}
            for name in SIDE_WORKLOADS:
                sw = Workload(name)
                side[name] = side_report(sw, args.side_steps, flush, peak)
                del sw
                torch.cuda.empty_cache()
            line["workloads"] = side
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch from the ncu captures
# summarised under profiles/.  Reads equal the algorithmic reads; the writes counted are those that
# had left the 126 MB L2 when the kernel ended (a container or the sums of C3 fit in it), so the
# totals of the decoders and of the fixed-width encoder lie below the algorithmic bytes.
ENCODE_TRAFFIC_BYTES = {"c3": 102_306_816 + 3_938_560, "c3-fixed": 102_282_752 + 4_993_024}
DECODE_TRAFFIC_BYTES = {"c3": 24_617_728 + 44_184_320, "c3-fixed": 102_410_752 + 57_455_872}
# the kernel that does the work of a call, where it is not the general one
ENCODE_KERNEL = {"c3-fixed": "encode_fixed4_kernel"}
DECODE_KERNEL = {"c3-fixed": "decode_fixed_kernel"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=sorted(WORKLOADS))
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-side-workloads", action="store_true",
                    help="do not time the other ResNet-sized configurations behind the headline workload")
    ap.add_argument("--side-steps", type=int, default=5)
    ap.add_argument("--d", type=int, default=None,
                    help="C4 workloads only: a shorter vector (for profiler captures, which must stay small)")
    ap.add_argument("--cpu-leg", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--container", default=None, help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.cpu_leg:
        cpu_leg(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
