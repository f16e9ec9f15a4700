#!/usr/bin/env python
"""Benchmark of the NUQ encode / decode+accumulate hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic gradients:
K simulated workers are encoded (K calls of nuq_encode on K distinct inputs that
are resident in HBM) and their K containers are decoded and summed by one call of
nuq_decode_accumulate.  The metric is GB/s of fp32 gradient data moved through
the path ("fp32 in": 4*d bytes per encode call, 4*d bytes per decode call).

    python bench.py --gpus N --steps K --warmup W [--workload c3|c2|c4-8192|...]
    python bench.py --impl reference          # the CPU oracle on the same workload

Prints ONE JSON line.  With N > 1 (under torchrun) every rank runs an independent
replica of the workload (the path has no exchange step); the value is the sum.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
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
    "c4-512": ("C4 flat Laplace d=2^30, bucket 512, s=4, ERC, K=2", 1 << 30, 512, 4, 0, 2),
    "c4-8192": ("C4 flat Laplace d=2^30, bucket 8192, s=4, ERC, K=2", 1 << 30, 8192, 4, 0, 2),
    "c4-65536": ("C4 flat Laplace d=2^30, bucket 65536, s=4, ERC, K=2", 1 << 30, 65536, 4, 0, 2),
    "c5-qsgd": ("C5 ResNet-50-sized, uniform levels k/16, L2 norm, ERC, K=8", 25_557_032, 8192, 4, 1 << 8, 8),
    "c5-qsgdinf": ("C5 ResNet-50-sized, uniform levels k/16, Linf norm, ERC, K=8", 25_557_032, 8192, 4, (1 << 8) | 1, 8),
}


def worker_input(workload, k, d):
    """gradient of simulated worker k (1-based) as a float32 numpy array"""
    from paper_1908_06077_b200 import inputs
    if workload == "c1":
        return inputs.c1_input()
    if workload == "c2":
        return inputs.c2_input(k)
    if workload.startswith("c3") or workload.startswith("c5"):
        return inputs.c3_input(k)
    return inputs.c4_input(k, d)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


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


def oracle_step(workload, steps, warmup):
    """the CPU oracle on the same workload: K encodes + one decode_accumulate per step, single thread"""
    import oracle as O
    desc, d, bucket, s, flags, K = WORKLOADS[workload]
    n = min(d, 1 << 22) if workload.startswith("c4") else d          # bounded sample for the 2^30 case
    gs = [worker_input(workload, k + 1, n)[:n] for k in range(K)]
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        streams = [O.encode(gs[k], bucket, s, flags, k + 1, 0)[0] for k in range(K)]
        rc, _ = O.decode_accumulate(streams, n, bucket, s)
        assert rc == 0
        if it >= warmup:
            times.append(time.perf_counter() - t0)
    t = sum(times) / len(times)
    sample = f"{K} encodes + 1 decode_accumulate of the first {n} elements of each worker's gradient"
    return (K + 1) * 4.0 * n / t / 1e9, t * 1e3, sample


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    desc, d, bucket, s, flags, K = WORKLOADS[args.workload]
    steps, warmup = max(1, min(args.steps, 2)), min(args.warmup, 1)
    value, ms, sample = oracle_step(args.workload, steps, warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": desc, "d": d, "bucket": bucket, "s": s, "K": K},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


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

    desc, d, bucket, s, flags, K = WORKLOADS[args.workload]
    if args.d is not None:
        if not args.workload.startswith("c4") or args.d < 1 or args.d > d:
            raise SystemExit("--d shortens the C4 workloads only")
        d = args.d
        desc += f" (shortened to d={d})"
    steps, warmup = args.steps, max(args.warmup, 3)

    # ---- inputs: K distinct worker gradients, generated on the host, resident in HBM ----
    host = []
    for k in range(K):
        t = torch.from_numpy(worker_input(args.workload, k + 1, d))
        host.append(t.pin_memory() if args.e2e_steps > 0 else t)
    gs = [h.cuda() for h in host]
    nbytes = nuq.encode_bound(d, bucket, s, flags)
    outs = [torch.empty(nbytes // 4, dtype=torch.int32, device="cuda") for _ in range(K)]
    bits = [torch.zeros(1, dtype=torch.int64, device="cuda") for _ in range(K)]
    acc = torch.empty(d, dtype=torch.float32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")        # > L2 (126 MB)
    wide = bucket > 8192

    def step(timed):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        flush.fill_(1)
        ev[0].record()
        for k in range(K):
            nuq.encode(gs[k], bucket, s, flags, seed=k + 1, offset=0, out=outs[k], out_bits=bits[k])
        ev[1].record()
        flush.fill_(2)                                                     # containers leave L2 too
        ev[2].record()
        nuq.decode_accumulate(outs, d, bucket, s, acc=acc)
        ev[3].record()
        return ev

    for _ in range(warmup):
        step(False)
    torch.cuda.synchronize()
    assert nuq.last_status() == 0
    container_bytes = [int(b.item()) // 8 for b in bits]

    sampler = ClockSampler(local)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    events = [step(True) for _ in range(steps)]
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    assert nuq.last_status() == 0
    t_enc = sum(e[0].elapsed_time(e[1]) for e in events) / steps           # ms per step, K encodes
    t_dec = sum(e[2].elapsed_time(e[3]) for e in events) / steps
    t_step = t_enc + t_dec

    # ---- end to end: pinned host gradients in, summed gradient out ------------------------
    e2e = None
    if args.e2e_steps > 0:
        acc_host = torch.empty(d, dtype=torch.float32).pin_memory()
        tl = []
        for it in range(args.e2e_steps + 1):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for k in range(K):
                gs[k].copy_(host[k], non_blocking=True)
                nuq.encode(gs[k], bucket, s, flags, seed=k + 1, offset=0, out=outs[k], out_bits=bits[k])
            nuq.decode_accumulate(outs, d, bucket, s, acc=acc)
            acc_host.copy_(acc, non_blocking=True)
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
        enc_achieved = enc_bytes / (enc_launch_ms / 1e3) / 1e9
        dec_achieved = dec_bytes / (t_dec / 1e3) / 1e9
        line = {
            "metric": METRIC,
            "value": aggregate_value(world, K, d, t_step),
            "unit": "GB/s", "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": t_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": desc, "d": d, "bucket": bucket, "s": s, "K": K,
                       "container_bits_per_element": 8.0 * mean_container / d,
                       "l2": "256 MB written before the encode phase and before the decode phase of every step",
                       "parallelism": "replicas only" if world > 1 else "1 GPU"},
            "encode_gbs_fp32_in": K * 4.0 * d / (t_enc / 1e3) / 1e9,
            "decode_gbs_fp32_in": 4.0 * d / (t_dec / 1e3) / 1e9,
            "encode_ms_per_call": enc_launch_ms, "decode_ms_per_call": t_dec,
            "roofline": {"kernel": "encode_kernel", "bound": "hbm", "achieved": enc_achieved, "peak": peak,
                         "unit": "GB/s", "frac": enc_achieved / peak, "peak_kind": f"of {peak_kind}",
                         "frac_of_nominal_8000": enc_achieved / 8000.0,
                         "traffic": ENCODE_TRAFFIC_BYTES.get(args.workload) if args.d is None else None},
            "roofline_decode": {"kernel": "decode_kernel", "bound": "hbm", "achieved": dec_achieved, "peak": peak,
                                "unit": "GB/s", "frac": dec_achieved / peak, "peak_kind": f"of {peak_kind}",
                                "frac_of_nominal_8000": dec_achieved / 8000.0,
                                "traffic": DECODE_TRAFFIC_BYTES.get(args.workload) if args.d is None else None},
            # encode (+ bucket norms) per worker; one decode kernel, two when all streams are fixed-width
            "gpu_launches": steps * (K * (2 if wide else 1) + (2 if (flags >> 16) & 0xff else 1)),
            "clocks": clocks,
        }
        if e2e is not None:
            line["e2e"] = e2e
        if world == 1 and not args.no_cpu_baseline:
            v, ms, sample = oracle_step(args.workload, 1, 0)
            line["cpu_baseline"] = {"value": v, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample,
                                    "ms_per_step": ms}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch from the ncu captures
# summarised under profiles/ (the decoder's write count is short under ncu: its write-back
# drains after the kernel has ended)
ENCODE_TRAFFIC_BYTES = {"c3": 102.31e6 + 3.78e6}
DECODE_TRAFFIC_BYTES = {"c3": 24.67e6 + 44.29e6}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=sorted(WORKLOADS))
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--d", type=int, default=None,
                    help="C4 workloads only: a shorter vector (for profiler captures, which must stay small)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
