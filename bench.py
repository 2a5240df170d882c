#!/usr/bin/env python
"""Benchmark of the LC-Checkpoint hot path on B200: one step = one compress of a 1.3 B-parameter fp32
snapshot (nbits 5) + one recovery that applies a chain of 4 streams, all HBM-resident.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0). ``value`` is GB/s of fp32 state through the whole step, aggregated over
all ranks (every rank runs an independent replica of the workload: the path does not shard).
``--impl reference`` times the CPU oracle on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "compress/recover GB/s of fp32 state on 1 B200, % HBM peak; compression ratio"
WORKLOAD = "xfmr1p3b"  # the workload the metric is quoted on; --workload picks another config for reference
CPU_SAMPLE_ELEMS = 1 << 27  # bounded oracle sample: first 134,217,728 elements of the workload
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measured_traffic(kernel, n):
    """DRAM bytes per launch of `kernel` from the committed ncu capture (profiles/traffic.txt holds bytes per
    element measured on a smaller case; every pass is a linear scan, so traffic scales with n). None if absent."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.txt")) as f:
            table = dict(line.split() for line in f if line.strip() and not line.startswith("#"))
        per_elem = table.get(kernel.split("<")[0])
        return None if per_elem is None else float(per_elem) * n
    except Exception:
        return None


# ------------------------------------------------------------------------------------------- clocks


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU; keeps the samples of the timed region.

    nvidia-smi takes a moment to start, so it is launched before the warm-up; ``mark_start`` and
    ``stop`` bracket the timed region and only samples that arrived between them are reported.
    """

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        import threading

        self.lines = []  # (arrival time, text)
        self.t_start = None
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line))

    def wait_ready(self, timeout=10.0):
        t0 = time.perf_counter()
        while self.proc is not None and not self.lines and time.perf_counter() - t0 < timeout:
            time.sleep(0.01)

    def mark_start(self):
        self.t_start = time.perf_counter()

    def stop(self):
        t_end = time.perf_counter()
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.03)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for t, line in list(self.lines):
            if self.t_start is not None and not (self.t_start <= t <= t_end + 0.02):
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ------------------------------------------------------------------------------------------- N > 1


def dist_setup(n_gpus):
    """Returns (rank, world, local_rank). One process per GPU under torchrun; single process otherwise."""
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        backend = "nccl" if os.environ.get("LC_BENCH_BACKEND", "nccl") == "nccl" else "gloo"
        dist.init_process_group(backend=backend)
        return dist.get_rank(), world, int(os.environ.get("LOCAL_RANK", "0"))
    if n_gpus != 1:
        raise SystemExit("--gpus %d needs torchrun with that many ranks" % n_gpus)
    return 0, 1, 0


def max_over_ranks(value, device=None):
    """Largest ``value`` over all ranks (the job is as slow as its slowest replica)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def aggregate_value(units_per_rank, world, max_ms):
    """Whole-job throughput: units of all ranks divided by the slowest rank's time (units/ms -> G/s)."""
    return units_per_rank * world / (max_ms * 1e-3) / 1e9


# ------------------------------------------------------------------------------------------- arms


def run_reference(args, rank):
    """The CPU oracle, as it stands, timed on a bounded sample of the workload (rank 0 only)."""
    if rank != 0:
        return None
    import numpy as np  # noqa: F401

    from oracle import lc_oracle
    from paper_2009_13003_b200 import synth

    cfg = synth.CONFIGS[WORKLOAD]
    # bounded sample: the oracle does about 12 M elements per second of (compress + chain-of-4 recover) on one
    # core, and the whole run (set-up, warm-up, steps) should end within a few minutes
    budget_s = 150.0
    m = int(budget_s / (args.steps + args.warmup + 2) * 12e6) // 4096 * 4096
    m = max(4096, min(CPU_SAMPLE_ELEMS, m, cfg.n))
    u0 = synth.base_state(cfg, "cpu", m).numpy()
    tracked, u, streams = u0.copy(), u0.copy(), []
    for t in range(1, cfg.chain + 1):
        u = u + synth.snapshot_delta(cfg, t, "cpu", m).numpy()
        s = lc_oracle.compress(tracked, u, cfg.nbits)
        streams.append(s)
        if t < cfg.chain:
            tracked = lc_oracle.recover(tracked, [s])
    times = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        lc_oracle.compress(tracked, u, cfg.nbits)
        lc_oracle.recover(u0, streams)
        if it >= args.warmup:
            times.append(time.perf_counter() - t0)
    ms = 1e3 * sum(times) / len(times)
    value = 2 * 4 * m / (ms * 1e-3) / 1e9
    sample = "first %d of %d elements, compress + recover(chain 4) per step" % (m, cfg.n)
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "n": cfg.n, "nbits": cfg.nbits, "recover_chain": cfg.chain,
                   "sample_elems": m},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def time_oracle_sample(cfg, n, u0, tracked, u, streams_dev):
    """cpu_baseline leg: the oracle on the first CPU_SAMPLE_ELEMS elements of the same device inputs."""
    from oracle import lc_oracle

    m = min(CPU_SAMPLE_ELEMS, n)
    u0_h, tr_h, u_h = (x[:m].cpu().numpy() for x in (u0, tracked, u))
    # the sample's own chain (tables depend on the whole vector, so the sample is coded on its own)
    t0 = time.perf_counter()
    s = lc_oracle.compress(tr_h, u_h, cfg.nbits)
    t_c = time.perf_counter() - t0
    t0 = time.perf_counter()
    lc_oracle.recover(u0_h, [s] * cfg.chain)
    t_r = time.perf_counter() - t0
    value = 2 * 4 * m / (t_c + t_r) / 1e9
    return {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle",
            "sample": "first %d of %d elements: 1 compress (%.2f s) + 1 recover of a chain of %d (%.2f s)"
                      % (m, n, t_c, cfg.chain, t_r),
            "compress_gbs": 4 * m / t_c / 1e9, "recover_gbs": 4 * m / t_r / 1e9}


def run_ours(args, rank, world, local_rank):
    import torch

    from paper_2009_13003_b200 import binding as lc
    from paper_2009_13003_b200 import synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    lc.lib()
    cfg = synth.CONFIGS[args.workload]
    n, nbits, chain = cfg.n, cfg.nbits, cfg.chain
    if args.elems:
        n = args.elems

    def recover_chain(dst):
        # lc_recover applies at most MAX_CHAIN streams; longer chains continue in place
        lc.recover_async(u0, streams[: lc.MAX_CHAIN], dst, ws)
        for first in range(lc.MAX_CHAIN, chain, lc.MAX_CHAIN):
            lc.recover_async(dst, streams[first: first + lc.MAX_CHAIN], dst, ws)

    # ---- setup (untimed): a chain of `chain` snapshots tracked as Algorithm 1 does
    u0 = synth.base_state(cfg, dev, n)
    tracked, u = u0.clone(), u0.clone()
    ws = lc.alloc_workspace(n, dev)
    streams = []
    for t in range(1, chain + 1):
        u += synth.snapshot_delta(cfg, t, dev, n)
        s = lc.compress(tracked, u, nbits, workspace=ws).clone()
        streams.append(s)
        if t < chain:
            lc.recover(tracked, [s], out=tracked, workspace=ws)
    # now: tracked = u~_{chain-1}, u = u_chain; the timed compress re-creates the last stream
    sbuf = lc.alloc_stream(n, nbits, dev)
    out = torch.empty_like(u0)
    stream_bytes = [int(s.numel()) for s in streams]
    torch.cuda.synchronize()
    # size of the last snapshot under the paper's three stages (Section 4.3: E, E+P, E+P+H), as fractions of
    # the full fp32 state; the first two by the paper's size model n*ceil(log2 k) + k*32 bits
    count, _, _ = lc.debug_bins(ws)
    k_e = int((count > 0).sum())
    nsym = int(lc.stream_info(streams[-1]).nsym)
    width = lambda k: max(1, (k - 1).bit_length())
    size_model = {"occupied_buckets": k_e, "kept_symbols": nsym,
                  "E": (n * width(k_e) + 32 * k_e) / (32.0 * n), "E+P": (n * width(nsym) + 32 * nsym) / (32.0 * n),
                  "E+P+H": 8.0 * stream_bytes[-1] / (32.0 * n)}

    def step():
        lc.compress_async(tracked, u, nbits, sbuf, ws)
        recover_chain(out)

    sampler = ClockSampler(local_rank) if rank == 0 else None
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    assert lc.last_status(ws) == 0
    if sampler:
        sampler.wait_ready()

    # ---- timed region
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.mark_start()
    for k in range(args.steps):
        ev[k][0].record()
        lc.compress_async(tracked, u, nbits, sbuf, ws)
        ev[k][1].record()
        recover_chain(out)
        ev[k][2].record()
    end = torch.cuda.Event(enable_timing=True)
    end.record()
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop() if sampler else None
    total_ms = ev[0][0].elapsed_time(end)
    comp_ms = [e[0].elapsed_time(e[1]) for e in ev]
    rec_ms = [e[1].elapsed_time(e[2]) for e in ev]
    assert lc.last_status(ws) == 0
    assert torch.equal(sbuf[: stream_bytes[-1]], streams[-1]), "timed compress did not reproduce the stream"
    ms_per_step = max_over_ranks(total_ms / args.steps, dev)
    comp = statistics.mean(comp_ms)
    rec = statistics.mean(rec_ms)

    # ---- kernel breakdown of the compress call (events between its kernels; outside the timed region)
    kms = [lc.compress_timed(tracked, u, nbits, sbuf, ws) for _ in range(3)]
    stats_ms, table_ms, encode_ms = (statistics.mean(x[i] for x in kms) for i in range(3))

    # ---- single-stream recovery (the tracked-state update of Algorithm 1 step 7), outside the timed region
    k1 = []
    for _ in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        lc.recover_async(u0, streams[:1], out, ws)
        b.record()
        torch.cuda.synchronize()
        k1.append(a.elapsed_time(b))
    rec1_ms = statistics.median(k1)
    # ---- compress with the tracked state advanced in the same call (Algorithm 1 steps 4-7 fused), against the
    # two calls it replaces (compress, then single-stream recovery); outside the timed region
    cu = []
    for _ in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        lc.compress_update_async(tracked, u, nbits, sbuf, out, ws)
        b.record()
        torch.cuda.synchronize()
        cu.append(a.elapsed_time(b))
    cu_ms = statistics.median(cu)
    assert lc.last_status(ws) == 0
    assert torch.equal(sbuf[: stream_bytes[-1]], streams[-1]), "fused compress did not reproduce the stream"
    recover_chain(out)  # `out` holds the whole chain's result again

    # ---- end to end through the host-buffer entry points (pinned host memory, copies inside)
    e2e = None
    if chain <= lc.MAX_CHAIN:
        e2e_steps = max(1, min(args.steps, 3))
        h = {k: v.cpu().pin_memory() for k, v in (("tracked", tracked), ("u", u), ("u0", u0))}
        hs = [s.cpu().pin_memory() for s in streams]
        h_sbuf = torch.empty(lc.stream_bound(n, nbits), dtype=torch.uint8).pin_memory()
        h_out = torch.empty(n, dtype=torch.float32).pin_memory()
        arena = torch.empty(lc.host_arena_bytes(n, nbits, chain), dtype=torch.uint8, device=dev)
        sizes = []
        for it in range(1 + e2e_steps):
            if it == 1:
                barrier()
                torch.cuda.synchronize()
                t0 = time.perf_counter()
            sizes.append(lc.compress_host(h["tracked"], h["u"], nbits, h_sbuf, arena))
            lc.recover_host(h["u0"], hs, h_out, arena)
        torch.cuda.synchronize()
        e2e_ms = max_over_ranks(1e3 * (time.perf_counter() - t0) / e2e_steps, dev)
        assert torch.equal(h_out, out.cpu()), "host-buffer path disagrees with the device path"
        h2d = 2 * 4 * n + 4 * n + sum(stream_bytes)
        d2h = sizes[-1] + 4 * n
        e2e = {"value": aggregate_value(2 * 4 * n, world, e2e_ms), "unit": "GB/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps}
        del arena, h, hs, h_sbuf, h_out

    if rank != 0:
        return None

    peak, peak_kind = measured_peak()
    decode_launches = sum((min(lc.MAX_CHAIN, chain - f) + 3) // 4 for f in range(0, chain, lc.MAX_CHAIN))
    sbar = [b / n for b in stream_bytes]
    kernels = {
        "stats_kernel": {"ms": stats_ms, "alg_bytes": 8.0 * n},
        "encode_kernel": {"ms": encode_ms, "alg_bytes": stream_bytes[-1] + 1.0 * n},
        "decode_kernel<%d>" % min(chain, 4): {"ms": rec, "alg_bytes": 8.0 * n + sum(stream_bytes)},
    }
    dom = max(kernels, key=lambda k: kernels[k]["ms"])
    achieved = kernels[dom]["alg_bytes"] / (kernels[dom]["ms"] * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_source": peak_kind + " (STREAM-style copy)",
                "traffic": measured_traffic(dom, n),
                "per_kernel": {k: {"ms": v["ms"], "achieved_gbs": v["alg_bytes"] / (v["ms"] * 1e-3) / 1e9,
                                   "frac": v["alg_bytes"] / (v["ms"] * 1e-3) / 1e9 / peak}
                               for k, v in kernels.items()}}
    comp_alg = (8.0 * n + stream_bytes[-1]) / (comp * 1e-3) / 1e9
    rec_alg = (8.0 * n + sum(stream_bytes)) / (rec * 1e-3) / 1e9
    result = {
        "metric": METRIC, "value": aggregate_value(2 * 4 * n, world, ms_per_step), "unit": "GB/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "n": n, "nbits": nbits, "recover_chain": chain,
                   "l2": ("no flush: every vector (%.2f GB) exceeds the 126 MB L2" % (4 * n / 1e9)) if 4 * n > 126e6
                   else "vectors fit the 126 MB L2: L2-resident figures",
                   "replicas": world},
        "compress": {"ms": comp, "state_gbs": 4 * n / (comp * 1e-3) / 1e9, "alg_gbs": comp_alg,
                     "frac_of_peak": comp_alg / peak,
                     "kernels_ms": {"stats": stats_ms, "table": table_ms, "encode": encode_ms}},
        "recover": {"ms": rec, "state_gbs": 4 * n / (rec * 1e-3) / 1e9, "alg_gbs": rec_alg,
                    "frac_of_peak": rec_alg / peak},
        "recover_k1": {"ms": rec1_ms, "alg_gbs": (8.0 * n + stream_bytes[0]) / (rec1_ms * 1e-3) / 1e9,
                       "frac_of_peak": (8.0 * n + stream_bytes[0]) / (rec1_ms * 1e-3) / 1e9 / peak},
        # algorithmic bytes of the fused call: read base and cur, write the tracked state and the stream
        "compress_update": {"ms": cu_ms, "separate_calls_ms": comp + rec1_ms,
                            "alg_gbs": (12.0 * n + stream_bytes[-1]) / (cu_ms * 1e-3) / 1e9,
                            "frac_of_peak": (12.0 * n + stream_bytes[-1]) / (cu_ms * 1e-3) / 1e9 / peak},
        "ratio": {"stream": 4.0 * n / stream_bytes[-1], "bits_per_element": 8.0 * sbar[-1]},
        "size_model": size_model,
        "roofline": roofline, "clocks": clocks, "e2e": e2e,
        "gpu_launches": (3 + decode_launches) * args.steps,  # stats, table, encode + decode launches per step
    }
    if world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = time_oracle_sample(cfg, n, u0, tracked, u, streams)
    return result


def run_sweep(args):
    """Sizes x distributions x nbits: compress and single-stream recover times and the ratio, as CSV on stdout.

    Not the benchmark line: a reference table (roofline curve over n and the degenerate cases). Vectors of
    2^24 elements and fewer fit the 126 MB L2, so their figures are L2-resident.
    """
    import torch

    from paper_2009_13003_b200 import binding as lc
    from paper_2009_13003_b200 import synth

    dev = torch.device("cuda", 0)
    lc.lib()
    peak, _ = measured_peak()
    print("n,dist,nbits,compress_ms,recover_ms,compress_state_gbs,recover_state_gbs,compress_alg_frac,"
          "recover_alg_frac,ratio,bits_per_element,nsym,max_len")
    for logn in (16, 20, 24, 28, 30):
        n = 1 << logn
        base = synth.normal(n, 0.02, dev, synth.SEED0 + 5)
        ws = lc.alloc_workspace(n, dev)
        out = torch.empty_like(base)
        for dist in synth.SWEEP_DISTS:
            b = torch.zeros_like(base) if dist.startswith("one_exp") else base
            cur = b + synth.sweep_delta(dist, n, dev, synth.SEED0 + 5 + logn)
            for nbits in ((2, 3, 4, 5, 6, 8) if logn <= 24 else (2, 5, 8)):
                sbuf = lc.alloc_stream(n, nbits, dev)
                times = {"c": [], "r": []}
                for it in range(3 + 5):
                    e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
                    e[0].record()
                    lc.compress_async(b, cur, nbits, sbuf, ws)
                    e[1].record()
                    torch.cuda.synchronize()
                    if lc.last_status(ws) != 0:
                        raise SystemExit("compress failed on %s n=%d nbits=%d: status %d" % (dist, n, nbits, lc.last_status(ws)))
                    info = lc.stream_info(sbuf)
                    s = sbuf[: info.total_bytes]
                    e[1].record()
                    lc.recover_async(b, [s], out, ws)
                    e[2].record()
                    torch.cuda.synchronize()
                    if it >= 3:
                        times["r"].append(e[1].elapsed_time(e[2]))
                    e[0].record()
                    lc.compress_async(b, cur, nbits, sbuf, ws)
                    e[1].record()
                    torch.cuda.synchronize()
                    if it >= 3:
                        times["c"].append(e[0].elapsed_time(e[1]))
                assert lc.last_status(ws) == 0
                c_ms, r_ms = statistics.median(times["c"]), statistics.median(times["r"])
                sb = int(info.total_bytes)
                print("%d,%s,%d,%.4f,%.4f,%.1f,%.1f,%.3f,%.3f,%.2f,%.3f,%d,%d" % (
                    n, dist, nbits, c_ms, r_ms, 4 * n / c_ms / 1e6, 4 * n / r_ms / 1e6,
                    (8.0 * n + sb) / c_ms / 1e6 / peak, (8.0 * n + sb) / r_ms / 1e6 / peak,
                    4.0 * n / sb, 8.0 * sb / n, info.nsym, info.max_len), flush=True)
                del sbuf
            del cur
        del base, ws, out
        torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--elems", type=int, default=0, help="override the element count (profiling on small cases)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default=WORKLOAD, choices=["lenet5", "resnet18", "vgg16", "xfmr1p3b"],
                    help="synthetic config; the metric is quoted on the default")
    ap.add_argument("--sweep", action="store_true", help="print the size x distribution x nbits table (CSV) instead")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.impl == "reference":
        rank = int(os.environ.get("RANK", "0"))
        res = run_reference(args, rank)
    else:
        rank, world, local_rank = dist_setup(args.gpus)
        res = run_ours(args, rank, world, local_rank)
        import torch.distributed as dist

        if dist.is_available() and dist.is_initialized():
            dist.destroy_process_group()
    if res is not None:
        print(json.dumps(res))


if __name__ == "__main__":
    main()
