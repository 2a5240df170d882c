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


def source_digest(cu_file):
    import hashlib

    path = os.path.join(ROOT, "paper_2009_13003_b200", "csrc", cu_file)
    with open(path, "rb") as f:
        return hashlib.sha1(f.read()).hexdigest()[:12]


def measured_traffic(kernel, n):
    """DRAM bytes per launch of `kernel` from the committed ncu capture. profiles/traffic.txt holds, per kernel,
    bytes per element measured on a smaller case (every pass is a linear scan, so traffic scales with n), the
    source file of the kernel and that file's digest when the counters were taken. None if there is no entry or
    the kernel's source has changed since."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.txt")) as f:
            for line in f:
                parts = line.split()
                if len(parts) == 4 and not line.startswith("#") and parts[0] == kernel.split("<")[0]:
                    return float(parts[1]) * n if source_digest(parts[2]) == parts[3] else None
    except Exception:
        pass
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

    def __init__(self, gpu_id):
        """gpu_id: what `nvidia-smi -i` takes. Pass the device's UUID: with CUDA_VISIBLE_DEVICES set, a CUDA ordinal
        is not nvidia-smi's index, and the samples would be another GPU's."""
        import threading

        self.lines = []  # (arrival time, text)
        self.t_start = None
        self.proc = None
        self.gpu_id = str(gpu_id)
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.gpu_id, "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
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
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "gpu": self.gpu_id}
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


def gpu_uuid(cuda_ordinal):
    """'GPU-<uuid>' of a CUDA device, the form nvidia-smi -i accepts; the ordinal itself if torch cannot tell."""
    try:
        import torch

        return "GPU-" + str(torch.cuda.get_device_properties(cuda_ordinal).uuid)
    except Exception:
        return str(cuda_ordinal)


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


def host_threads():
    """Threads the oracle's chunk-parallel mode gets: the cores this process may run on."""
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except Exception:
        return max(1, os.cpu_count() or 1)


ONE_CORE_SAMPLE_ELEMS = 1 << 25  # the single-threaded figure is taken on the first 33,554,432 elements


def oracle_sample_chain(cfg, m, threads):
    """Host copy of the workload's first m elements, tracked through cfg.chain snapshots the way Algorithm 1 does,
    by the oracle. Returns (u0, tracked state before the last snapshot, last state, streams). The sample is coded on
    its own: a stream's table depends on the whole vector it codes."""
    from oracle import lc_oracle
    from paper_2009_13003_b200 import synth

    u0 = synth.base_state(cfg, "cpu", m).numpy()
    tracked, u, streams = u0.copy(), u0.copy(), []
    for t in range(1, cfg.chain + 1):
        u = u + synth.snapshot_delta(cfg, t, "cpu", m).numpy()
        s = lc_oracle.compress(tracked, u, cfg.nbits, threads=threads)
        streams.append(s)
        if t < cfg.chain:
            tracked = lc_oracle.recover(tracked, [s], threads=threads)
    return u0, tracked, u, streams


def time_oracle(cfg, u0, tracked, u, streams, threads, repeats=1):
    """Seconds of one oracle compress of the last snapshot and of one recovery of the whole chain (best of repeats)."""
    from oracle import lc_oracle

    t_c = t_r = float("inf")
    for _ in range(repeats):
        t0 = time.perf_counter()
        lc_oracle.compress(tracked, u, cfg.nbits, threads=threads)
        t1 = time.perf_counter()
        lc_oracle.recover(u0, streams, threads=threads)
        t2 = time.perf_counter()
        t_c, t_r = min(t_c, t1 - t0), min(t_r, t2 - t1)
    return t_c, t_r


def oracle_baseline(cfg, n):
    """The cpu_baseline object: the oracle, as it stands, on the first CPU_SAMPLE_ELEMS elements of the workload with
    all host cores (its chunk-parallel mode), and on a smaller sample with one core (its plain single-threaded pass).
    Same sample and same mode as the `--impl reference` arm."""
    m = min(CPU_SAMPLE_ELEMS, n)
    threads = host_threads()
    chain = oracle_sample_chain(cfg, m, threads)
    t_c, t_r = time_oracle(cfg, *chain, threads=threads)
    m1 = min(ONE_CORE_SAMPLE_ELEMS, n)
    chain1 = oracle_sample_chain(cfg, m1, threads)
    c1, r1 = time_oracle(cfg, *chain1, threads=None)
    return {"value": 2 * 4 * m / (t_c + t_r) / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
            "sample": "first %d of %d elements: 1 compress (%.2f s) + 1 recover of a chain of %d (%.2f s), oracle's "
                      "chunk-parallel mode on %d threads" % (m, n, t_c, cfg.chain, t_r, threads),
            "compress_gbs": 4 * m / t_c / 1e9, "recover_gbs": 4 * m / t_r / 1e9,
            "one_core": {"value": 2 * 4 * m1 / (c1 + r1) / 1e9, "unit": "GB/s", "cores": 1,
                         "sample": "first %d elements, plain single-threaded oracle: compress %.2f s, recover %.2f s"
                                   % (m1, c1, r1),
                         "compress_gbs": 4 * m1 / c1 / 1e9, "recover_gbs": 4 * m1 / r1 / 1e9}}


def run_reference(args, rank):
    """The CPU oracle, as it stands, timed on a bounded sample of the workload (rank 0 only): every step is one
    compress + one recovery of the chain on the first CPU_SAMPLE_ELEMS elements, with all host cores."""
    if rank != 0:
        return None
    from paper_2009_13003_b200 import synth

    cfg = synth.CONFIGS[WORKLOAD]
    m = min(CPU_SAMPLE_ELEMS, cfg.n)
    threads = host_threads()
    chain = oracle_sample_chain(cfg, m, threads)
    times = []
    for it in range(args.warmup + args.steps):
        t_c, t_r = time_oracle(cfg, *chain, threads=threads)
        if it >= args.warmup:
            times.append(t_c + t_r)
    ms = 1e3 * sum(times) / len(times)
    value = 2 * 4 * m / (ms * 1e-3) / 1e9
    sample = ("first %d of %d elements, compress + recover(chain %d) per step, oracle's chunk-parallel mode on %d "
              "threads" % (m, cfg.n, cfg.chain, threads))
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "n": cfg.n, "nbits": cfg.nbits, "recover_chain": cfg.chain,
                   "sample_elems": m},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


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
    # size of the last snapshot under the paper's three stages (Section 4.3: E, E+P, E+P+H) as fractions of the full
    # fp32 state: measured on real streams (fixed-width indices with every bucket kept; fixed-width indices after
    # promotion; Huffman-coded), and beside them the paper's size model n*ceil(log2 k) + k*32 bits
    count, _, _ = lc.debug_bins(ws)
    k_e = int((count > 0).sum())
    nsym = int(lc.stream_info(streams[-1]).nsym)
    width = lambda k: max(1, (k - 1).bit_length())
    sbuf_e = lc.alloc_stream(n, 9, dev)
    bytes_e = int(lc.compress(tracked, u, 9, stream=sbuf_e, workspace=ws, fixed=True).numel())
    bytes_ep = int(lc.compress(tracked, u, nbits, stream=sbuf_e, workspace=ws, fixed=True).numel())
    del sbuf_e
    size_model = {"occupied_buckets": k_e, "kept_symbols": nsym,
                  "E": bytes_e / (4.0 * n), "E+P": bytes_ep / (4.0 * n), "E+P+H": stream_bytes[-1] / (4.0 * n),
                  "model_E": (n * width(k_e) + 32 * k_e) / (32.0 * n),
                  "model_E+P": (n * width(nsym) + 32 * nsym) / (32.0 * n)}

    def step():
        lc.compress_async(tracked, u, nbits, sbuf, ws)
        recover_chain(out)

    sampler = ClockSampler(gpu_uuid(local_rank)) if rank == 0 else None
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
    # ---- asynchronous execution (Section 3.2): statistics pass on the stream that owns the state, table and encode
    # on a side stream, beside a synthetic "next training iteration" (bf16 matrix products on the state's stream);
    # outside the timed region. exposed = what the state's stream waits for before its next work can start.
    state_s, side_s = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ev_read = torch.cuda.Event()
    ma = torch.randn(8192, 8192, device=dev, dtype=torch.bfloat16)
    mb = torch.randn(8192, 8192, device=dev, dtype=torch.bfloat16)
    mc = torch.empty_like(ma)

    def next_iteration():
        for _ in range(3):
            torch.matmul(ma, mb, out=mc)

    asy = {"exposed": [], "overlapped": [], "serial": [], "work": []}
    for it in range(5):
        torch.cuda.synchronize()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        with torch.cuda.stream(state_s):
            e[0].record()
            lc.compress_two_streams(tracked, u, nbits, sbuf, ws, state_s, side_s, ev_read)
            e[1].record()
            next_iteration()
            e[2].record()
            state_s.wait_stream(side_s)
            e[3].record()
        torch.cuda.synchronize()
        assert lc.last_status(ws) == 0
        f = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        with torch.cuda.stream(state_s):
            f[0].record()
            lc.compress_async(tracked, u, nbits, sbuf, ws)
            f[1].record()
            next_iteration()
            f[2].record()
        torch.cuda.synchronize()
        if it >= 1:
            asy["exposed"].append(e[0].elapsed_time(e[1]))
            asy["overlapped"].append(e[0].elapsed_time(e[3]))
            asy["serial"].append(f[0].elapsed_time(f[2]))
            asy["work"].append(f[1].elapsed_time(f[2]))
    assert torch.equal(sbuf[: stream_bytes[-1]], streams[-1]), "two-stream compress did not reproduce the stream"
    asy = {k: statistics.median(v) for k, v in asy.items()}
    del ma, mb, mc
    # ---- checkpoint merging (Section 3.2): the chain as one super-step stream; outside the timed region
    merge_ms = merged_bytes = None
    if chain <= lc.MAX_CHAIN:
        mg = []
        scratch = torch.empty_like(u0)
        for _ in range(4):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            lc.merge_async(u0, streams, nbits, sbuf, scratch, ws)
            b.record()
            torch.cuda.synchronize()
            mg.append(a.elapsed_time(b))
        assert lc.last_status(ws) == 0
        merge_ms = statistics.median(mg[1:])
        merged_bytes = int(lc.stream_info(sbuf).total_bytes)
        assert torch.equal(scratch, out), "merge did not recover the chain's state"
        del scratch

    # ---- code-table caching (Section 3.2): the last snapshot compressed twice against one length cache: the first
    # call fills the row of its used-symbol count, the second takes its lengths from there; outside the timed region
    cache = lc.alloc_length_cache(dev)
    cached = {"ms": [], "hit": 0, "bytes": 0}
    for it in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        lc.compress_cached_async(tracked, u, nbits, sbuf, ws, cache)
        b.record()
        torch.cuda.synchronize()
        if it >= 1:
            cached["ms"].append(a.elapsed_time(b))
    assert lc.last_status(ws) == 0
    info_c = lc.stream_info(sbuf)
    cached = {"ms": statistics.median(cached["ms"]), "hit": int(info_c.cached_lengths),
              "bytes_vs_plain": int(info_c.total_bytes) / stream_bytes[-1]}
    del cache

    # ---- variant: bucket means as representatives (LC_OPT_MEAN_REP); outside the timed region
    mr = []
    for it in range(4):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        lc.compress_opt_async(tracked, u, nbits, sbuf, ws, lc.OPT_MEAN_REP)
        b.record()
        torch.cuda.synchronize()
        if it >= 1:
            mr.append(a.elapsed_time(b))
    assert lc.last_status(ws) == 0 and lc.stream_info(sbuf).mean_rep == 1
    mean_rep = {"ms": statistics.median(mr)}

    # ---- per-layer granularity on the workload that has layers (ResNet-18-sized: 62 segments): one stream per
    # segment against one stream for the flat vector; outside the timed region
    per_layer = None
    if cfg.name == "resnet18" and n == cfg.n:
        begin = [0]
        for size in synth.resnet18_segments():
            begin.append(begin[-1] + size)
        seg_offsets, seg_total = lc.segments_layout(begin, nbits)
        seg_streams = torch.empty(seg_total, dtype=torch.uint8, device=dev)
        seg_out = torch.empty_like(u0)
        tc, tr = [], []
        for it in range(6):
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            e[0].record()
            lc.compress_segments_async(tracked, u, begin, nbits, seg_streams, ws)
            e[1].record()
            lc.recover_segments_async(tracked, [seg_streams], begin, nbits, seg_out, ws)
            e[2].record()
            torch.cuda.synchronize()
            if it >= 2:
                tc.append(e[0].elapsed_time(e[1]))
                tr.append(e[1].elapsed_time(e[2]))
        assert lc.last_status(ws) == 0
        seg_bytes = sum(int(lc.stream_info(seg_streams[o:]).total_bytes) for o in seg_offsets[:-1])
        flat_out = lc.recover(tracked, [streams[-1]])
        flat_err = float((flat_out - u).abs().double().sum())
        del flat_out
        seg_err = float((seg_out - u).abs().double().sum())
        per_layer = {"segments": len(begin) - 1, "compress_ms": statistics.median(tc), "recover_ms": statistics.median(tr),
                     "ratio": 4.0 * n / seg_bytes, "flat_ratio": 4.0 * n / stream_bytes[-1],
                     "abs_error_vs_flat": seg_err / flat_err if flat_err else None}
        del seg_streams, seg_out

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
    nominal = 8000.0  # GB/s, the HBM3e figure the target is worded against; fractions of it beside the measured ones
    # entropy of the last stream's symbols, from the counts in its symbol table (what a Huffman code can approach)
    import numpy as np

    tab = np.frombuffer(streams[-1][64: 64 + 16 * nsym].cpu().numpy().tobytes(),
                        dtype=[("key", "<u2"), ("len", "u1"), ("pad", "u1"), ("rep", "<u4"), ("count", "<u8")])
    pr = tab["count"][tab["count"] > 0].astype(np.float64) / n
    entropy_bits = float(-(pr * np.log2(pr)).sum())
    code_bits = float((tab["count"].astype(np.float64) * tab["len"]).sum() / n)
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
                "frac_of_nominal_8tbs": achieved / nominal,
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
                     "frac_of_peak": comp_alg / peak, "frac_of_nominal_8tbs": comp_alg / nominal,
                     "kernels_ms": {"stats": stats_ms, "table": table_ms, "encode": encode_ms}},
        "recover": {"ms": rec, "state_gbs": 4 * n / (rec * 1e-3) / 1e9, "alg_gbs": rec_alg,
                    "frac_of_peak": rec_alg / peak, "frac_of_nominal_8tbs": rec_alg / nominal},
        "recover_k1": {"ms": rec1_ms, "alg_gbs": (8.0 * n + stream_bytes[0]) / (rec1_ms * 1e-3) / 1e9,
                       "frac_of_peak": (8.0 * n + stream_bytes[0]) / (rec1_ms * 1e-3) / 1e9 / peak},
        # algorithmic bytes of the fused call: read base and cur, write the tracked state and the stream
        "compress_update": {"ms": cu_ms, "separate_calls_ms": comp + rec1_ms,
                            "alg_gbs": (12.0 * n + stream_bytes[-1]) / (cu_ms * 1e-3) / 1e9,
                            "frac_of_peak": (12.0 * n + stream_bytes[-1]) / (cu_ms * 1e-3) / 1e9 / peak},
        "table_caching": cached,
        "per_layer": per_layer,
        "mean_rep": mean_rep,
        # algorithmic bytes of a merge: read base and the chain's streams, write the merged stream
        "merge": None if merge_ms is None else {
            "ms": merge_ms, "streams_in": chain, "merged_ratio": 4.0 * n / merged_bytes,
            "alg_gbs": (4.0 * n + sum(stream_bytes) + merged_bytes) / (merge_ms * 1e-3) / 1e9,
            "frac_of_peak": (4.0 * n + sum(stream_bytes) + merged_bytes) / (merge_ms * 1e-3) / 1e9 / peak},
        # lc_compress_async beside a synthetic next iteration (3 bf16 products of 8192^2 matrices on the state's
        # stream): exposed = memset + statistics pass; overlapped / serial = both finished, two streams / one
        "async": {"exposed_ms": asy["exposed"], "next_iteration_ms": asy["work"], "overlapped_ms": asy["overlapped"],
                  "serial_ms": asy["serial"]},
        "ratio": {"stream": 4.0 * n / stream_bytes[-1], "bits_per_element": 8.0 * sbar[-1],
                  "code_bits_per_element": code_bits, "entropy_bits_per_element": entropy_bits},
        "size_model": size_model,
        "roofline": roofline, "clocks": clocks, "e2e": e2e,
        # per step: stats, table, encode; per group of up to four streams a prepare and a decode kernel
        "gpu_launches": (3 + 2 * decode_launches) * args.steps,
    }
    if world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = oracle_baseline(cfg, n)
    return result


def run_sweep(args):
    """Sizes x distributions x nbits: compress and single-stream recover times and the ratio, as CSV on stdout.

    Not the benchmark line: a reference table (roofline curve over n and the degenerate cases). Vectors of
    2^24 elements and fewer fit the 126 MB L2, so their plain figures are L2-resident; for those sizes the table
    also has cold figures, taken with the L2 flushed (a 256 MB buffer written) before every timed call.
    """
    import torch

    from paper_2009_13003_b200 import binding as lc
    from paper_2009_13003_b200 import synth

    dev = torch.device("cuda", 0)
    lc.lib()
    peak, _ = measured_peak()
    print("n,dist,nbits,compress_ms,recover_ms,compress_state_gbs,recover_state_gbs,compress_alg_frac,"
          "recover_alg_frac,ratio,bits_per_element,nsym,max_len,compress_cold_ms,recover_cold_ms")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
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
                cold = {"c": [], "r": []}
                if logn <= 24:
                    for it in range(5):
                        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
                        flush.zero_()
                        e[0].record()
                        lc.compress_async(b, cur, nbits, sbuf, ws)
                        e[1].record()
                        flush.zero_()
                        e[2].record()
                        lc.recover_async(b, [s], out, ws)
                        e[3].record()
                        torch.cuda.synchronize()
                        cold["c"].append(e[0].elapsed_time(e[1]))
                        cold["r"].append(e[2].elapsed_time(e[3]))
                cc, cr = (("%.4f" % statistics.median(cold[k])) if cold[k] else "" for k in ("c", "r"))
                print("%d,%s,%d,%.4f,%.4f,%.1f,%.1f,%.3f,%.3f,%.2f,%.3f,%d,%d,%s,%s" % (
                    n, dist, nbits, c_ms, r_ms, 4 * n / c_ms / 1e6, 4 * n / r_ms / 1e6,
                    (8.0 * n + sb) / c_ms / 1e6 / peak, (8.0 * n + sb) / r_ms / 1e6 / peak,
                    4.0 * n / sb, 8.0 * sb / n, info.nsym, info.max_len, cc, cr), flush=True)
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
