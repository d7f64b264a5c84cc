#!/usr/bin/env python
"""Benchmark of the EDEN hot path (encode + decode+mean) on B200.

One step = one pass of the whole hot path over one batch of synthetic input: eden_encode
of all n client vectors followed by eden_mean of the n messages.  The metric is GB/s of
fp32 input (n*d*4 bytes per step).  One JSON line is printed by rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5] [--impl reference]

With --gpus N > 1 (launched by torch.distributed.run) every rank runs an independent
replica of the workload (no collective on the data path; only the timing is reduced).
--impl reference times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "encode and decode+mean GB/s (fp32 in)"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
KERNEL_SOURCE = os.path.join(ROOT, "paper_2108_08842_b200", "csrc", "kernels_fast.cuh")
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_dram_traffic.txt")


def ncu_dram_bytes_per_coord():
    """DRAM bytes (read + write) per rotated coordinate and client of each kernel, from the
    ncu captures summarised under profiles/ (one client per launch there; traffic grows in
    proportion to the clients a launch covers).  Each line of the file names the kernel, the
    figure and the SHA-256 of the kernels' source file at the time of the capture: a figure
    taken on other source than the one now built is dropped, not reported."""
    import hashlib
    out = {}
    try:
        with open(KERNEL_SOURCE, "rb") as f:
            now = hashlib.sha256(f.read()).hexdigest()
        with open(TRAFFIC_FILE) as f:
            for line in f:
                line = line.split("#", 1)[0].split()
                if len(line) == 3 and line[2] == now:
                    out[line[0]] = float(line[1])
    except OSError:
        pass
    return out


def host_cores() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def config_of(work, extra=None):
    bits = sorted(set(float(b) for b in work.bits))
    cfg = {"workload": work.name, "n_clients": int(work.n), "d": int(work.d), "bits": bits,
           "packet_drop_prob": work.drop_prob, "value_law": work.description,
           "l2_policy": "inputs larger than L2 (no flush)"}
    if getattr(work, "quantiser", None):
        cfg["quantiser"] = work.quantiser
        cfg.pop("bits")
    if extra:
        cfg.update(extra)
    return cfg


# ------------------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([t.strip() for t in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 r[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------- inputs
def generate_vectors(work, out: np.ndarray, threads: int):
    def one(c):
        out[c] = work.vector(c)
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(one, range(work.n)))


# ------------------------------------------------------------------------------------- CPU oracle legs
def oracle_sample(work, clients, threads):
    """Times the oracle (as it stands) on `clients` of the workload: encode, then
    decode + mean of those clients.  Returns (seconds, bytes of fp32 input)."""
    import oracle as O
    xs = [work.vector(c) for c in clients]
    bits = [float(work.bits[c]) for c in clients]
    seeds = [int(work.seeds[c]) for c in clients]
    masks = None
    if work.drop_prob > 0:
        masks = [work.recv_mask(c, O.num_packets(O.rot_dim(work.d, bits[i]))) for i, c in enumerate(clients)]
    O.table(1)  # build tables outside the timed region
    for b in set(bits):
        O.table(O.code_width(b))
    t0 = time.perf_counter()
    enc = O.encode_all(xs, bits, seeds, threads=threads)
    mean, _ = O.mean([e["codes"] for e in enc], [float(np.float32(e["scale"])) for e in enc],
                     bits, seeds, work.d, masks, threads=threads)
    dt = time.perf_counter() - t0
    return dt, len(clients) * work.d * 4, mean


def full_config(work, n_total, world, sharded=False):
    return config_of(work, {"parallelism": ("senders split over %d ranks, one all-reduce" % world)
                            if sharded else "replicas x%d" % world,
                            "n_clients_total": int(n_total) * (1 if sharded else world)})


def run_reference(args):
    """The oracle, as it stands, on the host cores: per step `threads` clients of the workload
    in parallel, each at the workload's own dimension where the run still ends within a few
    minutes, else cut to the largest power of two that does (never below 2^22, so that the
    transform stays out of the caches and keeps most of its stages)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle as O
    from paper_2108_08842_b200 import synth
    work = synth.make(args.workload)
    cores = host_cores()
    threads = min(cores, work.n, 8)
    # seconds per coordinate and stage, from a probe of one client at 2^21 coordinates; large
    # transforms that share the memory bus run about twice as slow per butterfly as the probe
    probe = synth.make(args.workload, d=1 << 21, n=1)
    t_probe, _, _ = oracle_sample(probe, [0], 1)
    rate = 2.0 * t_probe / ((1 << 21) * 21.0)
    budget = 240.0 / (args.steps + args.warmup)
    d_s = work.d
    while d_s > (1 << 22):
        D = O.rot_dim(d_s, 1.0)
        if rate * D * np.log2(D) <= budget:
            break
        d_s = (1 << int(np.log2(d_s))) if d_s & (d_s - 1) else d_s >> 1
    sample = synth.make(args.workload, d=d_s, n=threads)
    times = []
    for step in range(args.warmup + args.steps):
        dt, nbytes, _ = oracle_sample(sample, list(range(threads)), threads)
        if step >= args.warmup:
            times.append(dt)
    ms = 1e3 * float(np.mean(times))
    value = threads * d_s * 4 / (ms * 1e-3) / 1e9
    desc = ("%d of the %d clients per step, %s coordinates each (%s), encode + decode+mean, %d threads" %
            (threads, work.n, d_s, "the workload's dimension" if d_s == work.d else
             "cut from %d to keep the run within minutes" % work.d, threads))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": full_config(work, work.n, max(1, args.gpus)),
            "sample": {"n_clients": threads, "d": int(d_s), "rotation_dim": int(O.rot_dim(d_s, 1.0))},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------- GPU arm
def run_gpu(args):
    import torch
    import torch.distributed as dist

    from paper_2108_08842_b200 import replicas
    rank, world, local_rank = replicas.rank_info()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    import __graft_entry__
    __graft_entry__.build()
    from paper_2108_08842_b200 import eden, synth

    # replicas (default): every rank has a round of its own.  --sharded: one round, its
    # senders split over the ranks, the mean finished by one all-reduce of d floats.
    work = synth.make(args.workload, d=args.d, n=args.n, seed=0 if args.sharded else rank)
    if args.bits is not None:
        work.bits = np.full(work.n, float(args.bits))
    n_total = work.n
    if args.sharded:
        if n_total < world:
            raise SystemExit("--sharded needs at least one sender per rank")
        work = work.share(replicas.shard_clients(n_total, rank, world))
    n, d = work.n, work.d
    cores = host_cores()
    dev = torch.device("cuda", local_rank)

    # inputs: generated on the host (pinned, also used by the end-to-end leg), then resident in HBM
    x_host = torch.empty((n, d), dtype=torch.float32, pin_memory=True)
    generate_vectors(work, x_host.numpy(), min(cores, 16))
    x_gpu = x_host.to(dev, non_blocking=True)
    bits, seeds = work.bits, work.seeds
    masks_np = masks_gpu = None
    if work.drop_prob > 0:
        masks_np = [work.recv_mask(c, eden.num_packets(d, float(bits[c]))) for c in range(n)]
        masks_gpu = [torch.from_numpy(m.view(np.int32)).to(dev) for m in masks_np]
    after = args.after_bits is not None
    if after:
        # Section 4.1's other order: the mask over the rotated coordinates (b < 1, no packet loss)
        if not 0.0 < args.after_bits < 1.0:
            raise SystemExit("--after-bits: a budget below one bit")
        work.bits = np.full(n, float(args.after_bits))
        work.drop_prob = 0.0
        bits = work.bits
        masks_np = masks_gpu = None
        work.quantiser = "sparsification after the rotation, b=%g" % args.after_bits
    ctx = eden.Context(local_rank, workspace_bytes_=eden.after_workspace_bytes(d, n) if after else None,
                       d_max=d, n_batch=n, host_staging=True)
    if args.sel_rounds:
        ctx.set_option(eden.OPT_SEL_ROUNDS, args.sel_rounds)
    if args.sel_inline:
        ctx.set_option(eden.OPT_SEL_AHEAD, 0)
    if args.slab_mib:
        ctx.set_option(eden.OPT_SLAB_MIB, args.slab_mib)
        ctx.set_option(eden.OPT_SLAB_STREAMS, args.slab_streams)
        ctx.set_option(eden.OPT_SLAB_SIDES, args.slab_sides)
    scales = torch.empty(n, dtype=torch.float32, device=dev)
    mean = torch.empty(d, dtype=torch.float32, device=dev)
    uniform = args.uniform_bits is not None
    if uniform:
        # Section 4.3's uniform-interval family: one index byte per rotated coordinate, and
        # the histogram an entropy coder would be built from
        delta = eden.uniform_delta(args.uniform_bits)
        if delta == 0.0:
            raise SystemExit("--uniform-bits: no supported interval width for this budget")
        deltas = np.full(n, delta)
        codes = [torch.empty(eden.uniform_index_bytes(d), dtype=torch.int8, device=dev) for _ in range(n)]
        hist = torch.empty((n, 256), dtype=torch.int32, device=dev)
        work.quantiser = "uniform intervals, b=%g, delta=%.6f" % (args.uniform_bits, delta)

        def encode_step():
            ctx.encode_uniform(x_gpu, deltas, seeds, codes, scales)
            ctx.index_histogram(codes, d, hist)

        def mean_step():
            ctx.mean_uniform(codes, scales, deltas, seeds, d, masks_gpu, mean)
    elif after:
        codes = [torch.empty(eden.after_code_bytes(d, float(b)), dtype=torch.uint8, device=dev) for b in bits]

        def encode_step():
            ctx.encode_sparsify_after(x_gpu, bits, seeds, codes, scales)

        def mean_step():
            ctx.mean_sparsify_after(codes, scales, bits, seeds, d, mean)
    else:
        codes = ctx.alloc_codes(d, bits)

        def encode_step():
            ctx.encode(x_gpu, bits, seeds, codes, scales)

        if args.sharded:
            def mean_step():
                replicas.sharded_mean(ctx, codes, scales, bits, seeds, d, n_total, masks_gpu, mean)
        else:
            def mean_step():
                ctx.mean(codes, scales, bits, seeds, d, masks_gpu, mean)
    torch.cuda.synchronize()

    def step():
        encode_step()
        mean_step()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    # Steps far below a millisecond (the paper's federated-learning sizes) are launch-latency
    # bound: bracketing each of their launches with events would itself halve the measured
    # rate.  There the K steps are timed without per-kernel events and the kernel table
    # comes from a second pass of K steps right after; everywhere else the events are
    # inside the timed region.
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record()
    step()
    p1.record()
    barrier()
    short_steps = p0.elapsed_time(p1) < 1.0 and not args.no_kernel_events
    events_in_region = not args.no_kernel_events and not short_steps

    # ---- timed region: K steps, CUDA events on the library's stream, clocks sampled meanwhile
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    launches0 = ctx.launch_count
    ctx.profile(events_in_region)
    e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    enc_ms = dec_ms = 0.0
    barrier()
    t_events = []
    for _ in range(args.steps):
        a, b, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        a.record()
        encode_step()
        b.record()
        mean_step()
        c.record()
        t_events.append((a, b, c))
    barrier()
    kernels = ctx.profile_collect() if events_in_region else {}
    ctx.profile(False)
    launches = ctx.launch_count - launches0
    if short_steps:
        ctx.profile(True)
        for _ in range(args.steps):
            step()
        barrier()
        kernels = ctx.profile_collect()
        ctx.profile(False)
    clocks = sampler.stop()
    total_ms = t_events[0][0].elapsed_time(t_events[-1][2])
    enc_ms = sum(a.elapsed_time(b) for a, b, c in t_events) / args.steps
    dec_ms = sum(b.elapsed_time(c) for a, b, c in t_events) / args.steps
    total_ms, enc_ms, dec_ms = replicas.max_over_ranks([total_ms, enc_ms, dec_ms], dev)
    ms_per_step = total_ms / args.steps
    in_bytes = n * d * 4
    if args.sharded:
        value = n_total * d * 4 / (ms_per_step * 1e-3) / 1e9
    else:
        value = replicas.whole_job_gbs(world, in_bytes, ms_per_step)

    # ---- roofline of the dominant kernel (by event time inside the timed region)
    peak, peak_kind = measured_hbm_peak()
    traffic_table = ncu_dram_bytes_per_coord()
    roofline = None
    if kernels:
        top_name = max(kernels, key=lambda k: kernels[k]["ms"])
        top = kernels[top_name]
        achieved = top["bytes"] / top["launches"] / (top["ms"] / top["launches"] * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": top_name, "achieved": achieved, "peak": peak,
                    "peak_source": "of " + peak_kind, "unit": "GB/s", "frac": achieved / peak,
                    "frac_of_nominal_8000": achieved / 8000.0,
                    "traffic": (traffic_table[top_name] * n * float(eden.rot_dim(d, float(bits[0])))
                                if top_name in traffic_table and len(set(map(float, bits))) == 1 and not after else None),
                    "traffic_source": "ncu dram__bytes_read+write, one client, scaled by clients per launch "
                                      "(profiles/ncu_dram_traffic.txt; null if the kernels changed since the capture)",
                    "algorithmic_bytes_per_launch": top["bytes"] / top["launches"],
                    "ms_per_launch": top["ms"] / top["launches"]}
    kernel_table = {k: {"launches": v["launches"], "ms": round(v["ms"], 4),
                        "share": round(v["ms"] / sum(x["ms"] for x in kernels.values()), 4),
                        "algo_GBps": round(v["bytes"] / (v["ms"] * 1e-3) / 1e9, 1) if v["ms"] > 0 else None}
                    for k, v in sorted(kernels.items(), key=lambda kv: -kv[1]["ms"])}

    # ---- accuracy of the GPU estimate against the true mean (untimed)
    true_mean = x_gpu.double().sum(dim=0) / n_total
    energy = (x_gpu.double() ** 2).sum() / n_total
    if args.sharded and world > 1:
        dist.all_reduce(true_mean)
        dist.all_reduce(energy)
    nmse = float(((mean.double() - true_mean) ** 2).sum() / energy)
    del true_mean
    status = ctx.status()

    # ---- end to end: same step through the host-buffer entry points (pinned memory),
    #      host->device and device->host copies inside the timed region
    e2e = None
    if not args.no_e2e and not uniform and not after and not args.sharded:
        codes_h = [torch.empty(eden.code_bytes(d, float(b)), dtype=torch.uint8, pin_memory=True).numpy()
                   for b in bits]
        scales_h = torch.empty(n, dtype=torch.float32, pin_memory=True).numpy()
        mean_h = torch.empty(d, dtype=torch.float32, pin_memory=True).numpy()
        xh = x_host.numpy()

        def e2e_step():
            ctx.encode_host(xh, bits, seeds, codes_h, scales_h)
            ctx.mean_host(codes_h, scales_h, bits, seeds, d, masks_np, mean_h)

        e2e_step()
        barrier()
        es = max(2, min(args.steps, 5))
        s_ev, t_ev = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s_ev.record()
        for _ in range(es):
            e2e_step()
        t_ev.record()
        barrier()
        e_ms = s_ev.elapsed_time(t_ev) / es
        e_ms = replicas.max_over_ranks([e_ms], dev)[0]
        code_bytes = sum(int(c.nbytes) for c in codes_h)
        mask_bytes = sum(int(m.nbytes) for m in masks_np) if masks_np else 0
        e2e = {"value": replicas.whole_job_gbs(world, in_bytes, e_ms), "unit": UNIT,
               "h2d_bytes_per_step": in_bytes + code_bytes + mask_bytes + 4 * n,
               "d2h_bytes_per_step": code_bytes + 4 * n + 4 * d, "ms_per_step": e_ms,
               "check": "max |mean_host - mean_dev| = %g" %
                        float(np.max(np.abs(mean_h - mean.cpu().numpy())))}

    # ---- CPU baseline: the oracle on a bounded sample of the same workload (rank 0, N = 1)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not uniform and not after and not args.sharded:
        # one wave of clients at the workload's own dimension (the same rotation the GPU is timed on)
        threads = min(cores, n, 8)
        sample = synth.make(args.workload, d=d, n=threads, seed=rank)
        if args.bits is not None:
            sample.bits = np.full(sample.n, float(args.bits))
        dt, nbytes, o_mean = oracle_sample(sample, list(range(threads)), threads)
        # the oracle's own accuracy on its sample (NMSE of its mean against the sample's true mean)
        o_true = np.zeros(d, dtype=np.float64)
        o_energy = 0.0
        for c in range(threads):
            xc = sample.vector(c).astype(np.float64)
            o_true += xc
            o_energy += float(np.dot(xc, xc))
        o_true /= threads
        o_nmse = float(np.sum((o_mean - o_true) ** 2) / (o_energy / threads))
        del o_true
        cpu = {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
               "nmse_vs_true_mean_of_sample": o_nmse,
               "sample": "%d of the %d clients of %s at its own dimension (%d coordinates, rotation of %d), "
                         "encode + decode+mean, %d threads, %.1f s" %
                         (threads, n, work.name, d, eden.rot_dim(d, float(bits[0])), threads, dt)}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "strong" if args.sharded else "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": full_config(work, n_total, world, args.sharded),
                "encode_gbs": in_bytes / (enc_ms * 1e-3) / 1e9, "decode_mean_gbs": in_bytes / (dec_ms * 1e-3) / 1e9,
                "encode_ms": enc_ms, "decode_mean_ms": dec_ms,
                "roofline": roofline, "kernels": kernel_table, "cpu_baseline": cpu, "e2e": e2e,
                "kernel_events": ("none" if args.no_kernel_events else
                                  "second pass of %d steps after the timed region (steps under 1 ms)" % args.steps
                                  if short_steps else "inside the timed region"),
                "gpu_launches": int(launches), "clocks": clocks, "nmse_vs_true_mean": nmse,
                "status_word": status}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------- the paper's sweep
def run_sweep(args):
    """The shape of the paper's encode-speed and error sweep (Section 5.2, its Figure 2 and the
    appendix on vNMSE against dimension): one LogNormal(0,1) vector, d = 2^10 ... 2^lmax by
    powers of four, b = 1..8.  Prints a markdown table: encode and decode time per vector
    (median of --steps runs after --warmup, CUDA events on the library's stream, L2 flushed
    before every run), GB/s of fp32 input, and the estimate's vNMSE beside the limit of
    Corollary 2.4, 1 / E[Q^2] - 1."""
    import math
    import torch
    import __graft_entry__
    __graft_entry__.build()
    from paper_2108_08842_b200 import eden, synth

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)       # larger than the 126 MB L2
    lmax = args.sweep_max_log2

    def limit(W):                                                       # Corollary 2.4 from the library's own table
        c, b = eden.table(W)
        edges = [-math.inf] + [float(t) for t in b] + [math.inf]
        cdf = lambda t: 0.5 * (1.0 + math.erf(t / math.sqrt(2.0)))
        eq2 = sum((cdf(edges[j + 1]) - cdf(edges[j])) * float(c[j]) ** 2 for j in range(len(c)))
        return 1.0 / eq2 - 1.0

    print("| d | b | encode us | encode GB/s | decode us | decode GB/s | vNMSE | Corollary 2.4 | ratio |")
    print("|---|---|---|---|---|---|---|---|---|")
    ctx = eden.Context(0, d_max=1 << lmax, n_batch=1)
    for L in range(10, lmax + 1, 2):
        d = 1 << L
        work = synth.make("sweep", d=d, n=1)
        x = torch.from_numpy(work.vectors()).to(dev)
        energy = float((x.double() ** 2).sum())
        for b in range(1, 9):
            bits = [float(b)]
            codes = ctx.alloc_codes(d, bits)
            scales = torch.empty(1, dtype=torch.float32, device=dev)
            out = torch.empty(d, dtype=torch.float32, device=dev)
            enc_t, dec_t = [], []
            for it in range(args.warmup + args.steps):
                flush.fill_(it & 0xFF)
                e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                e0.record()
                ctx.encode(x, bits, work.seeds, codes, scales)
                e1.record()
                flush.fill_((it + 1) & 0xFF)
                e1b = torch.cuda.Event(enable_timing=True)
                e1b.record()
                ctx.mean(codes, scales, bits, work.seeds, d, None, out)
                e2.record()
                torch.cuda.synchronize()
                if it >= args.warmup:
                    enc_t.append(e0.elapsed_time(e1) * 1e3)
                    dec_t.append(e1b.elapsed_time(e2) * 1e3)
            enc_us, dec_us = float(np.median(enc_t)), float(np.median(dec_t))
            vnmse = float(((out.double() - x[0].double()) ** 2).sum()) / energy
            lim = limit(b)
            print("| 2^%d | %d | %.1f | %.1f | %.1f | %.1f | %.5g | %.5g | %.3f |" %
                  (L, b, enc_us, 4.0 * d / enc_us / 1e3, dec_us, 4.0 * d / dec_us / 1e3, vnmse, lim, vnmse / lim))
            assert ctx.status() == 0
        del x
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5",
                    choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5", "sweep"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--n", type=int, default=None, help="override the number of clients (small profiling runs)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (small profiling runs)")
    ap.add_argument("--d", type=int, default=None, help="override the dimension (sweeps)")
    ap.add_argument("--bits", type=float, default=None, help="override every client's bit budget (sweeps)")
    ap.add_argument("--sharded", action="store_true",
                    help="one round with its senders split over the ranks and the mean finished by an "
                         "all-reduce (strong scaling) instead of independent replicas; device-resident timing only")
    ap.add_argument("--uniform-bits", type=float, default=None,
                    help="use the uniform-interval family (Section 4.3) at this entropy budget instead of the "
                         "Lloyd-Max tables; device-resident timing only (no end-to-end or CPU leg)")
    ap.add_argument("--no-kernel-events", action="store_true",
                    help="experiment: no per-kernel event bracketing in the timed region (no kernel table, no roofline)")
    ap.add_argument("--after-bits", type=float, default=None,
                    help="time Section 4.1's other order instead (eden_encode_sparsify_after / eden_mean_sparsify_after "
                         "at this budget below one bit for every sender, no packet loss); device-resident timing only")
    ap.add_argument("--sel-rounds", type=int, default=0,
                    help="experiment: form of the b < 1 mask selection (EDEN_OPT_SEL_ROUNDS; 0 keeps the default)")
    ap.add_argument("--sel-inline", action="store_true",
                    help="experiment: select the b < 1 masks in line instead of ahead on a side stream (EDEN_OPT_SEL_AHEAD 0)")
    ap.add_argument("--slab-streams", type=int, default=1)
    ap.add_argument("--slab-sides", type=int, default=3)
    ap.add_argument("--slab-mib", type=int, default=0,
                    help="experiment: launch the middle and row passes slab by slab (MiB of intermediate per slab)")
    ap.add_argument("--sweep", action="store_true",
                    help="print the LogNormal sweep table (d = 2^10 ... by powers of four, b = 1..8) instead of the JSON line")
    ap.add_argument("--sweep-max-log2", type=int, default=26)
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
