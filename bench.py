#!/usr/bin/env python
"""Benchmark of the GradiVeQ hot path on B200.

One "step" = one pass of the streaming path over one batch of synthetic gradients: fused
compress + N-way compressed-domain sum (Eq. 3 + Eq. 4), then decompress + mean (Eq. 5) and
the uncompressed tails.  The metric is GB/s of fp32 gradient through that path, N * M * 4
bytes per step.

The default workload is the largest configuration ("large": 100 M entries, 32 nodes), whose
step quantizes every node's compressed vectors before the sum (one pass:
gvq_compress_quantize_aggregate + gvq_decompress); the same step without the quantizer is
reported beside it, and the ResNet-50-shaped configuration (step, basis refresh, cheap
refresh) as a nested record.  Every step record carries the driver's burst (--steps) and a
"sustained" sub-record: the same loop run for at least a second with the SM clock sampled
inside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload large|resnet50|vgg16|...]
    python bench.py --impl reference ...      # the CPU oracle on the host cores

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_1811_03617_b200 import replicas, workloads as W  # noqa: E402

METRIC = "GB/s fp32 gradient via compress+N-sum+decompress"
UNIT = "GB/s"
LEVELS, QSEED = 7, 20181103       # "4-bit": sign + 3 magnitude bits

# DRAM bytes of one launch of the projection kernel from ncu (dram__bytes_read.sum, dram__bytes_write.sum), captured
# on a reduced-N case of the workload where the full one is too large to profile: every node's gradient is read
# once, so the reads grow in proportion to the node count, while the writes (s_sum) do not depend on it.
# (workload, quantized) -> (bytes read per node, bytes written per launch); absent where no capture exists.
NCU_TRAFFIC_BYTES = {("resnet50", False): (1_646_136_000 / 16, 15_988_224),      # captured at N = 16
                     ("large", True): (1_603_001_088 / 4, 48_755_712),           # captured at N = 4
                     ("large", False): (1_602_710_016 / 4, 49_875_712)}          # captured at N = 4


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            j = json.loads(p.read_text())
            return float(j["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, period_ms: int = 100):
        self.index, self.rows, self.proc, self.period_ms = index, [], None, period_ms

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", str(self.period_ms)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for name, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def config_of(w: W.Workload, world: int, quantized: bool):
    return {"workload": w.name, "d": w.d, "k": w.k, "N_nodes": w.N, "M": w.M, "S": w.S, "layers": w.n_layers,
            "qsgd_levels": LEVELS if quantized else 0,
            "l2": "inputs_exceed_l2" if w.N * w.M * 4 > 256e6 else "l2_resident", "parallelism": f"replicas{world}"}


def sub_workload(w: W.Workload, fraction: float) -> W.Workload:
    """The first `fraction` of every layer's slices (at least one), all N nodes: a bounded sample."""
    lens = []
    for m in w.layer_len:
        S = m // w.d
        keep = max(1, int(S * fraction)) if S > 0 else 0
        lens.append(min(m, keep * w.d + (m % w.d if keep == S else 0)))
    return W.custom(w.name + "_sample", w.ident, d=w.d, k=w.k, N=w.N, L=w.L, layer_len=lens,
                    sigma_abs=w.sigma_abs, drift=w.drift)


def oracle_rate(w: W.Workload, quantized: bool, target_s: float = 15.0):
    """Times the CPU oracle (as it stands) on a bounded sample of the workload.
    Returns (GB/s of gradient, description of the sample, threads, seconds per pass)."""
    import oracle
    oracle.build()
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.numpy(), mu_t.numpy()

    def run(frac):
        sw = sub_workload(w, frac)
        g = [x.numpy() for x in W.node_gradients(sw, iteration=w.L)]
        t0 = time.perf_counter()
        if quantized:
            oracle.pipeline_quantized(sw, g, Ut, mu, LEVELS, QSEED)
        else:
            oracle.pipeline(sw, g, Ut, mu)
        return time.perf_counter() - t0, sw

    frac = min(1.0, 2.0e6 / max(1, w.M))          # calibration: ~2M entries per node
    t_cal, sw = run(frac)
    scale = target_s / max(t_cal, 1e-3)
    frac2 = min(1.0, frac * scale)
    if frac2 > 1.5 * frac:
        t, sw = run(frac2)
    else:
        t = t_cal
    gbs = sw.N * sw.M * 4 / t / 1e9
    what = "compress + quantize + dequantise-and-sum + decompress" if quantized else "compress + aggregate + decompress"
    sample = (f"first {sw.S} of {w.S} slices ({sw.M} of {w.M} entries per node) x {sw.N} nodes, {what}, {t:.2f} s")
    return gbs, sample, oracle.num_threads(), t


def oracle_fit_time(w: W.Workload, n_layers: int = 8):
    """Times the CPU oracle's basis fit (mean, covariance, fp64 Jacobi) on a bounded sample: the first layers of the
    workload, all their slices, all L stored gradients."""
    import oracle
    oracle.build()
    nl = min(n_layers, w.n_layers)
    sw = W.custom(w.name + "_fit_sample", w.ident, d=w.d, k=w.k, N=w.N, L=w.L, layer_len=w.layer_len[:nl],
                  sigma_abs=w.sigma_abs, drift=w.drift, literal_sums=w.literal_sums)
    hist = W.stored_gradients(sw).numpy()
    t0 = time.perf_counter()
    oracle.fit_basis(sw, hist, N=w.N, samples_are_sums_of=w.N)
    t = time.perf_counter() - t0
    return {"ms": t * 1e3, "cores": oracle.num_threads(),
            "sample": f"first {nl} of {w.n_layers} layers ({sw.L * sw.S} of {w.L * w.S} sample slices)"}


def reference_arm(args, w, quantized):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    world = int(os.environ.get("WORLD_SIZE", "1"))
    vals = []
    sample = ""
    cores = 1
    seconds_per_step = 120.0 / max(1, args.steps + args.warmup)   # the whole run ends in about two minutes
    if args.reference_seconds > 0:
        seconds_per_step = min(seconds_per_step, args.reference_seconds)
    for i in range(args.warmup + args.steps):
        gbs, sample, cores, t = oracle_rate(w, quantized, target_s=min(15.0, seconds_per_step))
        if i >= args.warmup:
            vals.append((gbs, t))
    v = float(np.mean([x[0] for x in vals]))
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean([x[1] for x in vals]) * 1e3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(w, world, quantized),
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def exercise_unfused(gvq, w):
    torch.cuda.set_device(0)
    ctx = gvq.Context(w, device=0)
    gen = torch.Generator(device="cuda").manual_seed(W.BASE_SEED)
    s_nodes = [torch.randn((ctx.S, w.k), device="cuda", generator=gen) for _ in range(w.N)]
    q_nodes = [torch.empty((ctx.S, w.k), dtype=torch.int8, device="cuda") for _ in range(w.N)]
    norms = [torch.empty((ctx.S,), device="cuda") for _ in range(w.N)]
    s_sum = torch.empty((ctx.S, w.k), device="cuda")
    for _ in range(2):
        ctx.aggregate(s_nodes, s_sum)
        ctx.quantize_aggregate(s_nodes, 7, W.BASE_SEED, s_sum, q_nodes, norms)
        ctx.quantize(s_nodes[0], 7, W.BASE_SEED, 0, q_nodes[0], norms[0])
        ctx.dequantize_aggregate(q_nodes, norms, 7, s_sum)
    torch.cuda.synchronize()
    print(json.dumps({"exercised": ["gvq_aggregate", "gvq_quantize_aggregate", "gvq_quantize", "gvq_dequantize_aggregate"],
                      "workload": w.name}))


def _timed(fn, reps):
    """ms per call of fn over `reps` back-to-back calls between two events on the current stream."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


def sustained(fn, ms_guess, gpu_index, seconds=1.0):
    """The same loop for at least `seconds` of device time, with the SM clock sampled inside it."""
    reps = max(10, int(math.ceil(seconds * 1e3 / max(ms_guess, 1e-3) * 1.1)))
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    sampler = ClockSampler(gpu_index, period_ms=50).start()
    time.sleep(0.05)
    ms = _timed(fn, reps)
    clocks = sampler.stop()
    return ms, reps, clocks


class StreamBench:
    """One workload's buffers and its step in both forms (with / without the quantizer)."""

    def __init__(self, gvq, w, rank, local_rank):
        self.gvq, self.w, self.dev, self.local_rank = gvq, w, f"cuda:{local_rank}", local_rank
        self.ctx = gvq.Context(w, device=local_rank)
        # every rank is an independent replica with its own batch: the rank enters the seed through the node index
        self.g = [W.node_gradient(w, n, iteration=w.L, device=self.dev) for n in replicas.rank_node_ids(rank, w.N)]
        Ut_t, mu_t = W.random_basis(w)
        self.Ut, self.mu = Ut_t.to(self.dev), mu_t.to(self.dev)
        self.s_sum = torch.empty((self.ctx.S, w.k), device=self.dev)
        self.g_hat = torch.empty(w.M, device=self.dev)
        try:
            self.ctx.set_projection_path(2)
            self.ctx.set_projection_path(0)
            self.tensor_core = True
        except gvq.GvqError:
            self.tensor_core = False
        self.launches_per_step = 2 if self.tensor_core else 2 + (1 if w.tail_entries > 0 else 0)

    def project(self, quantized):
        if quantized:
            self.ctx.compress_quantize_aggregate(self.g, self.Ut, self.mu, LEVELS, QSEED, self.s_sum)
        else:
            self.ctx.compress_aggregate(self.g, self.Ut, self.mu, self.s_sum)

    def decompress(self):
        self.ctx.decompress(self.s_sum, self.Ut, self.mu, self.g, self.w.N, self.g_hat)

    def step(self, quantized):
        self.project(quantized)
        self.decompress()

    def kernels_alone(self, quantized, reps):
        """Per-kernel durations: `reps` launches of each kernel alone, back to back between two events (an event
        between the two launches of a step would serialise them, while a step lets the set-up of each kernel
        overlap the tail of its predecessor; and a single launch between two events would include the launch
        latency).  The inputs exceed L2 for the large workloads, so back-to-back launches stay cold."""
        k1 = _timed(lambda: self.project(quantized), reps)
        k3 = _timed(self.decompress, reps)
        return k1, k3

    def record(self, quantized, ms_per_step, k1_ms, k3_ms, peak, peak_kind, reps_alone):
        w = self.w
        k1_bytes = w.N * w.M * 4
        kernel = ("project_sum_tc_kernel<%d,%s,false>" % (w.k, "true" if quantized else "false")) if self.tensor_core \
            else "project_sum_kernel"
        cap = NCU_TRAFFIC_BYTES.get((w.name, quantized))
        roofline = {"bound": "hbm", "kernel": kernel, "achieved": k1_bytes / (k1_ms * 1e-3) / 1e9, "peak": peak,
                    "peak_kind": peak_kind, "unit": "GB/s", "frac": k1_bytes / (k1_ms * 1e-3) / 1e9 / peak,
                    "frac_of_datasheet_8000": k1_bytes / (k1_ms * 1e-3) / 1e9 / 8000.0,
                    "traffic": None if cap is None else int(cap[0] * w.N + cap[1]),
                    "traffic_from": None if cap is None else "ncu capture (reads scaled by the node count)",
                    "algorithmic_bytes": k1_bytes, "ms": k1_ms,
                    "timed_in": f"{reps_alone} back-to-back launches of the kernel alone between two events",
                    "path": {"algorithmic_bytes": w.stream_bytes(), "ms": ms_per_step,
                             "frac": w.stream_bytes() / (ms_per_step * 1e-3) / 1e9 / peak,
                             "frac_of_datasheet_8000": w.stream_bytes() / (ms_per_step * 1e-3) / 1e9 / 8000.0,
                             "decompress_ms": k3_ms,
                             "decompress_note": "back-to-back launches: its 4 M-byte output stays partly in L2"}}
        return roofline

    def sustained_record(self, quantized, ms_guess, peak):
        w = self.w
        ms, reps, clocks = sustained(lambda: self.step(quantized), ms_guess, self.local_rank)
        return {"ms_per_step": ms, "steps": reps, "seconds": ms * reps * 1e-3,
                "value": w.N * w.M * 4 / (ms * 1e-3) / 1e9, "unit": UNIT,
                "path_frac": w.stream_bytes() / (ms * 1e-3) / 1e9 / peak, "clocks": clocks}


def refresh_record(gvq, sb: StreamBench):
    """Basis refresh (covariance + eigendecomposition) and the cheap refresh, timed on their own."""
    w, ctx, dev = sb.w, sb.ctx, sb.dev
    out = {}
    hist = W.stored_gradients(w, device=dev)
    Ut_f = torch.empty_like(sb.Ut); mu_f = torch.empty_like(sb.mu)
    ev_f = torch.empty((w.n_layers, w.d), device=dev)
    ctx.fit_basis(hist, w.N, w.N, Ut_f, mu_f, ev_f)  # warm-up
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    sweeps = ctx.fit_basis(hist, w.N, w.N, Ut_f, mu_f, ev_f)
    b.record()
    torch.cuda.synchronize()
    out["refresh"] = {"ms": a.elapsed_time(b), "L": w.L, "samples": w.L * w.S, "max_sweeps": max(sweeps),
                      "hist_bytes": w.L * w.M * 4}
    # the cheap refresh: the k leading eigenpairs by subspace iteration from a pseudo-random start
    try:
        Ut_r = torch.empty_like(sb.Ut); mu_r = torch.empty_like(sb.mu)
        ev_r = torch.empty((w.n_layers, w.k), device=dev); tr_r = torch.empty((w.n_layers,), device=dev)
        iters = 6
        ctx.refresh_basis(hist, w.N, w.N, Ut_r, mu_r, ev_r, tr_r, iters=iters, warm_start=False)  # warm-up
        torch.cuda.synchronize()
        a.record()
        ctx.refresh_basis(hist, w.N, w.N, Ut_r, mu_r, ev_r, tr_r, iters=iters, warm_start=False)
        b.record()
        torch.cuda.synchronize()
        # agreement with the full fit: sine of the largest principal angle between the two row spaces
        P = Ut_r.double() - (Ut_r.double() @ Ut_f.double().transpose(1, 2)) @ Ut_f.double()
        sin_max = float(torch.linalg.matrix_norm(P, ord=2).max())
        out["refresh_topk"] = {"ms": a.elapsed_time(b), "iters": iters, "start": "pseudo-random",
                               "max_sin_angle_vs_full_fit": sin_max}
    except gvq.GvqError as exc:
        out["refresh_topk"] = {"unavailable": str(exc)}
    del hist
    ctx.set_workspace(None)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", choices=sorted(W.WORKLOADS))
    ap.add_argument("--nodes", type=int, default=0, help="override the workload's node count (profiler captures of a "
                                                          "reduced case; the line then names the count it used)")
    ap.add_argument("--qsgd", action="store_true", help="quantize the compressed vectors (levels = 7) before the sum "
                                                        "in the headline step of workloads other than 'large'")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--reference-seconds", type=float, default=0.0,
                    help="with --impl reference: host seconds one step's sample is sized for (default: 120 s over "
                         "all steps, at most 15 s a step)")
    ap.add_argument("--no-refresh", action="store_true", help="skip the basis-refresh timings")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the >= 1 s loops")
    ap.add_argument("--no-nested", action="store_true", help="skip the nested ResNet-50-shaped record")
    ap.add_argument("--qsgd-forms", action="store_true",
                    help="also time the quantized step as separate calls and as three launches")
    ap.add_argument("--ring", type=int, default=0, metavar="W",
                    help="also time ONE participant's kernels of Algorithm 1 on a ring of W (one node gradient held "
                         "here, transfers left out): W segment compressions, W - 1 additions, W decompressions")
    ap.add_argument("--monitor", action="store_true",
                    help="also time the step with Eq. 7's per-layer, per-node loss sums formed inside the projection")
    ap.add_argument("--exercise-unfused", action="store_true",
                    help="no timing: call the unfused entry points (aggregate, quantize, quantize_aggregate, "
                         "dequantize_aggregate) twice on compressed vectors of the workload's shape, for a profiler")
    args = ap.parse_args()
    w = W.WORKLOADS[args.workload]()
    if args.nodes > 0:
        w.N = args.nodes

    from paper_1811_03617_b200 import gvq
    if args.impl == "reference":
        reference_arm(args, w, w.name == "large" or args.qsgd)
        return
    gvq.lib()  # fails loudly if the CUDA library is missing

    if args.exercise_unfused:
        exercise_unfused(gvq, w)
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    dev = f"cuda:{local_rank}"
    peak, peak_kind = measured_peaks()
    sb = StreamBench(gvq, w, rank, local_rank)
    ctx = sb.ctx
    quantized = (w.name == "large" or args.qsgd) and sb.tensor_core
    K, Wm = args.steps, max(args.warmup, 3)
    KD = max(3, min(K, 50))

    # ---- the headline step: per-kernel pass, then the timed region of exactly K steps
    for _ in range(Wm):
        sb.step(quantized)
    barrier()
    k1_ms, k3_ms = sb.kernels_alone(quantized, KD)
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record()
    for _ in range(K):
        sb.step(quantized)
    t_end.record()
    barrier()
    total_ms = t_begin.elapsed_time(t_end)
    clocks = None
    if rank == 0:
        # nvidia-smi delivers a sample every ~100 ms; a short timed region ends before the first one, so the
        # very same loop keeps running (untimed) until a few samples under this load exist
        t_stop = time.perf_counter() + 1.5
        while len(sampler.rows) < 4 and time.perf_counter() < t_stop:
            for _ in range(20):
                sb.step(quantized)
            torch.cuda.synchronize()
        clocks = sampler.stop()
        clocks["window"] = "timed region + untimed continuation of the same loop"
    barrier()
    value, ms_per_step = replicas.job_throughput(w.N * w.M * 4, total_ms / K, world, dist, dev)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": config_of(w, world, quantized),
            "step": ("gvq_compress_quantize_aggregate + gvq_decompress" if quantized else
                     "gvq_compress_aggregate + gvq_decompress"),
            "gpu_launches": sb.launches_per_step * K,
            "roofline": sb.record(quantized, ms_per_step, k1_ms, k3_ms, peak, peak_kind, KD)}
    if rank == 0:
        line["clocks"] = clocks
    if not args.no_sustained:
        line["sustained"] = sb.sustained_record(quantized, ms_per_step, peak)
        barrier()

    # ---- the same workload without the quantizer (when the headline step quantizes)
    if quantized:
        for _ in range(3):
            sb.step(False)
        torch.cuda.synchronize()
        u1, u3 = sb.kernels_alone(False, KD)
        u_ms = _timed(lambda: sb.step(False), K)
        rec = {"step": "gvq_compress_aggregate + gvq_decompress", "ms_per_step": u_ms,
               "value": w.N * w.M * 4 / (u_ms * 1e-3) / 1e9, "unit": UNIT, "steps": K,
               "roofline": sb.record(False, u_ms, u1, u3, peak, peak_kind, KD)}
        if not args.no_sustained:
            rec["sustained"] = sb.sustained_record(False, u_ms, peak)
        line["unquantized"] = rec
        line["qsgd"] = {"levels": LEVELS, "seed": QSEED,
                        "one_pass": {"ms_per_step": ms_per_step, "value": value, "unit": UNIT,
                                     "frac_of_hbm_peak": line["roofline"]["path"]["frac"],
                                     "form": "gvq_compress_quantize_aggregate + gvq_decompress",
                                     "gpu_launches_per_step": 2}}
        barrier()

    # ---- end to end through the C ABI with HOST buffers (copies inside the timed region)
    if not args.no_e2e:
        g_host = [x.cpu().pin_memory() for x in sb.g]
        out_host = torch.empty(w.M, dtype=torch.float32).pin_memory()
        ctx.host_prepare()
        lv = LEVELS if quantized else 0
        ctx.allreduce_host(g_host, sb.Ut, sb.mu, out_host, lv, QSEED)  # warm-up, allocates the workspace
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            ctx.allreduce_host(g_host, sb.Ut, sb.mu, out_host, lv, QSEED)
        torch.cuda.synchronize()
        e2e_s = (time.perf_counter() - t0) / args.e2e_steps
        e2e_s = replicas.max_over_ranks(e2e_s, dist, dev)
        line["e2e"] = {"value": world * w.N * w.M * 4 / e2e_s / 1e9, "unit": UNIT, "ms_per_step": e2e_s * 1e3,
                       "h2d_bytes_per_step": w.N * w.M * 4, "d2h_bytes_per_step": w.M * 4,
                       "call": "gvq_allreduce_host_quantized" if quantized else "gvq_allreduce_host",
                       "steps": args.e2e_steps}
        ctx.set_workspace(None)
        del g_host, out_host

    # ---- the quantized step in its other forms (optional)
    if args.qsgd_forms and quantized:
        s_nodes = [torch.empty((ctx.S, w.k), device=dev) for _ in range(w.N)]
        q_nodes = [torch.empty((ctx.S, w.k), dtype=torch.int8, device=dev) for _ in range(w.N)]
        n_nodes = [torch.empty((ctx.S,), device=dev) for _ in range(w.N)]

        def qstep():
            ctx.compress_aggregate(sb.g, sb.Ut, sb.mu, sb.s_sum, s_nodes)
            for n in range(w.N):
                ctx.quantize(s_nodes[n], LEVELS, QSEED, n, q_nodes[n], n_nodes[n])
            ctx.dequantize_aggregate(q_nodes, n_nodes, LEVELS, sb.s_sum)
            sb.decompress()

        def bstep():
            ctx.compress_aggregate(sb.g, sb.Ut, sb.mu, sb.s_sum, s_nodes)
            ctx.quantize_aggregate(s_nodes, LEVELS, QSEED, sb.s_sum)
            sb.decompress()

        reps = max(3, min(K, 20))
        for name, fn, form, nl in (("separate_calls", qstep, "projection with per-node outputs, one quantize launch "
                                    "per node, dequantize-and-sum", 3 + w.N),
                                   ("batched", bstep, "gvq_compress_aggregate (per-node outputs) + "
                                    "gvq_quantize_aggregate + gvq_decompress", 3)):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            ms = _timed(fn, reps)
            line["qsgd"][name] = {"ms_per_step": ms, "value": w.N * w.M * 4 / (ms * 1e-3) / 1e9, "unit": UNIT,
                                  "frac_of_hbm_peak": w.stream_bytes() / (ms * 1e-3) / 1e9 / peak, "form": form,
                                  "gpu_launches_per_step": nl}
        del s_nodes, q_nodes, n_nodes

    # ---- one participant's share of Algorithm 1 (kernels only; no link on one GPU)
    if args.ring > 0:
        from paper_1811_03617_b200 import ring as R

        class _NoLink:
            rank, world = 0, args.ring

            def exchange(self, send, recv):
                return R._Done()

        engine = R.CudaSegmentEngine(w, args.ring, local_rank)
        part = R.RingParticipant(engine, _NoLink())
        for xb in part.x + [part.r]:
            xb.zero_()
        x_all = torch.zeros(max(ctx.layout.exchange_floats(), 4), device=dev)

        def rstep():
            part.run(sb.g[:1], args.ring, sb.Ut, sb.mu, sb.g_hat)

        def ustep():      # the same arithmetic without segments: what one library all-reduce would sit between
            ctx.compress_aggregate_partial(sb.g[:1], args.ring, sb.Ut, sb.mu, x_all)
            ctx.decompress_exchanged(x_all, sb.Ut, sb.mu, sb.g_hat)

        res = {}
        reps = max(3, min(K, 50))
        for name, fn in (("segmented", rstep), ("unsegmented", ustep)):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            res[name] = _timed(fn, reps)
        # the same launches replayed from a CUDA graph: what the kernels cost without the host's launch work
        cs = torch.cuda.Stream(device=dev)
        cs.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(cs):
            rstep()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=cs):
                rstep()
            for _ in range(3):
                graph.replay()
            cs.synchronize()
            ra, rb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ra.record(cs)
            for _ in range(reps):
                graph.replay()
            rb.record(cs)
            cs.synchronize()
            res["segmented_graph"] = ra.elapsed_time(rb) / reps
        torch.cuda.current_stream().wait_stream(cs)
        for c in engine.ctx:
            if c is not None:
                c.device_status()
        line["ring_participant"] = {
            "ring_size": args.ring, "nodes_held": 1, "ms_segmented": res["segmented"], "ms_segmented_cuda_graph": res["segmented_graph"],
            "ms_unsegmented": res["unsegmented"],
            "launches_segmented": 3 * args.ring - 1, "bytes_read_plus_written": 2 * w.M * 4,
            "floats_sent_per_step": part.floats_sent, "raw_ring_floats_per_step": 2 * (args.ring - 1) * w.M // args.ring,
            "note": "kernels of one participant only; the transfers they overlap with need more than one GPU"}
        engine.close()

    # ---- the same step with the local-loss monitor (Eq. 7) inside the projection
    if args.monitor:
        mon = torch.empty((w.n_layers, 2, w.N), dtype=torch.float64, device=dev)

        def mstep():
            ctx.compress_aggregate_monitored(sb.g, sb.Ut, sb.mu, sb.s_sum, mon)
            sb.decompress()

        try:
            for _ in range(3):
                mstep()
            torch.cuda.synchronize()
            m_ms = _timed(mstep, max(3, min(K, 50)))
            rel = (1.0 - mon[:, 1] / mon[:, 0]).flatten()
            line["monitor"] = {"ms_per_step": m_ms, "value": w.N * w.M * 4 / (m_ms * 1e-3) / 1e9, "unit": UNIT,
                               "frac_of_hbm_peak": w.stream_bytes() / (m_ms * 1e-3) / 1e9 / peak,
                               "relative_loss_min_max": [float(rel.min()), float(rel.max())],
                               "d2h_bytes_per_step": int(mon.numel() * 8)}
        except gvq.GvqError as exc:   # shapes without a fused form need the per-node outputs
            line["monitor"] = {"unavailable": str(exc)}

    # ---- basis refresh, timed on its own
    if not args.no_refresh:
        line.update(refresh_record(gvq, sb))

    # the device status of everything so far: a kernel that gave up on a bounded wait would show here
    ctx.device_status()

    # ---- the ResNet-50-shaped configuration as a nested record (step, refresh, cheap refresh)
    if w.name == "large" and not args.no_nested and args.nodes == 0:
        del sb.g
        torch.cuda.empty_cache()
        w4 = W.resnet50()
        sb4 = StreamBench(gvq, w4, rank, local_rank)
        for _ in range(Wm):
            sb4.step(False)
        torch.cuda.synchronize()
        r1, r3 = sb4.kernels_alone(False, KD)
        r_ms = _timed(lambda: sb4.step(False), K)
        nested = {"config": config_of(w4, world, False), "step": "gvq_compress_aggregate + gvq_decompress",
                  "ms_per_step": r_ms, "value": w4.N * w4.M * 4 / (r_ms * 1e-3) / 1e9, "unit": UNIT, "steps": K,
                  "roofline": sb4.record(False, r_ms, r1, r3, peak, peak_kind, KD)}
        if not args.no_sustained:
            nested["sustained"] = sb4.sustained_record(False, r_ms, peak)
        if not args.no_refresh:
            nested.update(refresh_record(gvq, sb4))
            if rank == 0 and world == 1 and not args.no_cpu_baseline:
                nested["refresh"]["cpu_oracle"] = oracle_fit_time(w4)
        sb4.ctx.device_status()
        line["resnet50"] = nested

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        gbs, sample, cores, _ = oracle_rate(w, quantized)
        line["cpu_baseline"] = {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
        if "refresh" in line and w.name != "large":
            line["refresh"]["cpu_oracle"] = oracle_fit_time(w)

    # the paper's own system-level numbers, as context only (other hardware, another metric: not the target)
    line["paper_context"] = {
        "what": "GradiVeQ with ring all-reduce, ResNet-32 / CIFAR-100, 6 nodes, compression ratio 8 (Section 4)",
        "aggregation_time_per_500_iterations_s": {"uncompressed": 850, "gradiveq": 162, "ratio": 5.25,
                                                  "hardware": "CPU cluster, 2 x ten-core Xeon E5-2630 v4 per node"},
        "end_to_end_training_time_reduction": 0.46,
        "gpu_cluster": {"speedup_vs_uncompressed": 4.0, "speedup_vs_4bit_qsgd": 1.40, "hardware": "one Tesla K80 per node"},
        "kernel_level_numbers_in_the_paper": None}

    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
