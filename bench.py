#!/usr/bin/env python
"""Benchmark of the GradiVeQ hot path on B200.

One "step" = one pass of the streaming path over one batch of synthetic gradients:
fused compress + N-way compressed-domain sum (Eq. 3 + Eq. 4), then decompress + mean
(Eq. 5) and the uncompressed tails.  The metric is GB/s of fp32 gradient through that
path, N * M * 4 bytes per step.  The basis refresh (covariance + eigendecomposition) is
timed separately and reported under "refresh".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet50|large|vgg16|...]
    python bench.py --impl reference ...      # the CPU oracle on the host cores

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
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


# DRAM bytes (read + write) of one launch of the dominant kernel, from one `ncu --set full` capture per
# workload (profiles/project_sum_tc_*.md); None where no capture exists.
NCU_TRAFFIC_BYTES = {"resnet50": 1_646_136_000 + 15_988_224}


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
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

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


def sub_workload(w: W.Workload, fraction: float) -> W.Workload:
    """The first `fraction` of every layer's slices (at least one), all N nodes: a bounded sample."""
    lens = []
    for m in w.layer_len:
        S = m // w.d
        keep = max(1, int(S * fraction)) if S > 0 else 0
        lens.append(min(m, keep * w.d + (m % w.d if keep == S else 0)))
    return W.custom(w.name + "_sample", w.ident, d=w.d, k=w.k, N=w.N, L=w.L, layer_len=lens,
                    sigma_abs=w.sigma_abs, drift=w.drift)


def oracle_rate(w: W.Workload, target_s: float = 15.0, repeats: int = 1):
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
        for _ in range(repeats):
            oracle.pipeline(sw, g, Ut, mu)
        return (time.perf_counter() - t0) / repeats, sw

    frac = min(1.0, 2.0e6 / max(1, w.M))          # calibration: ~2M entries per node
    t_cal, sw = run(frac)
    scale = target_s / max(t_cal, 1e-3)
    frac2 = min(1.0, frac * scale)
    if frac2 > 1.5 * frac:
        t, sw = run(frac2)
    else:
        t = t_cal
    gbs = sw.N * sw.M * 4 / t / 1e9
    sample = (f"first {sw.S} of {w.S} slices ({sw.M} of {w.M} entries per node) x {sw.N} nodes, "
              f"compress + aggregate + decompress, {t:.2f} s")
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


def reference_arm(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    sample = ""
    cores = 1
    seconds_per_step = 120.0 / max(1, args.steps + args.warmup)   # the whole run ends in about two minutes
    for i in range(args.warmup + args.steps):
        gbs, sample, cores, t = oracle_rate(w, target_s=min(15.0, seconds_per_step))
        if i >= args.warmup:
            vals.append((gbs, t))
    v = float(np.mean([x[0] for x in vals]))
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean([x[1] for x in vals]) * 1e3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "d": w.d, "k": w.k, "N_nodes": w.N, "M": w.M},
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet50", choices=sorted(W.WORKLOADS))
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-refresh", action="store_true", help="skip the basis-refresh timing")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--qsgd", action="store_true",
                    help="also time the path with every node's compressed vectors quantized (levels = 7) before the sum")
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

    if args.impl == "reference":
        reference_arm(args, w)
        return

    from paper_1811_03617_b200 import gvq
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

    # every rank is an independent replica of the workload with its own batch (weak scaling,
    # no data-path collective): the rank enters the seed through the node index
    dev = f"cuda:{local_rank}"
    ctx = gvq.Context(w, device=local_rank)
    g_dev = [W.node_gradient(w, n, iteration=w.L, device=dev) for n in replicas.rank_node_ids(rank, w.N)]
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.to(dev), mu_t.to(dev)
    s_sum = torch.empty((ctx.S, w.k), device=dev)
    g_hat = torch.empty(w.M, device=dev)

    def step():
        ctx.compress_aggregate(g_dev, Ut, mu, s_sum)
        ctx.decompress(s_sum, Ut, mu, g_dev, w.N, g_hat)

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    K = args.steps
    # Per-kernel durations, right before the timed region: KD launches of each kernel alone, back to back between
    # two events (an event between the two launches of a step would serialise them, while the timed region lets the
    # set-up of each kernel overlap the tail of its predecessor; and a single launch between two events would
    # include the launch latency).  Inputs exceed L2 for the large workloads, so back-to-back launches stay cold.
    KD = max(3, min(K, 50))
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    ev[0].record()
    for i in range(KD):
        ctx.compress_aggregate(g_dev, Ut, mu, s_sum)
    ev[1].record()
    ev[2].record()
    for i in range(KD):
        ctx.decompress(s_sum, Ut, mu, g_dev, w.N, g_hat)
    ev[3].record()
    barrier()
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record()
    for i in range(K):
        step()
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
                step()
            torch.cuda.synchronize()
        clocks = sampler.stop()
        clocks["window"] = "timed region + untimed continuation of the same loop"
    barrier()
    k1_ms = ev[0].elapsed_time(ev[1]) / KD
    k3_ms = ev[2].elapsed_time(ev[3]) / KD
    value, ms_per_step = replicas.job_throughput(w.N * w.M * 4, total_ms / K, world, dist, dev)
    # tensor-core shapes: projection + decompression (tails inside); others launch the tail sum on its own
    try:
        ctx.set_projection_path(2)
        ctx.set_projection_path(0)
        tensor_core = True
    except gvq.GvqError:
        tensor_core = False
    launches_per_step = 2 if tensor_core else 2 + (1 if w.tail_entries > 0 else 0)

    peak, peak_kind = measured_peaks()
    # dominant kernel: the fused projection + N-sum.  Algorithmic bytes per launch: every node's
    # gradient read once (N * M * 4) -- its output (S * k * 4) is not counted.
    k1_bytes = w.N * w.M * 4
    roofline = {"bound": "hbm", "kernel": "project_sum_tc_kernel" if tensor_core else "project_sum_kernel", "achieved": k1_bytes / (k1_ms * 1e-3) / 1e9, "peak": peak,
                "peak_kind": peak_kind, "unit": "GB/s", "frac": k1_bytes / (k1_ms * 1e-3) / 1e9 / peak,
                "frac_of_datasheet_8000": k1_bytes / (k1_ms * 1e-3) / 1e9 / 8000.0,
                "traffic": NCU_TRAFFIC_BYTES.get(w.name), "algorithmic_bytes": k1_bytes, "ms": k1_ms,
                "timed_in": f"{KD} back-to-back launches of the kernel alone between two events, right before the timed region",
                "path": {"algorithmic_bytes": w.stream_bytes(), "ms": ms_per_step,
                         "frac": w.stream_bytes() / (ms_per_step * 1e-3) / 1e9 / peak,
                         "frac_of_datasheet_8000": w.stream_bytes() / (ms_per_step * 1e-3) / 1e9 / 8000.0,
                         "decompress_ms": k3_ms,
                         "decompress_note": "back-to-back launches: its 4 M-byte output stays partly in L2"}}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "d": w.d, "k": w.k, "N_nodes": w.N, "M": w.M, "S": w.S,
                       "layers": w.n_layers, "l2": "inputs_exceed_l2" if w.N * w.M * 4 > 256e6 else "l2_resident",
                       "parallelism": f"replicas{world}"},
            "gpu_launches": launches_per_step * K, "roofline": roofline}

    if rank == 0:
        line["clocks"] = clocks

    # ---- end to end through the C ABI with HOST buffers (copies inside the timed region)
    if not args.no_e2e:
        g_host = [x.cpu().pin_memory() for x in g_dev]
        out_host = torch.empty(w.M, dtype=torch.float32).pin_memory()
        ctx.allreduce_host(g_host, Ut, mu, out_host)  # warm-up, allocates the workspace
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            ctx.allreduce_host(g_host, Ut, mu, out_host)
        torch.cuda.synchronize()
        e2e_s = (time.perf_counter() - t0) / args.e2e_steps
        e2e_s = replicas.max_over_ranks(e2e_s, dist, dev)
        line["e2e"] = {"value": world * w.N * w.M * 4 / e2e_s / 1e9, "unit": UNIT, "ms_per_step": e2e_s * 1e3,
                       "h2d_bytes_per_step": w.N * w.M * 4, "d2h_bytes_per_step": w.M * 4}
        ctx.set_workspace(None)
        del g_host, out_host

    # ---- the same path with the stochastic quantizer between projection and sum (optional step; part of the
    # "large" configuration, which quantizes s)
    if args.qsgd or w.name == "large":
        levels, seed = 7, 20181103
        s_nodes = [torch.empty((ctx.S, w.k), device=dev) for _ in range(w.N)]
        q_nodes = [torch.empty((ctx.S, w.k), dtype=torch.int8, device=dev) for _ in range(w.N)]
        n_nodes = [torch.empty((ctx.S,), device=dev) for _ in range(w.N)]

        def qstep():
            ctx.compress_aggregate(g_dev, Ut, mu, s_sum, s_nodes)
            for n in range(w.N):
                ctx.quantize(s_nodes[n], levels, seed, n, q_nodes[n], n_nodes[n])
            ctx.dequantize_aggregate(q_nodes, n_nodes, levels, s_sum)
            ctx.decompress(s_sum, Ut, mu, g_dev, w.N, g_hat)

        for _ in range(3):
            qstep()
        torch.cuda.synchronize()
        qa, qb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = max(3, min(K, 20))
        qa.record()
        for _ in range(reps):
            qstep()
        qb.record()
        torch.cuda.synchronize()
        q_ms = qa.elapsed_time(qb) / reps
        line["qsgd"] = {"levels": levels, "separate_calls": {
            "ms_per_step": q_ms, "value": w.N * w.M * 4 / (q_ms * 1e-3) / 1e9, "unit": UNIT,
            "form": "projection with per-node outputs, one quantize launch per node, dequantize-and-sum",
            "gpu_launches_per_step": 3 + w.N}}

        def bstep():
            ctx.compress_aggregate(g_dev, Ut, mu, s_sum, s_nodes)
            ctx.quantize_aggregate(s_nodes, levels, seed, s_sum)
            ctx.decompress(s_sum, Ut, mu, g_dev, w.N, g_hat)

        for _ in range(3):
            bstep()
        torch.cuda.synchronize()
        qa.record()
        for _ in range(reps):
            bstep()
        qb.record()
        torch.cuda.synchronize()
        b_ms = qa.elapsed_time(qb) / reps
        line["qsgd"]["batched"] = {"ms_per_step": b_ms, "value": w.N * w.M * 4 / (b_ms * 1e-3) / 1e9, "unit": UNIT,
                                   "frac_of_hbm_peak": w.stream_bytes() / (b_ms * 1e-3) / 1e9 / peak,
                                   "form": "gvq_compress_aggregate (per-node outputs) + gvq_quantize_aggregate + gvq_decompress",
                                   "gpu_launches_per_step": 3}

        def fstep():
            ctx.compress_quantize_aggregate(g_dev, Ut, mu, levels, seed, s_sum)
            ctx.decompress(s_sum, Ut, mu, g_dev, w.N, g_hat)

        try:
            for _ in range(3):
                fstep()
            torch.cuda.synchronize()
            qa.record()
            for _ in range(reps):
                fstep()
            qb.record()
            torch.cuda.synchronize()
            f_ms = qa.elapsed_time(qb) / reps
            line["qsgd"]["one_pass"] = {"ms_per_step": f_ms, "value": w.N * w.M * 4 / (f_ms * 1e-3) / 1e9, "unit": UNIT,
                                        "frac_of_hbm_peak": w.stream_bytes() / (f_ms * 1e-3) / 1e9 / peak,
                                        "form": "gvq_compress_quantize_aggregate + gvq_decompress",
                                        "gpu_launches_per_step": 2}
        except gvq.GvqError as exc:   # shapes without a tensor-core kernel
            line["qsgd"]["one_pass"] = {"unavailable": str(exc)}
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
            part.run(g_dev[:1], args.ring, Ut, mu, g_hat)

        def ustep():      # the same arithmetic without segments: what one library all-reduce would sit between
            ctx.compress_aggregate_partial(g_dev[:1], args.ring, Ut, mu, x_all)
            ctx.decompress_exchanged(x_all, Ut, mu, g_hat)

        res = {}
        for name, fn in (("segmented", rstep), ("unsegmented", ustep)):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            ra, rb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = max(3, min(K, 50))
            ra.record()
            for _ in range(reps):
                fn()
            rb.record()
            torch.cuda.synchronize()
            res[name] = ra.elapsed_time(rb) / reps
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
            ctx.compress_aggregate_monitored(g_dev, Ut, mu, s_sum, mon)
            ctx.decompress(s_sum, Ut, mu, g_dev, w.N, g_hat)

        try:
            for _ in range(3):
                mstep()
            torch.cuda.synchronize()
            ma, mb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = max(3, min(K, 50))
            ma.record()
            for _ in range(reps):
                mstep()
            mb.record()
            torch.cuda.synchronize()
            m_ms = ma.elapsed_time(mb) / reps
            rel = (1.0 - mon[:, 1] / mon[:, 0]).flatten()
            line["monitor"] = {"ms_per_step": m_ms, "value": w.N * w.M * 4 / (m_ms * 1e-3) / 1e9, "unit": UNIT,
                               "frac_of_hbm_peak": w.stream_bytes() / (m_ms * 1e-3) / 1e9 / peak,
                               "relative_loss_min_max": [float(rel.min()), float(rel.max())],
                               "d2h_bytes_per_step": int(mon.numel() * 8)}
        except gvq.GvqError as exc:   # shapes without a fused form need the per-node outputs
            line["monitor"] = {"unavailable": str(exc)}

    # ---- basis refresh, timed on its own (rank 0 reports)
    if not args.no_refresh:
        hist = W.stored_gradients(w, device=dev)
        Ut_f = torch.empty_like(Ut); mu_f = torch.empty_like(mu)
        ev_f = torch.empty((w.n_layers, w.d), device=dev)
        ctx.fit_basis(hist, w.N, w.N, Ut_f, mu_f, ev_f)  # warm-up
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        sweeps = ctx.fit_basis(hist, w.N, w.N, Ut_f, mu_f, ev_f)
        b.record()
        torch.cuda.synchronize()
        line["refresh"] = {"ms": a.elapsed_time(b), "L": w.L, "samples": w.L * w.S, "max_sweeps": max(sweeps),
                           "hist_bytes": w.L * w.M * 4}
        # the cheap refresh: the k leading eigenpairs by subspace iteration from a pseudo-random start
        try:
            Ut_r = torch.empty_like(Ut); mu_r = torch.empty_like(mu)
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
            line["refresh_topk"] = {"ms": a.elapsed_time(b), "iters": iters, "start": "pseudo-random",
                                    "max_sin_angle_vs_full_fit": sin_max}
        except gvq.GvqError as exc:
            line["refresh_topk"] = {"unavailable": str(exc)}
        del hist

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        gbs, sample, cores, _ = oracle_rate(w)
        line["cpu_baseline"] = {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
        if "refresh" in line:
            line["refresh"]["cpu_oracle"] = oracle_fit_time(w)

    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
