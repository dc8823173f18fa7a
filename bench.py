#!/usr/bin/env python
"""Benchmark of the masked conv-GEMM path on synthetic layer stacks.

One step = one pass of the whole path (mask compaction, implicit-im2col gather, tensor-core
GEMM on the kept rows, bias+ReLU scatter epilogue with zero fill) over every layer of the
workload, through the C-ABI library.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 3] [--impl ours|reference]

With N > 1 (launched by torch.distributed.run) every rank runs its own replica of the
batch (lowered rows are independent: the batch is split across GPUs, there is no collective
on the data path); the timed region is bracketed by barriers and the maximum over ranks is
reported.  `--impl reference` times the CPU oracle instead (rank 0 only).
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "masked conv-GEMM actual TFLOP/s"
RECOMPACT_FLAG = 2          # ASX_RECOMPACT: every step rebuilds the kept-row list (S1) from the mask
L2_BYTES = 126 * 1024 * 1024


# DRAM traffic of the fused kernels from one ncu capture of the default workload (ResNet-18 stack, batch 64):
# dram__bytes_read.sum + dram__bytes_write.sum averaged over the 20 fused-kernel launches of a step
# (12.79 MB read + 2.35 MB written; ncu flushes the caches before every captured launch, so reads are
# cold-cache and most of a launch's output is still in L2 when its counters stop).  The figure belongs to
# the kernel sources whose digest is recorded with it; with any other sources the bench reports null.
NCU_TRAFFIC = {"workload_config": 3, "bytes_per_launch": 15.15e6,
               "csrc_sha256": "31c31102a1af22b7012d9a7e070229ec88cbaf102c67d75daddabe819296c3ee"}


def csrc_digest() -> str:
    """Digest of the sources the fused kernel is compiled from."""
    import hashlib
    h = hashlib.sha256()
    for name in ("asx_internal.h", "conv_common.cuh", "masked_conv_sm100.cu", "masked_conv_patch_sm100.cu", "ptx_sm100.cuh"):
        h.update(name.encode())
        with open(os.path.join(ROOT, "paper_2309_06626_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def measured_traffic(cfg: int, only: str):
    if cfg != NCU_TRAFFIC["workload_config"] or only or csrc_digest() != NCU_TRAFFIC["csrc_sha256"]:
        return None
    return NCU_TRAFFIC["bytes_per_launch"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def workload_name(cfg: int) -> str:
    return {1: "single 3x3 conv 56x56x64->64 bs1, 50% rows dropped, block 1",
            2: "ResNet-18 conv stack 224x224 bs1, 30% row sparsity, block 1",
            3: "ResNet-18 conv stack 224x224 bs64, 50% row sparsity, block 4",
            4: "CSP-Darknet-like conv stack 640x640 bs16, 40% row sparsity, block 2",
            5: "3x3 conv 28x28x256->256 bs128 sparsity/block sweep"}[cfg]


# --------------------------------------------------------------------------------------------
# clocks
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.thread, self.idx = [], None, None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.idx)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self, t0: float, t1: float):
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [r for r in self.rows if t0 <= r[0] <= t1] or self.rows
        for _, line in rows:
            f = [c.strip() for c in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------------------------
# the CPU oracle leg (cpu_baseline and --impl reference)
def oracle_problems(cfg: int):
    probs = []
    for spec in wl.config(cfg):
        s1 = wl.with_batch(spec, 1)          # the first image of the batch; same seeds
        probs.append((s1, wl.make_x(s1), wl.make_w(s1), wl.make_b(s1), wl.make_layer_mask(s1)))
    return probs


def oracle_pass(probs, frac: float):
    """Runs the oracle on the first ceil(frac*P) output positions of image 0 of every layer.
    Returns (seconds, kept FLOPs)."""
    import oracle
    flops, t0 = 0, time.perf_counter()
    for s, x, w, b, m in probs:
        n = max(1, int(np.ceil(frac * s.P)))
        sel = np.arange(n, dtype=np.int64)
        oracle.masked_conv_rows(x, w, b, m, s.stride, s.pad, True, sel)
        flops += 2 * int(m[:n].sum()) * s.K * s.N
    return time.perf_counter() - t0, flops


def cpu_baseline(cfg: int, budget_s: float = 12.0):
    """The oracle as it stands on the host cores: at the workload's sparsity (it skips dropped rows, whose
    value is zero by definition) and, on a smaller budget, with all-ones masks (sparsity 0)."""
    import oracle
    oracle.build()
    probs = oracle_problems(cfg)
    t_cal, _ = oracle_pass(probs, 1.0)
    reps = int(max(1, min(64, budget_s / max(t_cal, 1e-3))))
    t, f = 0.0, 0
    for _ in range(reps):
        dt, df = oracle_pass(probs, 1.0)
        t += dt; f += df
    probs0 = [(s1, x, w, b, np.ones_like(m)) for s1, x, w, b, m in probs]
    t0c, _ = oracle_pass(probs0, 1.0)
    reps0 = int(max(1, min(32, 0.5 * budget_s / max(t0c, 1e-3))))
    t0, f0 = 0.0, 0
    for _ in range(reps0):
        dt, df = oracle_pass(probs0, 1.0)
        t0 += dt; f0 += df
    return {"value": f / t / 1e12, "unit": "TFLOP/s", "cores": oracle.n_threads(), "kind": "oracle",
            "sample": f"image 0 of every layer of the workload, all output rows, {reps} passes "
                      f"({f / 1e9:.1f} GFLOP kept, {t:.1f} s)",
            "value_sparsity0": f0 / t0 / 1e12,
            "sample_sparsity0": f"the same with all-ones masks, {reps0} passes ({f0 / 1e9:.1f} GFLOP, {t0:.1f} s)",
            "speedup_vs_sparsity0": (t0 / reps0) / (t / reps)}


def cpu_alg2_baseline(cfg: int, budget_s: float = 8.0):
    """The paper's own three CPU stages in fp32 (indirection buffer over kept positions, dense product
    on the reduced range, reverse in-place expansion; oracle/alg2_fp32.c), timed on the same sample as
    the oracle: a second reported baseline, closer to what the paper ran on its CPU."""
    import oracle
    oracle.build()
    probs = [(s, oracle.bf16_round(x), oracle.bf16_round(w), b, m) for s, x, w, b, m in oracle_problems(cfg)]

    def one_pass():
        t0, f = time.perf_counter(), 0
        for s, x, w, b, m in probs:
            oracle.alg2_fp32(x, w, b, m, s.stride, s.pad, True)
            f += 2 * int(m.sum()) * s.K * s.N
        return time.perf_counter() - t0, f
    t_cal, _ = one_pass()
    reps = int(max(1, min(64, budget_s / max(t_cal, 1e-3))))
    t, f = 0.0, 0
    for _ in range(reps):
        dt, df = one_pass()
        t += dt; f += df
    return {"value": f / t / 1e12, "unit": "TFLOP/s", "cores": oracle.n_threads(), "kind": "paper stages, fp32",
            "sample": f"image 0 of every layer of the workload, {reps} passes ({f / 1e9:.1f} GFLOP kept, {t:.1f} s)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    oracle.build()
    probs = oracle_problems(args.config)
    t_cal, _ = oracle_pass(probs, 1.0)
    target = 120.0 / max(1, args.steps + args.warmup)
    frac = min(1.0, target / max(t_cal, 1e-3))
    for _ in range(args.warmup):
        oracle_pass(probs, frac)
    t, f = 0.0, 0
    for _ in range(args.steps):
        dt, df = oracle_pass(probs, frac)
        t += dt; f += df
    val = f / t / 1e12
    sample = (f"per step: the first {frac * 100:.2f}% of the output rows of image 0 of every layer "
              f"({f / args.steps / 1e9:.3f} GFLOP kept)")
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": workload_name(args.config)},
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": oracle.n_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)
    return 0


# --------------------------------------------------------------------------------------------
# the GPU leg
class DeviceLayer:
    def __init__(self, spec, torch, asx, dense_twin=True, score=None, f32=False):
        self.spec = spec
        dt = torch.float32 if f32 else torch.bfloat16          # storage type of x, w and y
        x, w, b = wl.make_x(spec), wl.make_w(spec), wl.make_b(spec)
        # masks: seeded blocks of rows (default), or the paper's generator from one input-resolution score
        self.mask = (wl.make_layer_mask(spec) if score is None
                     else asx.mask_from_scores(score, spec.Ho, spec.Wo, spec.sparsity_pct / 100.0))
        self.x_host = torch.from_numpy(x).to(dt).pin_memory()
        self.x = self.x_host.cuda()
        self.w = torch.from_numpy(w).to(dt).cuda()
        self.b = torch.from_numpy(b).cuda()
        self.y = torch.empty((spec.Nb, spec.Ho, spec.Wo, spec.C_out), dtype=dt, device="cuda")
        self.y_host = torch.empty(self.y.shape, dtype=dt).pin_memory()
        self.layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, spec.kh, spec.kw, spec.stride, spec.pad)
        self.layer.set_mask(self.mask)
        self.dense = None
        if dense_twin:
            self.dense = asx.MaskedConvLayer(spec.C_in, spec.C_out, spec.kh, spec.kw, spec.stride, spec.pad)
            self.dense.set_mask(np.ones(spec.P, np.uint8))
        kept_rows = int(self.mask.sum()) * spec.Nb
        self.kept_rows = kept_rows
        self.flops = wl.algorithmic_flops(spec, kept_rows)
        self.flops_dense = wl.algorithmic_flops(spec, spec.M)
        self.bytes = wl.algorithmic_bytes(spec, self.mask, 4 if f32 else 2)
        self.ptrs = (self.x.data_ptr(), spec.Nb, spec.H, spec.W, self.w.data_ptr(), self.b.data_ptr(),
                     self.y.data_ptr())
        # fused kernel (it rebuilds the kept-row list itself for masks of up to 32768 rows, else the two
        # compaction passes run first), plus the staging of x and w when C_in is not a multiple of 8 (4 in fp32):
        # one launch in the 2x2-block form of a stride-2 first layer, else one padding launch each
        sh = spec.pad & 1
        blocks2x2 = (not f32 and spec.C_in <= 4 and spec.stride == 2 and spec.W % 2 == 0 and spec.H % 2 == 0
                     and (spec.kw + sh + 1) // 2 == 4 and spec.kh + sh <= 32)
        staging = 1 if blocks2x2 else (2 if spec.C_in % (4 if f32 else 8) else 0)
        self.launches = 1 + (0 if self.mask.size <= 32768 else 2) + staging

    def step(self, st, flags, layer=None, recompact=True):
        L = layer or self.layer
        rc = L.run_raw(*self.ptrs, flags | (RECOMPACT_FLAG if recompact else 0), st)
        if rc:
            raise RuntimeError(f"asx call failed with status {rc} on {self.spec.name}")


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2309_06626_b200 as asx
    from paper_2309_06626_b200 import build as asx_build
    from paper_2309_06626_b200.dist_util import max_over_ranks, shard_batch, whole_job_rate

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        asx_build.build()
    if world > 1:
        dist.barrier()
    asx.lib()
    peaks = load_peaks()
    st_obj = torch.cuda.current_stream()
    st = int(st_obj.cuda_stream)
    f32 = args.dtype == "f32"
    # the activation (and storage) flags of every asx_run below
    RELU = (asx.ACT_SILU if args.act == "silu" else asx.ACT_RELU) | (asx.F32 if f32 else 0)
    if f32:
        # fp32 storage, TF32 contraction: no measured TF32 peak exists, so the bf16 figures are scaled by
        # the nominal dense ratio of the two tensor-core rates (1.1 / 2.25 PFLOP/s)
        ratio = 1.1 / 2.25
        peaks = dict(peaks, bf16_tflops=peaks["bf16_tflops"] * ratio,
                     bf16_tflops_sustained=peaks["bf16_tflops_sustained"] * ratio)

    specs = wl.config(args.config)
    if args.only:
        specs = [s for s in specs if any(s.name.startswith(p) for p in args.only.split(","))]
        if not specs:
            raise SystemExit(f"--only {args.only}: no such layer")
    strong = (args.scaling == "strong" and world > 1)
    if strong:
        # the batch of every layer is split across the ranks (images [lo, hi) of each); the masks are
        # shared by the images, so every rank keeps the whole mask and kept-row list
        shards = [shard_batch(s.Nb, rank, world) for s in specs]
        if any(hi <= lo for lo, hi in shards):
            raise SystemExit("--scaling strong needs at least one image per rank in every layer")
        specs = [wl.with_batch(s, hi - lo) for s, (lo, hi) in zip(specs, shards)]
    score = None
    if args.mask == "scores":
        score = wl.make_score(args.config, max(s.H for s in specs), max(s.W for s in specs))
    layers = [DeviceLayer(s, torch, asx, dense_twin=(args.config != 5), score=score, f32=f32) for s in specs]
    torch.cuda.synchronize()
    footprint = sum(L.x.numel() * 2 + L.y.numel() * 2 + L.w.numel() * 2 for L in layers)

    def one_step(dense=False, recompact=True, stream=None):
        for L in layers:
            L.step(stream if stream is not None else st, RELU, L.dense if (dense and L.dense is not None) else None, recompact)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # The 1x1 projection of a down-sampling block reads the block's input, like the block's first 3x3
    # convolution, and meets the main branch only at the block's residual add: in the network the two are
    # independent.  With fork_proj the captured graph runs it on a side branch beside conv1 -> conv2 of its
    # block.  (Layers that depend on each other in the network are never overlapped.)
    fork = (not args.no_fork_proj) and any(L.spec.name.endswith(".proj") for L in layers)

    def capture(dense=False, recompact=True, chained=False):
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        with torch.cuda.graph(g):
            main = torch.cuda.current_stream()
            cst = int(main.cuda_stream)
            joined = True
            for i, L in enumerate(layers):
                name = L.spec.name
                lay = L.dense if (dense and L.dense is not None) else L.layer
                fl = RELU | (RECOMPACT_FLAG if recompact else 0)
                if fork and name.endswith(".0.conv1") and any(M.spec.name == name[:-5] + "proj" for M in layers):
                    P = next(M for M in layers if M.spec.name == name[:-5] + "proj")
                    side.wait_stream(main)
                    with torch.cuda.stream(side):
                        play = P.dense if (dense and P.dense is not None) else P.layer
                        rc = play.run_raw(*(P.ptrs_chained if chained else P.ptrs), fl, int(side.cuda_stream))
                        if rc:
                            raise RuntimeError(f"asx call failed with status {rc} during capture")
                    joined = False
                if fork and name.endswith(".proj"):
                    if not joined:
                        main.wait_stream(side)           # the residual add of the block would sit here
                        joined = True
                    continue
                rc = lay.run_raw(*(L.ptrs_chained if chained else L.ptrs), fl, cst)
                if rc:
                    raise RuntimeError(f"asx call failed with status {rc} during capture ({name})")
            if not joined:
                main.wait_stream(side)
        return g

    def time_replays(g, n):
        """Mean device time per replay of n back-to-back replays, and median / min of n2 single replays."""
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(st_obj)
        for _ in range(n):
            g.replay()
        a1.record(st_obj)
        torch.cuda.synchronize()
        mean = a0.elapsed_time(a1) / n
        n2 = max(3, min(n, 200))
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n2)]
        for x0, x1 in evs:
            x0.record(st_obj)
            g.replay()
            x1.record(st_obj)
        torch.cuda.synchronize()
        singles = sorted(x0.elapsed_time(x1) for x0, x1 in evs)
        return mean, statistics.median(singles), singles[0]

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        one_step()
    barrier()

    # ---- one step captured in a CUDA graph (the layer stack is launch-bound otherwise)
    graph = None
    if not args.no_graph:
        graph = capture()
        for _ in range(3):
            graph.replay()
        barrier()

    # ---- timed region: K steps, device time by CUDA events on the launching stream
    K = args.steps
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    e0.record(st_obj)
    for k in range(K):
        if graph is not None:
            graph.replay()
        else:
            one_step()
    e1.record(st_obj)
    barrier()
    t_wall1 = time.time()
    ms_total = max_over_ranks(e0.elapsed_time(e1), device="cuda")
    ms_step = ms_total / K
    ms_median = ms_min = None
    if graph is not None:
        _, ms_median, ms_min = time_replays(graph, min(K, 200))

    # ---- per-layer time in the step's own regime: the replay time of the captured prefix [0..i] minus that
    # of [0..i-1] (in-line order, no graph branch), i.e. what layer i adds to a graph-replayed step with
    # its set-up overlapping the previous kernel's tail as in the timed region
    in_step_ms = None
    if graph is not None and not args.no_marginal:
        in_step_ms, prev = [], 0.0
        for i in range(1, len(layers) + 1):
            pg = torch.cuda.CUDAGraph()
            with torch.cuda.graph(pg):
                cst = int(torch.cuda.current_stream().cuda_stream)
                for L in layers[:i]:
                    rc = L.layer.run_raw(*L.ptrs, RELU | RECOMPACT_FLAG, cst)
                    if rc:
                        raise RuntimeError(f"asx call failed with status {rc} during capture")
            t = time_replays(pg, 50)[0]
            in_step_ms.append(t - prev)
            prev = t
            del pg

    # ---- a second view: every launch of the fused kernel alone between an event pair (a spin kernel is
    # queued first so that the host runs ahead).  These per-launch times are SERIALISED: the event pair
    # keeps a launch from overlapping its neighbours, which the graph replay above allows (programmatic
    # dependent launch), so they add up to more than a step.  They rank the layers; the step time is above.
    n_probe = max(3, min(K, 30))
    probe_events = []
    for k in range(n_probe):
        torch.cuda._sleep(6_000_000)
        row = []
        for L in layers:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(st_obj)
            rc = L.layer.run_raw(*L.ptrs, RELU | RECOMPACT_FLAG, st)
            b.record(st_obj)
            if rc:
                raise RuntimeError(f"asx call failed with status {rc}")
            row.append((a, b))
        probe_events.append(row)
    barrier()
    for L in layers:
        if L.layer.device_status() != 0:
            raise RuntimeError("a kernel reported a bounded-wait timeout")
    forms = [L.layer.last_run_form() for L in layers]

    flops_step = sum(L.flops for L in layers)
    dense_flops_step = sum(L.flops_dense for L in layers)
    if strong:     # the ranks' shards differ by at most one image: sum them instead of multiplying
        tot = torch.tensor([float(flops_step), float(dense_flops_step)], dtype=torch.float64, device="cuda")
        dist.all_reduce(tot)
        job_flops, job_dense_flops = float(tot[0].item()), float(tot[1].item())
    else:
        job_flops, job_dense_flops = world * flops_step, world * dense_flops_step
    value = (job_flops / (ms_step * 1e-3) if strong else whole_job_rate(flops_step, ms_step, world)) / 1e12

    per_layer_ms = [statistics.median(row[i][0].elapsed_time(row[i][1]) for row in probe_events)
                    for i in range(len(layers))]
    serial_ms = sum(per_layer_ms)
    # Peak: the burst figure for a timed region of under a second (the clocks stay at their maximum),
    # the sustained one above; both fractions are reported.
    burst = (ms_total < 1000.0)
    peak_tf = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
    achieved = flops_step / (ms_step * 1e-3) / 1e12
    roofs = [max(L.flops / (peak_tf * 1e12), L.bytes / (peaks["hbm_gbs"] * 1e9)) * 1e3 for L in layers]
    roof_ms = sum(roofs)
    tensor_bound_layers = sum(1 for L in layers if L.flops / (peak_tf * 1e12) >= L.bytes / (peaks["hbm_gbs"] * 1e9))

    # ---- the same kernels at sparsity 0 (all-ones masks), the stored list without the per-step compaction,
    # and cuDNN dense convolution: each captured in a CUDA graph and timed like the headline
    K0 = max(3, min(K, 200))
    ms_dense = ms_frozen = ms_chained = None
    if graph is not None and args.config != 5:
        for _ in range(3):
            one_step(dense=True)
        torch.cuda.synchronize()
        ms_dense = time_replays(capture(dense=True), K0)[0]
    if graph is not None:
        one_step(recompact=False)
        torch.cuda.synchronize()
        ms_frozen = time_replays(capture(recompact=False), K0)[0]
    # ---- the step with every layer reading, where the shapes allow it, the output buffer of the layer that
    # feeds it in the network (the previous layer of the list; for a block's projection the block's input)
    # instead of a buffer of its own: the inputs are then warm in L2 as they would be in the network.  A side
    # figure: the headline keeps the cold, independent buffers.
    chained_layers = 0
    if graph is not None and args.config != 5:
        last_main, block_in = None, None
        for L in layers:
            src = None
            if L.spec.name.endswith(".proj"):
                src = block_in
            else:
                src = last_main
                if L.spec.name.endswith(".0.conv1"):
                    block_in = last_main
                last_main = L
            L.ptrs_chained = L.ptrs
            if src is not None and tuple(src.y.shape) == tuple(L.x.shape) and src.y.dtype == L.x.dtype:
                L.ptrs_chained = (src.y.data_ptr(),) + tuple(L.ptrs[1:])
                chained_layers += 1
        if chained_layers:
            for L in layers:                 # once outside the capture: a new input pointer re-encodes tensor maps
                rc = L.layer.run_raw(*L.ptrs_chained, RELU | RECOMPACT_FLAG, st)
                if rc:
                    raise RuntimeError(f"asx call failed with status {rc} on {L.spec.name} (chained inputs)")
            torch.cuda.synchronize()
            ms_chained = time_replays(capture(chained=True), K0)[0]

    cudnn_ms = None
    if rank == 0 and not args.no_cudnn:
        import torch.nn.functional as F
        views = [(L.x.permute(0, 3, 1, 2), L.w.permute(0, 3, 1, 2), L.b.to(L.x.dtype), L.spec) for L in layers]

        def cudnn_step():
            for xv, wv, bv, s in views:
                F.conv2d(xv, wv, bv, stride=s.stride, padding=s.pad)
        for _ in range(3):
            cudnn_step()
        torch.cuda.synchronize()
        try:
            cg = torch.cuda.CUDAGraph()
            with torch.cuda.graph(cg):
                cudnn_step()
            cudnn_ms = time_replays(cg, K0)[0]
        except Exception:                      # a cuDNN algorithm that cannot be captured: eager timing
            torch.cuda.synchronize()
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record(st_obj)
            for _ in range(K0):
                cudnn_step()
            c1.record(st_obj)
            torch.cuda.synchronize()
            cudnn_ms = c0.elapsed_time(c1) / K0

    # ---- end to end: host buffers, H2D of every layer's input and D2H of every output inside the timed region
    Ke = max(3, min(K, 10))
    h2d = sum(L.x_host.numel() * L.x_host.element_size() for L in layers)
    d2h = sum(L.y_host.numel() * L.y_host.element_size() for L in layers)

    # Copies in, kernels and copies out run on three streams, ordered per layer by events, so that the
    # two directions of the host link and the kernels overlap across layers and steps; every step still
    # copies every layer's input from pinned host memory and every output back.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in layers]
    ev_done = [torch.cuda.Event() for _ in layers]
    ev_out = [torch.cuda.Event() for _ in layers]

    def e2e_step():
        for i, L in enumerate(layers):
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_done[i])             # the previous step's kernel has read x
                L.x.copy_(L.x_host, non_blocking=True)
                ev_in[i].record(s_in)
            st_obj.wait_event(ev_in[i])
            st_obj.wait_event(ev_out[i])                # the previous step's copy of y has left
            L.step(st, RELU)
            ev_done[i].record(st_obj)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[i])
                L.y_host.copy_(L.y, non_blocking=True)
                ev_out[i].record(s_out)
    e2e_step()
    barrier()
    tw0 = time.perf_counter()
    for _ in range(Ke):
        e2e_step()
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - tw0) * 1e3 / Ke
    e2e_ms = max_over_ranks(e2e_ms, device="cuda")
    e2e_val = job_flops / (e2e_ms * 1e-3) / 1e12
    t_gpu_end = time.time()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0
    sampler.stop()
    clocks = sampler.summary(t_wall0, t_wall1)
    clocks["window"] = "the timed region"
    if clocks["samples"] < 2:       # a timed region shorter than the sampling period
        clocks = sampler.summary(0, t_gpu_end)
        clocks["window"] = "the whole GPU phase of this run (the timed region was shorter than two sampling periods of 50 ms)"
    cpu = None if args.no_cpu_baseline else cpu_baseline(args.config)
    cpu_alg2 = None if args.no_cpu_baseline else cpu_alg2_baseline(args.config)

    # ---- S1 alone on a mask large enough to be HBM-bound (the per-layer masks are a few KB)
    s1 = None
    if not args.no_s1:
        rows = 1 << 27
        gen = torch.Generator(device="cuda"); gen.manual_seed(wl.BASE_SEED)
        big = (torch.rand(rows, device="cuda", generator=gen) < 0.5).to(torch.uint8)
        kept_big = torch.empty(rows, dtype=torch.int32, device="cuda")
        cnt_big = torch.empty(1, dtype=torch.int32, device="cuda")
        nb = asx.lib().asx_compact_scratch_bytes(rows)
        scr = torch.empty((nb + 7) // 8, dtype=torch.int64, device="cuda")

        def s1_call():
            rc = asx.lib().asx_compact(big.data_ptr(), rows, kept_big.data_ptr(), cnt_big.data_ptr(),
                                       scr.data_ptr(), scr.numel() * 8, st)
            if rc:
                raise RuntimeError(f"asx_compact failed with status {rc}")
        for _ in range(3):
            s1_call()
        torch.cuda.synchronize()
        if asx.lib().asx_compact_status(scr.data_ptr(), st) != 0:
            raise RuntimeError("compaction reported a bounded-wait timeout")
        s0, s1e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record(st_obj)
        for _ in range(10):
            s1_call()
        s1e.record(st_obj)
        torch.cuda.synchronize()
        ms = s0.elapsed_time(s1e) / 10
        kept_n = int(cnt_big.item())
        gbs = (rows + 4 * kept_n) / (ms * 1e-3) / 1e9
        s1 = {"rows": rows, "kept": kept_n, "ms": ms, "gbs": gbs, "bytes": "rows + 4*kept (mask read, list written)",
              "frac_of_hbm_peak": gbs / peaks["hbm_gbs"], "peak_gbs": peaks["hbm_gbs"]}
        del big, kept_big, scr

    # ---- the data-dependent mask kernel alone (HBM-bound: rows*C*2 bytes read, rows written)
    mfa = None
    if not args.no_s1:
        rows_a, C_a = 1 << 22, 64                                   # 512 MB of bf16 activations, larger than L2
        act = torch.randn((rows_a, C_a), device="cuda", dtype=torch.bfloat16).relu_()
        act[::3] = 0
        mask_a = torch.empty(rows_a, dtype=torch.uint8, device="cuda")

        def mfa_call():
            rc = asx.lib().asx_mask_from_activation(act.data_ptr(), rows_a, C_a, mask_a.data_ptr(), st)
            if rc:
                raise RuntimeError(f"asx_mask_from_activation failed with status {rc}")
        for _ in range(3):
            mfa_call()
        torch.cuda.synchronize()
        m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        m0.record(st_obj)
        for _ in range(10):
            mfa_call()
        m1.record(st_obj)
        torch.cuda.synchronize()
        ms_a = m0.elapsed_time(m1) / 10
        gbs_a = (rows_a * C_a * 2 + rows_a) / (ms_a * 1e-3) / 1e9
        mfa = {"rows": rows_a, "C": C_a, "ms": ms_a, "gbs": gbs_a, "bytes": "rows*C*2 read + rows written",
               "frac_of_hbm_peak": gbs_a / peaks["hbm_gbs"], "peak_gbs": peaks["hbm_gbs"],
               "kept": int(mask_a.sum().item())}
        del act, mask_a

    # ---- layer chaining: two consecutive 3x3 layers of the stack, dense intermediate vs compact intermediate
    chain = None
    pair = [L for L in layers if L.spec.kh == 3 and L.spec.stride == 1 and L.spec.C_in == L.spec.C_out
            and L.spec.C_in % 8 == 0 and L.mask.size == L.spec.P]
    if not args.no_s1 and not f32 and len(pair) >= 2 and pair[0].spec.H == pair[1].spec.H and pair[0].spec.C_in == pair[1].spec.C_in:
        A, B = pair[0], pair[1]
        sa = A.spec
        kept_a, kept_b = int(A.mask.sum()), int(B.mask.sum())
        mid_dense = torch.empty((sa.Nb, sa.Ho, sa.Wo, sa.C_out), dtype=torch.bfloat16, device="cuda")
        mid_comp = torch.empty((sa.Nb * kept_a, sa.C_out), dtype=torch.bfloat16, device="cuda")
        out_comp = torch.empty((sa.Nb * kept_b, B.spec.C_out), dtype=torch.bfloat16, device="cuda")
        LA = asx.MaskedConvLayer(sa.C_in, sa.C_out, 3, 3, 1, sa.pad)
        LB = asx.MaskedConvLayer(B.spec.C_in, B.spec.C_out, 3, 3, 1, B.spec.pad)
        LA.set_mask(A.mask)
        LB.set_mask(B.mask)
        LB.set_input_mask(A.mask)
        flush = torch.empty(L2_BYTES * 2, dtype=torch.uint8, device="cuda")

        def pair_dense():
            for (Lh, xin, yout) in ((LA, A.x, mid_dense), (LB, mid_dense, B.y)):
                rc = Lh.run_raw(xin.data_ptr(), sa.Nb, sa.H, sa.W, (A.w if Lh is LA else B.w).data_ptr(),
                                (A.b if Lh is LA else B.b).data_ptr(), yout.data_ptr(), RELU | RECOMPACT_FLAG, st)
                if rc:
                    raise RuntimeError(f"asx_run failed with status {rc}")

        def pair_compact():
            rc = LA.run_raw(A.x.data_ptr(), sa.Nb, sa.H, sa.W, A.w.data_ptr(), A.b.data_ptr(), mid_comp.data_ptr(),
                            RELU | RECOMPACT_FLAG | 8, st)
            rc = rc or LB.run_raw(mid_comp.data_ptr(), sa.Nb, sa.Ho, sa.Wo, B.w.data_ptr(), B.b.data_ptr(),
                                  out_comp.data_ptr(), RELU | RECOMPACT_FLAG | 8 | 16, st)
            if rc:
                raise RuntimeError(f"asx_run failed with status {rc}")

        def timed(fn):
            ts = []
            for i in range(13):
                flush.fill_(i)                                   # the pair starts from a cold L2
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(st_obj)
                fn()
                e1.record(st_obj)
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1))
            return statistics.median(ts[3:])
        ms_pd, ms_pc = timed(pair_dense), timed(pair_compact)
        chain = {"layers": [A.spec.name, B.spec.name], "ms_dense_intermediate": ms_pd, "ms_compact_intermediate": ms_pc,
                 "intermediate_bytes_dense": mid_dense.numel() * 2, "intermediate_bytes_compact": mid_comp.numel() * 2}
        LA.close(); LB.close()
        del flush, mid_dense, mid_comp, out_comp

    sweep = None
    if args.config == 5:
        base = {L.spec.block: per_layer_ms[i] for i, L in enumerate(layers) if L.spec.sparsity_pct == 0}
        sweep = [{"sparsity_pct": L.spec.sparsity_pct, "block": L.spec.block, "ms": per_layer_ms[i],
                  "tflops": L.flops / (per_layer_ms[i] * 1e-3) / 1e12,
                  "speedup_vs_sparsity0": base[L.spec.block] / per_layer_ms[i],
                  "ideal_speedup": layers[i].spec.M / max(1, L.kept_rows)}
                 for i, L in enumerate(layers)]

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": K,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "strong" if strong else "weak",
        "vs_baseline": None, "dtype": "tf32" if f32 else "bf16", "data": "synthetic",
        "config": {"workload": workload_name(args.config) + (f" [only {args.only}]" if args.only else ""),
                   "layers": len(layers),
                   "l2": f"inputs larger than L2: each step cycles {footprint / 1e6:.0f} MB of distinct "
                         f"layer buffers (L2 is {L2_BYTES / 1e6:.0f} MB)",
                   "step": "per layer: one asx_run with ASX_RECOMPACT = mask compaction (inside the fused kernel "
                           "for masks <= 32768 rows) + gather/GEMM/scatter"
                           + ("" if graph is None else "; one step = one CUDA-graph replay")
                           + ("; the 1x1 projection of each down-sampling block runs on a graph branch beside that block's "
                              "conv1 -> conv2, as in the network" if (fork and graph is not None) else ""),
                   "activation": args.act,
                   "storage": "fp32 (TF32 contraction)" if f32 else "bf16",
                   "mask": "one mask per layer shared by the batch"
                           + ("" if args.mask == "blocks" else "; masks from one random input-resolution score, average-pooled"
                              " to each layer and ranked (Algorithm 1, getMask)")},
        "ms_per_step_median": ms_median, "ms_per_step_min": ms_min,
        "clocks": clocks,
        "e2e": {"value": e2e_val, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms},
        "gpu_launches": K * sum(L.launches for L in layers),
        "roofline": {
            "bound": "tensor", "kernel": "masked_conv_sm100_kernel / masked_conv_patch_sm100_kernel (one launch per layer)",
            "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s",
            # frac is the spec quantity: per layer the slower of its kept-row FLOPs at the tensor peak and
            # its algorithmic bytes at the HBM peak, summed over the layers, over the measured step time
            "frac": roof_ms / ms_step,
            "frac_definition": "sum over layers of max(t_mma, t_hbm) / graph-replayed ms_per_step "
                               f"({tensor_bound_layers} of {len(layers)} layers are tensor-bound by that rule)",
            "frac_tensor_only": achieved / peak_tf,
            "frac_tensor_only_vs_other_peak": achieved / (peaks["bf16_tflops_sustained"] if burst else peaks["bf16_tflops"]),
            "layer_roofs_ms_per_step": roof_ms,
            "kernel_ms_per_step": ms_step,
            "kernel_ms_note": "the graph-replayed step: the fused kernel's launches (plus the stem's staging kernel), "
                              "overlapping by programmatic dependent launch as in the timed region",
            "in_step_ms_sum": None if in_step_ms is None else sum(in_step_ms),
            "in_step_note": "per_layer.ms_in_step: replay time of the captured prefix of layers [0..i] minus that of [0..i-1]; "
                            "sums to the step in in-line order",
            "serialised_kernel_ms_per_step": serial_ms,
            "serialised_note": "sum of per-launch times taken with an event pair around every launch (no overlap between "
                               "launches, launch gaps included): ranks the layers, exceeds the step time by construction",
            "traffic": measured_traffic(args.config, args.only or (args.mask != "blocks") or (args.act != "relu") or f32),
            "traffic_unit": "bytes per launch (ncu dram read + write, average over the step's fused-kernel launches)",
            "algorithmic_bytes_per_launch": sum(L.bytes for L in layers) / len(layers),
            "peak_source": f"{peaks['source']}: {'burst' if burst else 'sustained'} bf16 matmul figure, chosen because the timed "
                           f"region lasted {ms_total:.0f} ms (burst {peaks['bf16_tflops']:.1f}, sustained "
                           f"{peaks['bf16_tflops_sustained']:.1f} TFLOP/s; HBM copy {peaks['hbm_gbs']:.0f} GB/s)"
                           + (" x 1.1/2.25, the nominal ratio of the dense TF32 and bf16 rates" if f32 else ""),
            # the other half of the metric and the side legs, kept here so that they are stored with the record
            "metric_parts": {
                "dense_equivalent_tflops": job_dense_flops / (ms_step * 1e-3) / 1e12,
                "speedup_vs_sparsity0": (ms_dense / ms_step) if ms_dense else None,
                "ms_per_step_sparsity0": ms_dense,
                "speedup_vs_cudnn_dense": (cudnn_ms / ms_step) if cudnn_ms else None,
                "cudnn_dense_ms_per_step": cudnn_ms,
                "ms_per_step_without_recompaction": ms_frozen,
                "ms_per_step_chained_inputs": ms_chained,
                "chained_inputs_layers": chained_layers,
                "arms_timed_as": "CUDA-graph replays, all three" if graph is not None else "eager launches",
                "ideal_speedup_vs_sparsity0": dense_flops_step / max(1, flops_step)},
            "digest": {
                "s1_compaction": None if s1 is None else {k: s1[k] for k in ("rows", "ms", "gbs", "frac_of_hbm_peak")},
                "mask_from_activation": None if mfa is None else {k: mfa[k] for k in ("rows", "C", "ms", "gbs", "frac_of_hbm_peak")},
                "chain": chain,
                "sweep": None if sweep is None else [{k: e[k] for k in ("sparsity_pct", "block", "tflops", "speedup_vs_sparsity0")}
                                                     for e in sweep],
                "window_patch_layers": sum(1 for f in forms if f == 4), "row_gather_layers": sum(1 for f in forms if f in (2, 3))}},
        "cpu_baseline": cpu,
        "cpu_alg2_fp32": cpu_alg2,
        "s1_compaction": s1,
        "mask_from_activation": mfa,
        "chain": chain,
        "sweep": sweep,
        "per_layer": [{"name": L.spec.name, "M": L.spec.M, "K": L.spec.K, "N": L.spec.N, "kept_rows": L.kept_rows,
                       "ms_in_step": None if in_step_ms is None else in_step_ms[i],
                       "ms_serialised": per_layer_ms[i], "tflops": L.flops / (per_layer_ms[i] * 1e-3) / 1e12,
                       "gbs": L.bytes / (per_layer_ms[i] * 1e-3) / 1e9, "roof_ms": roofs[i],
                       "form": {0: "none", 1: "naive", 2: "row gather (copies)", 3: "row gather (TMA)", 4: "window patch"}[forms[i]]}
                      for i, L in enumerate(layers)],
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", type=int, default=3, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--act", default="relu", choices=["relu", "silu"],
                    help="epilogue activation of every layer (silu: the YOLOv5-style variant; the headline uses relu)")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"],
                    help="storage of x, w and y: bf16, or fp32 (the paper's storage; the contraction then runs in TF32)")
    ap.add_argument("--mask", default="blocks", choices=["blocks", "scores"],
                    help="blocks: seeded blocks of dropped rows; scores: the paper's getMask from one random score")
    ap.add_argument("--no-s1", action="store_true", help="skip the stand-alone compaction bandwidth leg")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-cudnn", action="store_true")
    ap.add_argument("--only", default="", help="comma-separated layer-name prefixes: run a sub-stack (profiling)")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="with N > 1 ranks: every rank runs the whole batch (weak, the default) or its share of the images (strong)")
    ap.add_argument("--no-fork-proj", action="store_true",
                    help="keep the 1x1 projections of down-sampling blocks in line instead of on a graph branch")
    ap.add_argument("--no-marginal", action="store_true", help="skip the per-layer in-step times (one graph capture per layer)")
    ap.add_argument("--no-graph", action="store_true", help="launch every step eagerly instead of replaying a CUDA graph")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
