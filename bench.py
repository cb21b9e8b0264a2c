#!/usr/bin/env python
"""Benchmark of the fused decode + masked-GEMM path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one pass of the whole path (fetch the tile factors, Boolean product, prune W, dense
product, epilogue) over one batch of seeded synthetic activations.  Rank 0 prints ONE JSON line.
With N > 1 (launched by torch.distributed.run) every rank runs the same layer on its own batch
(independent batches, no data-path collective): weak scaling, time = max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1905_05686_b200 import synth  # noqa: E402

METRIC = "fused decode+masked-GEMM TFLOP/s and effective HBM GB/s vs roofline"
DEFAULT_WORKLOAD = "ffn_16384x4096"
L2_BYTES = 126 * 1024 * 1024
# dram__bytes_read.sum + dram__bytes_write.sum of the dominant kernel, one launch, from the ncu capture
# summarised under profiles/ (null for workloads without a capture of the current kernel)
NCU_TRAFFIC_BYTES = {
    ("ffn_16384x4096", 4096): 403_700_000,      # 292.0 MB read + 111.7 MB written (profiles/gemm_tc_pair2_ffn_16384x4096.md)
    ("lenet_fc1", 32): 1_050_000,               # both launches (K-split kernel + reduction)
    ("decode_4096", 0): 530_000,                # the 2 MiB mask is still in L2 when the kernel ends
    ("decode_32768", 0): 104_000_000,
    ("alexnet_fc", 1): 76_200_000,
    ("alexnet_fc", 16): 78_900_000,             # both launches
    ("alexnet_fc", 128): 97_800_000,            # both launches
    ("conv3x3_256", 12544): 59_100_000,         # Y (6.4 MB) is still in L2 when the kernel ends
    ("alexnet_fc", -1): 76_250_000,
    ("ffn_16384x4096", -1): 135_640_000,
    ("ffn_16384x4096", -2): 432_300_000,        # dX: 412.4 MB read + 19.9 MB written
    ("ffn_16384x4096", -3): 409_300_000,        # dW: 295.0 MB read + 114.3 MB written
}
# The other configurations, timed after the headline workload and reported in "others" (L2 flushed between calls).
# batch -1: not the layer's forward pass but the cost evaluation of Algorithm 1's inner loop on its weights and index
OTHER_WORKLOADS = [("lenet_fc1", 32), ("decode_4096", 0), ("decode_32768", 0), ("alexnet_fc", 1), ("alexnet_fc", 16),
                   ("alexnet_fc", 128), ("conv3x3_256", 12544), ("alexnet_fc", -1), ("ffn_16384x4096", -1),
                   ("ffn_16384x4096", -2), ("ffn_16384x4096", -3),   # -2: dX, -3: dW of the masked backward pass
                   ("alexnet_fc", -4)]                               # -4: one iteration of the per-tile NMF of |W|


# ------------------------------------------------------------------------------------------ helpers
def algorithmic_bytes(layer: synth.Layer, batch: int, y_bytes: int = 2) -> int:
    """Bytes the method itself must move once: W, packed factors, X, Y."""
    gr, gc = layer.grid
    idx = gr * gc * (layer.tile_rows + layer.tile_cols) * layer.kw * 4
    return 2 * layer.rows * layer.cols + idx + 2 * batch * layer.cols + y_bytes * batch * layer.rows


def decode_bytes(layer: synth.Layer) -> int:
    gr, gc = layer.grid
    return gr * gc * (layer.tile_rows + layer.tile_cols) * layer.kw * 4 + layer.mask_words * 4


def dense_flops(layer: synth.Layer, batch: int) -> int:
    return 2 * batch * layer.rows * layer.cols


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
            except ValueError:
                continue
            for n, v in zip(names, r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def reduce_max(value: float, dist=None) -> float:
    """Max of a per-rank timing over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return value
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank draws its own activations; weights and index are the same layer on every rank."""
    return base_seed + 1000 * rank


# ------------------------------------------------------------------------------------------ CPU oracle legs
_ORACLE_INPUTS = {}


def oracle_sample_run(layer: synth.Layer, batch: int, target_s: float = 15.0, rows_sample=None):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload: the full index decode
    of the layer plus the masked product for the first `sb` batch rows.  Returns (flops, seconds, text)."""
    import oracle

    key = (layer.name, batch)
    if key not in _ORACLE_INPUTS:                       # generating the inputs is not part of the timed work
        _ORACLE_INPUTS.clear()
        _ORACLE_INPUTS[key] = (synth.make_factors(layer), synth.make_weights(layer), synth.make_activations(layer, batch))
    (Ip, Iz), Wb, Xb = _ORACLE_INPUTS[key]
    t0 = time.perf_counter()
    M = oracle.decode_mask(Ip, Iz, layer.rows, layer.cols)
    t_dec = time.perf_counter() - t0
    if rows_sample is None:
        t0 = time.perf_counter()
        oracle.masked_gemm(Wb, M, Xb[:1])
        t1 = max(time.perf_counter() - t0, 1e-4)
        rows_sample = int(max(1, min(batch, (target_s - t_dec) / t1)))
    t0 = time.perf_counter()
    y_ref = oracle.masked_gemm(Wb, M, Xb[:rows_sample])
    t_gemm = time.perf_counter() - t0
    flops = dense_flops(layer, rows_sample)
    text = "full index decode (%d x %d) + masked product for the first %d of %d batch rows" % (
        layer.rows, layer.cols, rows_sample, batch)
    return flops, t_dec + t_gemm, text, rows_sample, y_ref


def run_reference(args):
    import oracle

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    layer = synth.CONFIGS[args.workload]
    batch = args.batch or layer.batches[-1]
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    # one step = one bounded sample; size it so warm-up + steps stay within a few minutes in total
    per_step = max(2.0, min(15.0, 150.0 / (steps + warmup)))
    rows_sample = None
    times = []
    flops = 0
    text = ""
    for i in range(warmup + steps):
        flops, sec, text, rows_sample, _ = oracle_sample_run(layer, batch, per_step, rows_sample)
        if i >= warmup:
            times.append(sec)
    ms = 1e3 * float(np.mean(times))
    value = flops / (ms * 1e-3) / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "batch": batch, "rows": layer.rows, "cols": layer.cols,
                   "tile": [layer.tile_rows, layer.tile_cols], "rank": layer.rank, "density": layer.density},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": oracle.threads(), "kind": "oracle", "sample": text},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------------------ GPU arm
def roofline_of(workload, batch, work_bytes, work_flops, kernel_ms, peaks):
    """Roofline of one launch: the bound is the one that needs the longer time at the measured peaks."""
    t_hbm = work_bytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = work_flops / (peaks["bf16_tflops"] * 1e12)
    if t_hbm >= t_tc:
        achieved = work_bytes / (kernel_ms * 1e-3) / 1e9
        r = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"]}
    else:
        achieved = work_flops / (kernel_ms * 1e-3) / 1e12
        r = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
             "frac": achieved / peaks["bf16_tflops"], "frac_of_sustained_peak": achieved / peaks["bf16_tflops_sustained"]}
    r["traffic"] = NCU_TRAFFIC_BYTES.get((workload, batch))
    r["peak_source"] = "of " + peaks["source"]
    r["kernel_ms"] = kernel_ms
    return r


def kernel_label(B, layer, batch):
    if not batch:
        return "decode"
    if batch < 0:
        return {-1: "index_cost", -2: "backward dX (forward kernel on the transposed layer)",
                -3: "backward dW (persistent pair kernel on MN-major dY and X, index applied in the epilogue)",
                -4: "nmf, one multiplicative update of Mz and Mp (fp32 CUDA cores)"}[batch]
    plan = B.masked_gemm_plan(layer, batch)
    name = B.ALGO_NAMES[plan.algo]
    if plan.algo == B.ALGO_TENSOR:
        name += " tile%d%s panel%d splits%d stages%d" % (plan.batch_tile, " pair" if plan.cta_pair else "", plan.panel_columns,
                                                          plan.k_splits, plan.stages)
    return name


def setup_workload(B, workload, batch, rank=0):
    """Device buffers and the step function of one workload.  Returns a dict."""
    import torch

    layer = synth.CONFIGS[workload]
    decode_only = not layer.batches
    special = batch if (batch is not None and batch < 0) else 0
    cost_only = special == -1
    batch = 0 if decode_only else (batch or layer.batches[-1])
    Ip, Iz = synth.make_factors(layer)
    ipw, izw = synth.pack_ip(Ip), synth.pack_iz(Iz)
    ip, iz = B.to_device_words(ipw), B.to_device_words(izw)
    w = {"layer": layer, "batch": batch, "decode_only": decode_only, "Ip": Ip, "Iz": Iz, "ipw": ipw, "izw": izw}
    if decode_only:
        out = torch.empty((layer.rows, (layer.cols + 31) // 32), dtype=torch.int32, device="cuda")
        w.update(step=lambda: B.lrbi_decode_mask(layer, ip, iz, out), out=out,
                 work_bytes=decode_bytes(layer), work_flops=0)
    elif special in (-2, -3):
        nb = layer.batches[-1]
        Wb = synth.make_weights(layer)
        Xb = synth.make_activations(layer, nb)
        dYb = synth.make_activations(synth.Layer("dy_" + layer.name, layer.cols, layer.rows, layer.tile_cols, layer.tile_rows,
                                                 layer.rank, layer.density), nb)
        X, dY = B.to_device_bf16(Xb), B.to_device_bf16(dYb)
        flops = dense_flops(layer, nb)
        if special == -2:
            Wt = B.lrbi_transpose_bf16(B.to_device_bf16(Wb))
            out = torch.empty((nb, layer.cols), dtype=torch.bfloat16, device="cuda")
            w.update(step=lambda: B.lrbi_masked_gemm_dx(layer, Wt, ip, iz, dY, dX=out), out=out, work_flops=flops,
                     work_bytes=algorithmic_bytes(layer, nb))
        else:
            ws = torch.empty(B.lib().lrbi_masked_gemm_dw_workspace(__import__("ctypes").byref(B.Layout.of(layer)), nb), dtype=torch.uint8, device="cuda")
            out = torch.empty((layer.rows, layer.cols), dtype=torch.bfloat16, device="cuda")
            w.update(step=lambda: B.lrbi_masked_gemm_dw(layer, dY, X, ip, iz, dW=out, workspace=ws), out=out, work_flops=flops,
                     work_bytes=2 * nb * (layer.rows + layer.cols) + 2 * layer.rows * layer.cols)
    elif special == -4:
        gr, gc = layer.grid
        tiles, tm, tn, k = gr * gc, layer.tile_rows, layer.tile_cols, layer.rank
        W = B.to_device_bf16(synth.make_weights(layer))
        rng = np.random.default_rng(0)
        mp = torch.from_numpy((rng.random((tiles, tm, k)) * 0.1 + 0.01).astype(np.float32)).cuda()
        mz = torch.from_numpy((rng.random((tiles, k, tn)) * 0.1 + 0.01).astype(np.float32)).cuda()
        ws = torch.empty(B.lib().lrbi_nmf_workspace(__import__("ctypes").byref(B.Layout.of(layer))), dtype=torch.uint8, device="cuda")
        # two products of 2 k tm tn flops, two Gram matrices and two k-term denominators per element, per tile
        flops = tiles * (4 * k * tm * tn + 2 * k * k * (tm + tn) + 2 * k * k * (tm + tn))
        w.update(step=lambda: B.lrbi_nmf_update(layer, W, mp, mz, 1, workspace=ws), out=mp, work_flops=flops, alu=True,
                 work_bytes=2 * 2 * layer.rows * layer.cols + 4 * 4 * tiles * k * (tm + tn))
    elif cost_only:
        gr, gc = layer.grid
        W = B.to_device_bf16(synth.make_weights(layer))
        out = torch.empty((gr * gc, 4), dtype=torch.int64, device="cuda")
        theta = 1.5 * layer.w_std                       # |W| >= 1.5 sigma: about 13 % of a Gaussian layer kept
        w.update(step=lambda: B.lrbi_index_cost(layer, W, theta, ip, iz, out=out), out=out, work_flops=0,
                 work_bytes=2 * layer.rows * layer.cols + gr * gc * ((layer.tile_rows + layer.tile_cols) * layer.kw * 4 + 32))
    else:
        Wb = synth.make_weights(layer)
        xlayer = synth.Layer(**{**layer.__dict__, "seed": rank_seed(layer.seed, rank)})
        Xb = synth.make_activations(xlayer, batch)
        W, X = B.to_device_bf16(Wb), B.to_device_bf16(Xb)
        Y = torch.empty((batch, layer.rows), dtype=torch.bfloat16, device="cuda")
        w.update(step=lambda: B.lrbi_masked_gemm(layer, W, ip, iz, X, Y=Y), out=Y, Wb=Wb, Xb=Xb,
                 work_bytes=algorithmic_bytes(layer, batch), work_flops=dense_flops(layer, batch))
    w["keep"] = (ip, iz)
    return w


def time_calls(fn, n, warmup, flush_buf=None, stream=None):
    """Per-call device times (ms) with CUDA events on the launching stream."""
    import torch

    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
    for i in range(n):
        if flush_buf is not None:
            flush_buf.add_(1)                      # rewrites a buffer larger than L2 between timed calls
        starts[i].record()
        fn()
        ends[i].record()
    torch.cuda.synchronize()
    return [s.elapsed_time(e) for s, e in zip(starts, ends)]


def run_ours(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    from paper_1905_05686_b200 import binding as B

    B.lib()
    peaks = load_peaks()
    wl = setup_workload(B, args.workload, args.batch, rank)
    layer, batch, decode_only, step = wl["layer"], wl["batch"], wl["decode_only"], wl["step"]
    work_bytes, work_flops = wl["work_bytes"], wl["work_flops"]
    Ip, Iz, ipw, izw = wl["Ip"], wl["Iz"], wl["ipw"], wl["izw"]
    if not decode_only:
        Wb, Xb, Y = wl["Wb"], wl["Xb"], wl["out"]
    flush = None
    footprint = work_bytes
    if footprint <= L2_BYTES:
        flush = torch.zeros(256 * 1024 * 1024 // 4, dtype=torch.int32, device="cuda")

    # ---- device-timed region: K steps, barrier + synchronize on both sides, max over ranks
    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = B.launch_count()
    t_wall0 = time.perf_counter()
    if flush is None:
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        ev[0].record()
        for i in range(args.steps):
            step()
            ev[i + 1].record()
        torch.cuda.synchronize()
        per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
        total_ms = ev[0].elapsed_time(ev[-1])
    else:
        per_step = time_calls(step, args.steps, 0, flush)
        total_ms = float(sum(per_step))
    launches = B.launch_count() - launches0
    # keep the sampler alive long enough to see the load, then stop it
    while time.perf_counter() - t_wall0 < 0.6:
        step()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if world > 1:
        dist.barrier()
    total_ms = reduce_max(total_ms, dist if world > 1 else None)
    ms_per_step = total_ms / args.steps
    if B.device_status() != 0:
        raise SystemExit("device status word is not clean: %d" % B.device_status())

    unit = "GB/s" if decode_only else "TFLOP/s"
    if decode_only:
        value = world * work_bytes / (ms_per_step * 1e-3) / 1e9
    else:
        value = world * work_flops / (ms_per_step * 1e-3) / 1e12

    # ---- end to end through the host-buffer entry point (pinned host X and Y, copies inside the timing)
    e2e = None
    if not decode_only:
        hl = B.HostLayer(layer, Wb, ipw, izw, batch)
        Xh = torch.from_numpy(Xb.view(np.int16)).view(torch.bfloat16).pin_memory()
        Yh = torch.empty((batch, layer.rows), dtype=torch.bfloat16).pin_memory()
        for _ in range(3):
            hl.forward_host(Xh, Yh)
        n_e2e = max(3, min(args.steps, 10))
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            hl.forward_host(Xh, Yh)            # returns when Y_host is complete
        e2e_ms = 1e3 * (time.perf_counter() - t0) / n_e2e
        e2e_ms = reduce_max(e2e_ms, dist if world > 1 else None)
        e2e = {"value": world * work_flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": int(Xh.numel() * 2), "d2h_bytes_per_step": int(Yh.numel() * 2),
               "api": "lrbi_layer_forward_host (weights and index resident, X and Y in pinned host memory)"}
        # the host-buffer call works through the batch in chunks, so K may be split differently:
        # same values up to fp32 summation order and one bf16 rounding
        y_dev, y_host = Y.float().cpu(), Yh.float()
        if not (torch.linalg.norm(y_dev - y_host) <= 4e-3 * torch.linalg.norm(y_dev)):
            raise SystemExit("host-buffer entry point disagrees with the device entry point")
        hl.close()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- roofline of the dominant kernel (one launch per step for this workload)
    launches_per_step = launches / args.steps
    kernel_ms = float(np.mean(per_step))
    roofline = roofline_of(args.workload, batch, work_bytes, work_flops, kernel_ms, peaks)
    roofline["launches_per_step"] = launches_per_step

    # ---- CPU oracle on a bounded sample of the same workload
    cpu, parity = None, None
    if not args.no_cpu_baseline:
        import oracle
        if decode_only:
            t0 = time.perf_counter()
            M_ref = oracle.decode_mask(Ip, Iz, layer.rows, layer.cols)
            sec = time.perf_counter() - t0
            cpu = {"value": work_bytes / sec / 1e9, "unit": "GB/s", "cores": oracle.threads(), "kind": "oracle",
                   "sample": "the whole index decode, once", "seconds": sec}
            bad = int((wl["out"].cpu().numpy().view(np.uint32) != synth.pack_mask(M_ref)).sum())
            parity = {"mask_words_differing": bad, "against": "oracle"}
            if bad:
                raise SystemExit("the timed kernel's mask disagrees with the oracle in %d words" % bad)
        else:
            flops, sec, text, rows_sample, y_ref = oracle_sample_run(layer, batch, 15.0)
            cpu = {"value": flops / sec / 1e12, "unit": "TFLOP/s", "cores": oracle.threads(), "kind": "oracle",
                   "sample": text, "seconds": sec}
            # the rows the oracle has just computed, against what the timed kernel left in Y
            y_gpu = Y[:rows_sample].float().cpu().numpy().astype(np.float64)
            rel = float(np.linalg.norm(y_gpu - y_ref) / max(np.linalg.norm(y_ref), 1e-300))
            parity = {"rel_fro": rel, "rows": int(rows_sample), "tolerance": 5e-3, "against": "oracle (fp64)"}
            if not rel <= 5e-3:
                raise SystemExit("the timed kernel's Y disagrees with the oracle: relative Frobenius error %g" % rel)

    # ---- the other configurations (rank 0, after the headline numbers are taken)
    others = []
    if args.others and world == 1:
        del wl, step
        if not decode_only:
            del Y
        torch.cuda.empty_cache()
        flush2 = torch.zeros(256 * 1024 * 1024 // 4, dtype=torch.int32, device="cuda")
        for name, ob in OTHER_WORKLOADS:
            if name == args.workload and (ob == batch or not ob):
                continue                                  # the headline workload itself
            ow = setup_workload(B, name, ob)
            if os.environ.get("LRBI_BENCH_TRACE"):
                print("timing %s %s" % (name, ob), file=sys.stderr, flush=True)
            l0 = B.launch_count()
            ts = time_calls(ow["step"], args.other_steps, 3, flush2)
            nl = (B.launch_count() - l0) / (args.other_steps + 3)
            ms = float(np.mean(ts))
            rl = roofline_of(name, ow["batch"], ow["work_bytes"], ow["work_flops"], ms, peaks)
            if ow.get("alu"):
                # fp32 FMA roof: 148 SMs x 128 lanes x 2 flop at the maximum SM clock (1965 MHz) = 74.4 TFLOP/s
                ach = ow["work_flops"] / (ms * 1e-3) / 1e12
                rl = {"bound": "alu", "achieved": ach, "peak": 74.4, "unit": "TFLOP/s", "frac": ach / 74.4, "traffic": None,
                      "peak_source": "derived: 148 SMs x 128 fp32 lanes x 2 x 1.965 GHz", "kernel_ms": ms}
            others.append({"workload": name, "batch": ow["batch"], "kernel": kernel_label(B, ow["layer"], ow["batch"]),
                           "ms": ms, "ms_median": float(np.median(ts)), "launches_per_step": nl,
                           "algorithmic_bytes": ow["work_bytes"], "dense_flops": ow["work_flops"], "roofline": rl})
            del ow
        if B.device_status() != 0:
            raise SystemExit("device status word is not clean after the other workloads: %d" % B.device_status())

    line = {
        "metric": METRIC, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u32" if decode_only else "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "batch": batch, "rows": layer.rows, "cols": layer.cols,
                   "tile": [layer.tile_rows, layer.tile_cols], "rank": layer.rank, "density": layer.density,
                   "kernel": kernel_label(B, layer, batch),
                   "l2": "inputs larger than L2" if flush is None else "L2 flushed between timed calls (256 MiB rewrite)",
                   "algorithmic_bytes": work_bytes, "dense_flops": work_flops,
                   "effective_hbm_gbs": work_bytes / (ms_per_step * 1e-3) / 1e9},
        "clocks": clocks, "gpu_launches": int(launches), "roofline": roofline,
    }
    if e2e:
        line["e2e"] = e2e
    if cpu:
        line["cpu_baseline"] = cpu
    if parity:
        line["parity"] = parity
    if others:
        line["others"] = others
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(synth.CONFIGS))
    ap.add_argument("--batch", type=int, default=0, help="override the batch of the workload")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-others", dest="others", action="store_false",
                    help="skip the other configurations (reported in the \"others\" array of the line)")
    ap.add_argument("--other-steps", type=int, default=30)
    args = ap.parse_args()
    if args.impl == "reference":
        if args.steps == 50 and args.warmup == 5:
            args.steps, args.warmup = 3, 1
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
