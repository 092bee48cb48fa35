#!/usr/bin/env python
"""Benchmark of the 2:4-sparse INT8 linear-layer path on B200.

One step = one per-inference pass of a transformer block's four linear layers
(QKV, proj, fc1+GELU, fc2) over one batch of synthetic activations: for every
layer, activation quantisation (FP16 -> INT8, per-tensor absmax scale) followed
by the fused sparse GEMM + de-quantise/bias/GELU epilogue writing FP16.  The
offline weight preparation (prune -> quantise -> compress -> pack) runs once
before the timed region and is reported separately under "prep".

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on the
host cores instead (a deliberately plain program: context, not a target).
"""
from __future__ import annotations

import argparse
import collections
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2305_10727_b200 import inputs  # noqa: E402

METRIC = "sparse INT8 GEMM effective TOPS (dense-equivalent 2*M*N*K / time), ViT-B block linears at batch 64"
UNIT = "TOPS"
STEP_TEXT = "per layer: quant_act (per-tensor absmax scale + quantise) + sparse GEMM with fused epilogue, FP16 out"
NOMINAL_SPARSE_INT8_TOPS = 9000.0      # NVIDIA's dense-half figure for B200 INT8 with 2:4 sparsity (4 x 2250 BF16)
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM traffic of the step's GEMM launches comes from the ncu summary committed under profiles/ (a line
# "dram_bytes_gemm_launches_per_step <bytes> kernel_sha <sha>"); it is reported only while the kernel
# sources still hash to the value recorded there.
TRAFFIC_SUMMARY = os.path.join(ROOT, "profiles", "gemm_i8_sparse_deit_base_block.md")
KERNEL_SOURCES = ("gemm_i8.cu", "ptx.cuh", "quant_math.cuh", "common.cuh")


def kernel_sha():
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2305_10727_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload_key):
    """(bytes per step, launches) of the GEMM launches from the committed ncu summary, or (None, None)."""
    try:
        with open(TRAFFIC_SUMMARY) as f:
            for line in f:
                parts = line.split()
                if len(parts) >= 7 and parts[0] == "dram_bytes_gemm_launches_per_step" and parts[1] == workload_key:
                    if parts[6] == kernel_sha():
                        return float(parts[2]), int(parts[4])
    except OSError:
        pass
    return None, None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


def layer_flops(M, L):
    return 2.0 * M * L.N * L.K


def layer_bytes(M, L):
    # algorithmic bytes of the fused GEMM: INT8 activations in, compressed weight (0.625 B/param)
    # plus scale and bias vectors in, FP16 out
    return M * L.K + 0.625 * L.N * L.K + 8 * L.N + 2.0 * M * L.N


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.tmp = None

    def start(self):
        try:
            self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.tmp.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        self.tmp.close()
        try:
            os.unlink(self.tmp.name)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# --------------------------------------------------------------------------- reference arm
def run_reference(args, cfg):
    """The CPU oracle, as it stands, on a bounded sample of the same workload.

    Each step runs the block's four layers on the first `rows` token rows; rows is sized from a
    short calibration so that the whole --steps/--warmup run stays near a minute of CPU work.
    """
    import oracle
    oracle.build()
    layers = cfg.layers

    def make(rows):
        data = []
        for li, L in enumerate(layers):
            d = inputs.make_layer_inputs(cfg, li, M=rows)
            data.append((L, d, oracle.prepare_weight(d["W"])))
        return data

    cores = oracle.host_cores()

    def step(data):
        for L, d, prep in data:
            oracle.layer_forward(d["X"], prep, d["bias"], act=1 if L.gelu else 0, threads=cores)

    rows = args.ref_rows
    if rows <= 0:
        cal = make(16)
        t0 = time.perf_counter()
        step(cal)
        per_row = (time.perf_counter() - t0) / 16
        budget_s = 60.0
        rows = int(budget_s / max(per_row, 1e-9) / (args.steps + args.warmup))
        rows = max(4 * cores, min(rows, 512 * cores, cfg.M))
    data = make(rows)
    flops = sum(layer_flops(rows, L) for L in layers)
    for _ in range(args.warmup):
        step(data)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step(data)
    dt = (time.perf_counter() - t0) / args.steps
    value = flops / dt / 1e12
    sample = "first %d token rows of each of the %d layers (of M=%d) per step" % (rows, len(layers), cfg.M)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3 * (cfg.M / rows),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": cfg.name, "M": cfg.M, "layers": [[L.name, L.K, L.N] for L in layers],
                   "step": STEP_TEXT, "launch": "host threads", "l2": "not applicable (CPU)",
                   "parallelism": "%d host threads over row blocks" % cores,
                   "note": "ms_per_step is the sampled step scaled to all M rows"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------------- GPU arm
def run_gpusq(args, cfg):
    import torch
    import torch.distributed as dist

    from paper_2305_10727_b200 import binding as B
    from paper_2305_10727_b200 import replicas

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libgpusq has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    B.load()
    peaks = load_peaks()
    M = cfg.M
    layers = cfg.layers

    # ---- inputs (seeded, synthetic) and offline weight preparation on the device
    host = [inputs.make_layer_inputs(cfg, li, seed=rank) for li in range(len(layers))]
    state = []
    prep_us = {}
    for li, L in enumerate(layers):
        h = host[li]
        W = torch.from_numpy(h["W"]).to(dev)
        X = torch.from_numpy(h["X"]).to(dev)
        bias = torch.from_numpy(h["bias"]).to(dev)
        Wp = torch.empty_like(W)
        Wq = torch.empty((L.N, L.K), dtype=torch.int8, device=dev)
        ws = torch.empty((L.N,), dtype=torch.float32, device=dev)
        vals = torch.empty((L.N, L.K // 2), dtype=torch.int8, device=dev)
        meta = torch.empty((L.N, L.K // 8), dtype=torch.uint8, device=dev)
        Wpk = torch.empty((B.packed_bytes(L.N, L.K),), dtype=torch.uint8, device=dev)

        def prep_once():
            B.prune24(W, Wp=Wp)
            B.quant_weight(Wp, Wq=Wq, w_scale=ws)
            B.compress24(Wq, vals=vals, meta=meta)
            B.pack24(vals, meta, Wpacked=Wpk)

        prep_once()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(5):
            prep_once()
        e1.record()
        torch.cuda.synchronize()
        prep_us[L.name] = e0.elapsed_time(e1) * 1e3 / 5
        state.append(dict(L=L, X=X, bias=bias, Wq=Wq, ws=ws, Wpk=Wpk,
                          Xq=torch.empty((M, L.K), dtype=torch.int8, device=dev),
                          xs=torch.empty((1,), dtype=torch.float32, device=dev),
                          wsb=torch.zeros((B.quant_act_workspace(M, L.K),), dtype=torch.uint8, device=dev),
                          Y=torch.empty((M, L.N), dtype=torch.float16, device=dev)))
    status = torch.zeros(4, dtype=torch.int32, device=dev)

    def layer_quant(s):
        B.quant_act(s["X"], Xq=s["Xq"], x_scale=s["xs"], workspace=s["wsb"])

    def layer_gemm(s):
        B.spgemm_i8(s["Xq"], s["Wpk"], s["L"].N, s["ws"], s["xs"], s["bias"],
                    act=B.ACT_GELU if s["L"].gelu else B.ACT_NONE, out_type=B.OUT_F16, Y=s["Y"], status_buf=status)

    def layer_gemm_dense(s):
        B.gemm_i8_dense(s["Xq"], s["Wq"], s["ws"], s["xs"], s["bias"],
                        act=B.ACT_GELU if s["L"].gelu else B.ACT_NONE, out_type=B.OUT_F16, Y=s["Y"],
                        status_buf=status)

    def step():
        for s in state:
            layer_quant(s)
            layer_gemm(s)

    launches_per_step = 2 * len(state)        # quant_act (one cooperative launch) + GEMM per layer

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    stream = torch.cuda.Stream()
    torch.cuda.set_stream(stream)
    graph = None
    if args.launch == "graph":
        for _ in range(2):
            step()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step()
        run_step = graph.replay
    else:
        run_step = step

    # ---- headline: K whole steps, inputs resident in HBM
    for _ in range(max(args.warmup, 3)):
        run_step()
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        run_step()
    e1.record(stream)
    barrier()
    ms_step = e0.elapsed_time(e1) / args.steps

    # ---- durations of the individual launches, in the context of the step.  Event record nodes between
    # the kernels of a graph add several microseconds of idle time per node and would be charged to the
    # kernels, so each duration is taken as a difference of whole-loop times instead: K replays of the
    # full step minus K replays of the step with that launch left out, every loop bracketed by CUDA
    # events on the launch stream.
    def loop_ms(fn_step):
        for _ in range(2):
            fn_step()
        torch.cuda.synchronize()
        run = fn_step
        if args.launch == "graph":
            gx = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gx, stream=stream):
                fn_step()
            run = gx.replay
        for _ in range(3):
            run()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        for _ in range(args.steps):
            run()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / args.steps

    def step_without(skip_gemm=(), skip_quant=(), gemm=None):
        gemm = gemm or layer_gemm

        def fn():
            for i, s in enumerate(state):
                if i not in skip_quant:
                    layer_quant(s)
                if i not in skip_gemm:
                    gemm(s)
        return fn

    all_idx = tuple(range(len(state)))
    single = len(state) == 1            # a one-layer step: leaving the layer out leaves nothing to time
    ms_full = loop_ms(step_without())
    ms_no_gemm = loop_ms(step_without(skip_gemm=all_idx))
    ms_no_quant = loop_ms(step_without(skip_quant=all_idx))
    gemm_us, quant_us, dense_us = {}, {}, {}
    for i, s in enumerate(state):
        name = s["L"].name
        if single:
            gemm_us[name] = [max(ms_full - ms_no_gemm, 1e-3) * 1e3]
            quant_us[name] = [max(ms_full - ms_no_quant, 1e-3) * 1e3]
        else:
            gemm_us[name] = [max(ms_full - loop_ms(step_without(skip_gemm=(i,))), 1e-3) * 1e3]
            quant_us[name] = [max(ms_full - loop_ms(step_without(skip_quant=(i,))), 1e-3) * 1e3]
    # the same step with the activation scales supplied (calibrated once, as the paper's deployed model
    # does with its learned scales) instead of computed from every batch: extra information
    def step_static_scale():
        for s in state:
            B.quant_act(s["X"], Xq=s["Xq"], x_scale=s["xs"], scale_mode=B.SCALE_GIVEN)
            layer_gemm(s)
    ms_static = loop_ms(step_static_scale)

    # the block with the MLP chained in INT8, as the deployed model chains its quantise / de-quantise nodes
    # (Sec. 2.2): fc1 writes requantised INT8 (GELU fused, output scale calibrated once with quant_act on
    # its FP16 output) and fc2 reads those codes directly, so fc2's quant_act disappears: extra information
    ms_chain = None
    names = [s["L"].name for s in state]
    if "fc1" in names and "fc2" in names:
        f1, f2 = state[names.index("fc1")], state[names.index("fc2")]
        if f1["L"].N == f2["L"].K:
            cal_q = torch.empty((M, f1["L"].N), dtype=torch.int8, device=dev)
            y_scale = torch.empty((1,), dtype=torch.float32, device=dev)
            layer_quant(f1)
            layer_gemm(f1)
            B.quant_act(f1["Y"], Xq=cal_q, x_scale=y_scale, workspace=f2["wsb"])    # calibration of the output scale

            def step_chain():
                for s in state:
                    if s is f1:
                        layer_quant(s)
                        B.spgemm_i8(s["Xq"], s["Wpk"], s["L"].N, s["ws"], s["xs"], s["bias"], act=B.ACT_GELU,
                                    out_type=B.OUT_I8, out_scale=y_scale, Y=cal_q, status_buf=status)
                    elif s is f2:
                        B.spgemm_i8(cal_q, s["Wpk"], s["L"].N, s["ws"], y_scale, s["bias"], act=B.ACT_NONE,
                                    out_type=B.OUT_F16, Y=s["Y"], status_buf=status)
                    else:
                        layer_quant(s)
                        layer_gemm(s)
            ms_chain = loop_ms(step_chain)

            # The whole block chained as the deployed model runs it (Sec. 2.2, Sec. 4.1): activation scales
            # are constants (calibrated here once, learned in the paper), so every quantise node is one
            # pass, fc1 writes INT8 and fc2 reads it.  What sits between the linears of a real block
            # (attention, LayerNorm, residuals: FP16, not sparsified, Sec. 3.2) is not part of this path
            # and not timed; each linear reads its own resident FP16 input as in the headline step.
            def chain_static(skip_mlp=False):
                def fn():
                    for s in state:
                        if s is f1:
                            if skip_mlp:
                                continue
                            B.quant_act(s["X"], Xq=s["Xq"], x_scale=s["xs"], scale_mode=B.SCALE_GIVEN)
                            B.spgemm_i8(s["Xq"], s["Wpk"], s["L"].N, s["ws"], s["xs"], s["bias"], act=B.ACT_GELU,
                                        out_type=B.OUT_I8, out_scale=y_scale, Y=cal_q, status_buf=status)
                        elif s is f2:
                            if skip_mlp:
                                continue
                            B.spgemm_i8(cal_q, s["Wpk"], s["L"].N, s["ws"], y_scale, s["bias"], act=B.ACT_NONE,
                                        out_type=B.OUT_F16, Y=s["Y"], status_buf=status)
                        else:
                            B.quant_act(s["X"], Xq=s["Xq"], x_scale=s["xs"], scale_mode=B.SCALE_GIVEN)
                            layer_gemm(s)
                return fn
            ms_chain_static = loop_ms(chain_static())
            ms_chain_static_no_mlp = loop_ms(chain_static(skip_mlp=True)) if len(state) > 2 else 0.0

            # The MLP with a scale computed from the data and still no second pass: fc1 writes FP16 and
            # reports its largest magnitude, the quantise node derives the scale from it (one launch, one
            # pass), fc2 reads the codes.
            y_amax = torch.zeros((1,), dtype=torch.float32, device=dev)
            y1_scale = torch.empty((1,), dtype=torch.float32, device=dev)

            def mlp_dynamic(skip_mlp=False):
                def fn():
                    for s in state:
                        if s is f1:
                            if skip_mlp:
                                continue
                            layer_quant(s)
                            y_amax.zero_()
                            B.spgemm_i8_absmax(s["Xq"], s["Wpk"], s["L"].N, s["ws"], s["xs"], s["bias"], act=B.ACT_GELU,
                                               Y=s["Y"], y_absmax=y_amax, status_buf=status)
                        elif s is f2:
                            if skip_mlp:
                                continue
                            B.quant_act_absmax(f1["Y"], y_amax, Xq=cal_q, x_scale=y1_scale)
                            B.spgemm_i8(cal_q, s["Wpk"], s["L"].N, s["ws"], y1_scale, s["bias"], act=B.ACT_NONE,
                                        out_type=B.OUT_F16, Y=s["Y"], status_buf=status)
                        else:
                            layer_quant(s)
                            layer_gemm(s)
                return fn
            ms_mlp_dyn = loop_ms(mlp_dynamic())
            ms_mlp_dyn_rest = loop_ms(mlp_dynamic(skip_mlp=True)) if len(state) > 2 else 0.0
    # the paper's intermediate FP16 2:4 sparse model (Sec. 3.4): the same four layers on binary16
    # weights and activations, no quantise node, FP32 accumulation: extra information
    ms_half, half_layer_us = None, {}
    if all(s["L"].K % 8 == 0 and s["L"].N % 8 == 0 for s in state):
        for s in state:
            Wt = torch.from_numpy(host[state.index(s)]["W"]).to(dev)
            hv, hm = B.compress24_f16(B.prune24(Wt))
            s["Wpk16"] = B.pack24_f16(hv, hm)
            del Wt, hv, hm

        def half_gemm(s):
            B.spgemm_f16(s["X"], s["Wpk16"], s["L"].N, bias=s["bias"],
                         act=B.ACT_GELU if s["L"].gelu else B.ACT_NONE, out_type=B.OUT_F16, Y=s["Y"], status_buf=status)

        def step_half(skip=()):
            def fn():
                for i, s in enumerate(state):
                    if i not in skip:
                        half_gemm(s)
            return fn
        ms_half = loop_ms(step_half())
        for i, s in enumerate(state):
            half_layer_us[s["L"].name] = round((ms_half if single else
                                                max(ms_half - loop_ms(step_half(skip=(i,))), 1e-3)) * 1e3, 2)
    # the paper's INT4 model (Sec. 3.1: pair-wise 4:8 sparsity; 0.3125 bytes per weight): the same step with
    # 4-bit weights and activations, computed exactly on the INT8 2:4 path with regrouped columns (this GPU
    # has no 4-bit tensor-core kind, so the paper's extra 4-bit speed-up does not exist here): extra information
    ms_int4 = None
    if all(s["L"].K % 16 == 0 for s in state):
        for s in state:
            Wt = torch.from_numpy(host[state.index(s)]["W"]).to(dev)
            Wq4, s["ws4"] = B.quant_weight4(B.prune48(Wt))
            s["Wpk4"] = B.pack24(*B.expand48(*B.compress48(Wq4)))
            del Wt, Wq4

        def step_int4():
            for s in state:
                B.quant_act4(s["X"], Xq=s["Xq"], x_scale=s["xs"], workspace=s["wsb"])
                B.spgemm_i8(s["Xq"], s["Wpk4"], s["L"].N, s["ws4"], s["xs"], s["bias"],
                            act=B.ACT_GELU if s["L"].gelu else B.ACT_NONE, out_type=B.OUT_F16, Y=s["Y"], status_buf=status)
        ms_int4 = loop_ms(step_int4)
    ms_dense = loop_ms(step_without(gemm=layer_gemm_dense))
    for i, s in enumerate(state):
        name = s["L"].name
        dense_us[name] = [max(ms_dense - (ms_no_gemm if single else
                                          loop_ms(step_without(skip_gemm=(i,), gemm=layer_gemm_dense))), 1e-3) * 1e3]
    gemm_block_us = (ms_full - ms_no_gemm) * 1e3
    dense_block_us = (ms_dense - ms_no_gemm) * 1e3
    clocks = sampler.stop()
    status_host = status.cpu().tolist()
    # the status word of every layer's activation-quantisation workspace (0 unless a bounded wait expired)
    quant_status = [B.quant_act_status(s["wsb"]) for s in state]
    if any(status_host) or any(quant_status):
        raise SystemExit("a device-side wait expired: GEMM status %s, quant_act status %s" % (status_host, quant_status))

    ms_step = replicas.max_over_ranks(ms_step, dev)          # the slowest rank's time

    flops_step = sum(layer_flops(M, L) for L in layers)
    value = replicas.whole_job_throughput(flops_step, ms_step * 1e-3, world) / 1e12

    # ---- roofline of the dominant kernel (the sparse GEMM, all shapes of the step).  Two roofs: the tensor
    # pipe (dense-equivalent ops / peak) and HBM (algorithmic bytes / measured copy bandwidth); the one
    # that needs the longer time for these shapes binds, and `frac` is the fraction of THAT roof.  The
    # tensor peak is derived from the measured cuBLAS BF16 figure of the regime the timed region ran in
    # (burst: milliseconds at full clocks; sustained: a seconds-long loop under the power cap) times the
    # nominal INT8-2:4 : BF16 ratio; the fraction of the nominal 9000 TOPS is reported beside it.
    gemm_mean = {k: statistics.fmean(v) for k, v in gemm_us.items()}
    gemm_total_us = gemm_block_us
    achieved = flops_step / (gemm_total_us * 1e-6) / 1e12
    sparse_ratio = NOMINAL_SPARSE_INT8_TOPS / NOMINAL_BF16_TFLOPS
    timed_region_s = ms_step * 1e-3 * args.steps
    regime = "burst" if timed_region_s < 1.0 else "sustained"
    tensor_peak = (peaks["bf16_tflops"] if regime == "burst" else peaks["bf16_tflops_sustained"]) * sparse_ratio
    bytes_step = sum(layer_bytes(M, L) for L in layers)
    hbm_achieved = bytes_step / (gemm_total_us * 1e-6) / 1e9
    t_tensor_us = flops_step / (tensor_peak * 1e12) * 1e6
    t_hbm_us = bytes_step / (peaks["hbm_gbs"] * 1e9) * 1e6
    per_layer = {}
    for L in layers:
        us = gemm_mean[L.name]
        per_layer[L.name] = {
            "K": L.K, "N": L.N, "us": round(us, 2),
            "tops": round(layer_flops(M, L) / us / 1e6, 1),
            "frac_nominal_sparse_peak": round(layer_flops(M, L) / us / 1e6 / NOMINAL_SPARSE_INT8_TOPS, 4),
            "hbm_gbs": round(layer_bytes(M, L) / us / 1e3, 1),
            "hbm_frac": round(layer_bytes(M, L) / us / 1e3 / peaks["hbm_gbs"], 4),
            "dense_variant_us": round(statistics.fmean(dense_us[L.name]), 2),
            "speedup_vs_dense_variant": round(statistics.fmean(dense_us[L.name]) / us, 3),
            "quant_act_us": round(statistics.fmean(quant_us[L.name]), 2),
        }
    traffic, traffic_launches = recorded_traffic(args.config)
    common = {
        "kernel": "gemm_i8_kernel<sparse>", "launches_per_step": len(layers),
        "traffic": traffic, "traffic_note": None if traffic is None else
        "ncu dram__bytes_read.sum + dram__bytes_write.sum summed over the %d GEMM launches of one step, L2 not flushed "
        "between launches (profiles/gemm_i8_sparse_deit_base_block.md)" % traffic_launches,
        "algorithmic_bytes": bytes_step, "tensor_time_us": round(t_tensor_us, 2), "hbm_time_us": round(t_hbm_us, 2),
        "tensor_achieved_tops": round(achieved, 1), "tensor_peak_tops": round(tensor_peak, 1),
        "tensor_peak_source": "%s BF16 %s x %.0f (nominal INT8-sparse : BF16 ratio)" % (peaks["_source"], regime, sparse_ratio),
        "tensor_frac": round(achieved / tensor_peak, 4),
        "frac_of_nominal_9000": round(achieved / NOMINAL_SPARSE_INT8_TOPS, 4),
        "hbm_achieved_gbs": round(hbm_achieved, 1), "hbm_peak_gbs": peaks["hbm_gbs"],
        "hbm_frac": round(hbm_achieved / peaks["hbm_gbs"], 4),
        "gemm_block_us": round(gemm_total_us, 2),
        "timing": "CUDA events around %d replays of the step with and without the GEMM launches; the difference is the GEMMs' time in context" % args.steps,
        "dense_variant_block_us": round(dense_block_us, 2), "speedup_vs_dense_variant": round(dense_block_us / gemm_block_us, 3),
    }
    if t_hbm_us >= t_tensor_us:
        roofline = {"bound": "hbm", "achieved": round(hbm_achieved, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": round(hbm_achieved / peaks["hbm_gbs"], 4),
                    "peak_source": "%s copy bandwidth" % peaks["_source"]}
    else:
        roofline = {"bound": "tensor", "achieved": round(achieved, 1), "peak": round(tensor_peak, 1), "unit": "TFLOP/s",
                    "frac": round(achieved / tensor_peak, 4), "peak_source": common["tensor_peak_source"]}
    roofline.update(common)

    # ---- end to end through the public API with host buffers (pinned), copies inside the timed region
    e2e = None
    if not args.no_e2e:
        hX = [torch.from_numpy(h["X"]).pin_memory() for h in host]
        hY = [torch.empty((M, L.N), dtype=torch.float16).pin_memory() for L in layers]
        h2d = sum(x.numel() * 2 for x in hX)
        d2h = sum(y.numel() * 2 for y in hY)

        # Three streams, as a serving loop would run it: host -> device copies of the next layer's
        # activations, the kernels, and device -> host copies of finished outputs overlap (the two copy
        # directions use separate DMA engines).  Events order each layer's copy-in -> kernels -> copy-out
        # and keep a step from overwriting buffers the previous step still uses.
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        ev_in = [torch.cuda.Event() for _ in state]
        ev_done = [torch.cuda.Event() for _ in state]
        ev_out = [torch.cuda.Event() for _ in state]
        first = [True]

        def e2e_step():
            for i, (s, hx, hy) in enumerate(zip(state, hX, hY)):
                if not first[0]:
                    s_in.wait_event(ev_done[i])          # last step's kernels have read X
                with torch.cuda.stream(s_in):
                    s["X"].copy_(hx, non_blocking=True)
                    ev_in[i].record(s_in)
                stream.wait_event(ev_in[i])
                if not first[0]:
                    stream.wait_event(ev_out[i])         # last step's copy-out has read Y
                layer_quant(s)
                layer_gemm(s)
                ev_done[i].record(stream)
                s_out.wait_event(ev_done[i])
                with torch.cuda.stream(s_out):
                    hy.copy_(s["Y"], non_blocking=True)
                    ev_out[i].record(s_out)
            first[0] = False

        for _ in range(3):
            e2e_step()
        barrier()
        n_e2e = max(3, min(args.steps, 10))
        e0.record(stream)
        s_in.wait_event(e0)
        s_out.wait_event(e0)
        for _ in range(n_e2e):
            e2e_step()
        for ev in ev_out:
            stream.wait_event(ev)
        e1.record(stream)
        barrier()
        ms_e2e = e0.elapsed_time(e1) / n_e2e
        ms_e2e = replicas.max_over_ranks(ms_e2e, dev)
        e2e = {"value": round(world * flops_step / (ms_e2e * 1e-3) / 1e12, 2), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": round(ms_e2e, 4), "steps": n_e2e}

    # ---- CPU baseline: the oracle on a bounded sample (rank 0, N = 1 only): on one core, and with its
    # row blocks spread over all host cores (the same plain routines, called once per block of rows)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        cores = oracle.host_cores()
        rows_all = min(M, args.ref_rows)
        rows_one = min(M, max(256, args.ref_rows // 4))
        preps = [oracle.prepare_weight(host[li]["W"]) for li in range(len(layers))]

        def oracle_seconds(rows, threads):
            t = 0.0
            for li, L in enumerate(layers):
                Xs = np.ascontiguousarray(host[li]["X"][:rows])
                t0 = time.perf_counter()
                oracle.layer_forward(Xs, preps[li], host[li]["bias"], act=1 if L.gelu else 0, threads=threads)
                t += time.perf_counter() - t0
            return t

        t_one = oracle_seconds(rows_one, 1)
        t_all = oracle_seconds(rows_all, cores)
        tops_one = sum(layer_flops(rows_one, L) for L in layers) / t_one / 1e12
        tops_all = sum(layer_flops(rows_all, L) for L in layers) / t_all / 1e12
        cpu_baseline = {"value": tops_all, "unit": UNIT, "cores": cores, "kind": "oracle", "value_1core": tops_one,
                        "sample": "quantise + GEMM + epilogue of every layer: first %d of %d token rows on %d cores (%.1f s), "
                                  "first %d rows on one core (%.1f s)" % (rows_all, M, cores, t_all, rows_one, t_one)}

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": round(ms_step, 5), "block_us": round(ms_step * 1e3, 2),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": cfg.name, "M": M, "layers": [[L.name, L.K, L.N] for L in layers],
                       "step": STEP_TEXT,
                       "launch": args.launch, "l2": "inputs exceed L2: a step touches %.0f MB" % ((bytes_step + sum(2.0 * M * L.K for L in layers)) / 1e6),
                       "parallelism": "replicas, tokens sharded, no collective" if world > 1 else "single GPU"},
            "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
            "step_us_x_sm_mhz": None if not clocks.get("sm_mhz") else round(ms_step * 1e3 * clocks["sm_mhz"], 1),
            "layers": per_layer, "prep_us": {k: round(v, 2) for k, v in prep_us.items()},
            "static_scale_step": {"block_us": round(ms_static * 1e3, 2),
                                  "value": round(flops_step / (ms_static * 1e-3) / 1e12, 2), "unit": UNIT,
                                  "note": "same step with supplied activation scales (GPUSQ_SCALE_GIVEN); rank 0 only"},
            "int8_chained_mlp_step": None if ms_chain is None else {
                "block_us": round(ms_chain * 1e3, 2), "value": round(flops_step / (ms_chain * 1e-3) / 1e12, 2),
                "unit": UNIT, "note": "fc1 writes requantised INT8 (calibrated scale) that fc2 reads: 7 launches; rank 0 only"},
            "chained_block_step": None if ms_chain is None else {
                "block_us": round(ms_chain_static * 1e3, 2), "value": round(flops_step / (ms_chain_static * 1e-3) / 1e12, 2),
                "unit": UNIT, "mlp_us": round((ms_chain_static - ms_chain_static_no_mlp) * 1e3, 2),
                "launches": 2 * len(state) - 1,
                "note": "supplied activation scales (one-pass quantise nodes), fc1 writes INT8 that fc2 reads; mlp_us = "
                        "quantise + fc1 (GELU, INT8 out) + fc2 in context; rank 0 only"},
            "mlp_dynamic_scale_step": None if ms_chain is None else {
                "block_us": round(ms_mlp_dyn * 1e3, 2), "mlp_us": round((ms_mlp_dyn - ms_mlp_dyn_rest) * 1e3, 2),
                "note": "computed scales everywhere; fc1 writes FP16 and its largest magnitude (gpusq_spgemm_i8_absmax), "
                        "fc2's quantise node is one pass (gpusq_quant_act_absmax); rank 0 only"},
            "int4_model_step": None if ms_int4 is None else {
                "block_us": round(ms_int4 * 1e3, 2), "value": round(flops_step / (ms_int4 * 1e-3) / 1e12, 2), "unit": UNIT,
                "weight_bytes_per_param": 0.3125,
                "note": "4-bit weights (pair-wise 4:8) and 4-bit activations, exact on the INT8 2:4 path; rank 0 only"},
            "fp16_sparse_step": None if ms_half is None else {
                "block_us": round(ms_half * 1e3, 2), "value": round(flops_step / (ms_half * 1e-3) / 1e12, 2),
                "unit": "TFLOP/s (dense-equivalent)", "layers_us": half_layer_us,
                "frac_of_measured_bf16_sustained_x2": round(flops_step / (ms_half * 1e-3) / 1e12 / (2.0 * peaks["bf16_tflops_sustained"]), 4),
                "note": "the FP16 2:4 sparse model: four gpusq_spgemm_f16 launches on FP16 activations, no quantise node; rank 0 only"},
            "device_status": status_host, "quant_act_status": quant_status,
            "peaks": {k: v for k, v in peaks.items() if k in ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained", "_source")},
        }
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


# ------------------------------------------------------------------- patch-embedding workload
def run_patch_embed(args, pcfg):
    """One step = gpusq_patch_quant (scale computed) + the sparse GEMM on the patch rows, FP16 out.

    A step touches less than L2, so the timed loop walks over enough (image, Xq, Y) buffer sets to
    exceed it; single GPU only (the layer runs once per image batch and shards like any other layer).
    """
    import torch

    from paper_2305_10727_b200 import binding as B

    if int(os.environ.get("WORLD_SIZE", "1")) != 1:
        raise SystemExit("--patch is a single-GPU measurement")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libgpusq has no CPU fallback")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    B.load()
    peaks = load_peaks()
    h = inputs.make_patch_inputs(pcfg)
    T, K, Kp, D = pcfg.tokens, pcfg.K, pcfg.Kp, pcfg.D
    Wf = B.flatten_conv_weight(torch.from_numpy(h["W4"]).to(dev), Kp)
    Wq, ws = B.quant_weight(B.prune24(Wf))
    vals, meta = B.compress24(Wq)
    Wpk = B.pack24(vals, meta)
    bias = torch.from_numpy(h["bias"]).to(dev)
    img_bytes, xq_bytes, y_bytes = h["img"].size * 2, T * Kp, T * D * 2
    step_bytes = 2 * img_bytes + 2 * xq_bytes + y_bytes          # image read twice, Xq written and read
    nbuf = max(2, int(math.ceil(2.5 * 126e6 / (img_bytes + xq_bytes + y_bytes))))
    img0 = torch.from_numpy(h["img"]).to(dev)
    sets = [dict(img=img0.clone(), Xq=torch.empty((T, Kp), dtype=torch.int8, device=dev),
                 Y=torch.empty((T, D), dtype=torch.float16, device=dev)) for _ in range(nbuf)]
    xs = torch.empty((1,), dtype=torch.float32, device=dev)
    wsb = torch.zeros((B.quant_act_workspace(T, Kp),), dtype=torch.uint8, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)

    def quant(s, given=False):
        if given:
            B.patch_quant(s["img"], pcfg.P, Kp, s["Xq"], xs, scale_mode=B.SCALE_GIVEN)
        else:
            B.patch_quant(s["img"], pcfg.P, Kp, s["Xq"], xs, workspace=wsb)

    def gemm(s):
        B.spgemm_i8(s["Xq"], Wpk, D, ws, xs, bias, out_type=B.OUT_F16, Y=s["Y"], status_buf=status)

    stream = torch.cuda.Stream()
    torch.cuda.set_stream(stream)
    replays = max(1, int(math.ceil(args.steps / nbuf)))
    steps = replays * nbuf

    def loop_ms(fn):
        """Milliseconds per step of `fn(set)` run over all buffer sets, replayed from a graph."""
        for s in sets[:2]:
            fn(s)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for s in sets:
                fn(s)
        for _ in range(max(3, int(math.ceil(max(args.warmup, 3) / nbuf)))):
            g.replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        for _ in range(replays):
            g.replay()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / steps

    sampler = ClockSampler(0)
    sampler.start()
    ms_step = loop_ms(lambda s: (quant(s), gemm(s)))
    clocks = sampler.stop()
    ms_quant = loop_ms(quant)
    ms_quant_given = loop_ms(lambda s: quant(s, True))
    ms_gemm = loop_ms(gemm)
    ms_given_step = loop_ms(lambda s: (quant(s, True), gemm(s)))
    flops = 2.0 * T * K * D                                     # Sec. 3.3: 2 N C H W D_embed
    value = flops / (ms_step * 1e-3) / 1e12

    # ---- end to end: image batch from pinned host memory in, embeddings out, every step
    e2e = None
    if not args.no_e2e:
        pin_in = torch.from_numpy(h["img"]).pin_memory()
        pin_out = torch.empty((T, D), dtype=torch.float16).pin_memory()
        s0 = sets[0]

        def e2e_step():
            s0["img"].copy_(pin_in, non_blocking=True)
            quant(s0)
            gemm(s0)
            pin_out.copy_(s0["Y"], non_blocking=True)

        for _ in range(3):
            e2e_step()
        torch.cuda.synchronize()
        n_e2e = 20
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        b.record(stream)
        torch.cuda.synchronize()
        ms_e2e = a.elapsed_time(b) / n_e2e
        e2e = {"value": round(flops / (ms_e2e * 1e-3) / 1e12, 2), "unit": UNIT, "h2d_bytes_per_step": img_bytes,
               "d2h_bytes_per_step": y_bytes, "ms_per_step": round(ms_e2e, 4), "steps": n_e2e}
    status_host = status.cpu().tolist()

    # ---- CPU baseline: the oracle on the first images of the batch
    cpu_baseline = None
    if not args.no_cpu_baseline:
        import oracle
        nb = max(1, min(pcfg.B, int(3e9 // (float(T // pcfg.B) * Kp * D))))      # about 3 G multiply-adds
        prep = oracle.patch_embed_weight(h["W4"], Kp)
        t0 = time.perf_counter()
        oracle.patch_embed_forward(h["img"][:nb], prep, pcfg.P, h["bias"])
        t_cpu = time.perf_counter() - t0
        cpu_baseline = {"value": flops * nb / pcfg.B / t_cpu / 1e12, "unit": UNIT, "cores": 1, "kind": "oracle",
                        "sample": "first %d of %d images (quantise + patch rows + GEMM + epilogue), %.1f s"
                                  % (nb, pcfg.B, t_cpu)}

    quant_bytes = 2 * img_bytes + xq_bytes                       # maximum pass + quantise pass
    line = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": 1, "steps": steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms_step, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": pcfg.name, "images": pcfg.B, "C": pcfg.C, "H": pcfg.H, "W": pcfg.W, "P": pcfg.P,
                   "tokens": T, "K": K, "K_padded": Kp, "D": D,
                   "step": "gpusq_patch_quant (scale computed: 2 launches) + sparse GEMM with fused epilogue, FP16 out",
                   "launch": "graph", "l2": "the loop walks over %d buffer sets, %.0f MB" % (nbuf, nbuf * (img_bytes + xq_bytes + y_bytes) / 1e6),
                   "parallelism": "single GPU"},
        "roofline": {"bound": "hbm", "kernel": "act_absmax_kernel + patch_quant_kernel",
                     "achieved": round(quant_bytes / (ms_quant * 1e-3) / 1e9, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": round(quant_bytes / (ms_quant * 1e-3) / 1e9 / peaks["hbm_gbs"], 4), "traffic": None,
                     "peak_source": "%s copy bandwidth" % peaks["_source"],
                     "timing": "CUDA events around %d graph replays of the two launches alone over the buffer sets" % replays,
                     "patch_quant_us": round(ms_quant * 1e3, 2), "patch_quant_given_us": round(ms_quant_given * 1e3, 2),
                     "gemm_us": round(ms_gemm * 1e3, 2),
                     "gemm_tops": round(flops / (ms_gemm * 1e-3) / 1e12, 1),
                     "step_hbm_gbs": round(step_bytes / (ms_step * 1e-3) / 1e9, 1)},
        "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": 3 * steps, "clocks": clocks,
        "static_scale_step": {"us": round(ms_given_step * 1e3, 2), "note": "same step with a supplied image scale: 2 launches"},
        "device_status": status_host,
        "peaks": {k: v for k, v in peaks.items() if k in ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained", "_source")},
    }
    print(json.dumps(line))


# ------------------------------------------------------------------- time per tile of a few CTA pairs
def run_tile_sweep(args, cfg):
    """Time per output tile of one CTA pair, with and without the other SMs' traffic.

    The GEMM launches are held to `pairs` CTA pairs (measurement hook of gpusq_testing.h) and the
    tokens are cut so that every pair works on 8 and then on 16 tiles of 224 tokens: the difference
    is eight tile periods in steady state, the rest the launch's fixed cost.  `pairs` = 9 leaves
    130 of 148 SMs idle (what one pair can do by itself); `pairs` = all is the loaded GPU.  One JSON
    line; single GPU; not a throughput figure.
    """
    import torch

    from paper_2305_10727_b200 import binding as B

    if int(os.environ.get("WORLD_SIZE", "1")) != 1:
        raise SystemExit("--tile-sweep is a single-GPU measurement")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libgpusq has no CPU fallback")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    B.load()
    stream = torch.cuda.Stream()
    torch.cuda.set_stream(stream)
    block_t = 224
    B.set_block_tokens(block_t)
    sm_mhz = None

    def timed_us(fn, nbuf):
        for i in range(nbuf):
            fn(i)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(nbuf):
                fn(i)
        for _ in range(max(3, args.warmup)):
            g.replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        for _ in range(10):
            g.replay()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / (10 * nbuf) * 1e3

    all_pairs = torch.cuda.get_device_properties(dev).multi_processor_count // 2
    rows = []
    sampler = ClockSampler(0)
    sampler.start()
    try:
        # the layers of the block, and one shape whose main loop is two k blocks: the epilogue alone
        short = collections.namedtuple("Shape", "name N K")("k256", cfg.layers[0].N, 256)
        for L in list(cfg.layers) + [short]:
            d = inputs.random_layer(1000 + L.N + L.K, 64, L.N, L.K)
            Wq, ws = B.quant_weight(B.prune24(torch.from_numpy(d["W"]).to(dev)))
            Wpk = B.pack24(*B.compress24(Wq))
            bias = torch.from_numpy(d["bias"]).to(dev)
            cols = (L.N + 255) // 256
            xs = torch.tensor([0.01], dtype=torch.float32, device=dev)
            osc = torch.tensor([0.05], dtype=torch.float32, device=dev)
            status = torch.zeros(4, dtype=torch.int32, device=dev)
            for kind, act, ot in (("f16", 0, B.OUT_F16), ("f16+gelu", 1, B.OUT_F16), ("i8", 0, B.OUT_I8)):
                for pairs in (9, all_pairs):
                    B.set_max_clusters(pairs)
                    t = []
                    for per_pair in (8, 16):
                        # tiles = cols x token tiles = pairs x per_pair
                        tok_tiles = max(1, (pairs * per_pair) // cols)
                        M = tok_tiles * block_t
                        Xq = torch.randint(-127, 128, (M, L.K), dtype=torch.int8, device=dev)
                        odt = torch.float16 if ot == B.OUT_F16 else torch.int8
                        Y = [torch.empty((M, L.N), dtype=odt, device=dev) for _ in range(4)]
                        t.append((timed_us(lambda i: B.spgemm_i8(Xq, Wpk, L.N, ws, xs, bias, act=act, out_type=ot,
                                                                  out_scale=osc, Y=Y[i], status_buf=status), 4),
                                  -(-(cols * tok_tiles) // pairs)))
                    per_tile = (t[1][0] - t[0][0]) / (t[1][1] - t[0][1])
                    rows.append({"layer": L.name, "N": L.N, "K": L.K, "out": kind, "pairs": pairs,
                                 "us_8_tiles": round(t[0][0], 2), "us_16_tiles": round(t[1][0], 2),
                                 "tiles_per_pair": [t[0][1], t[1][1]],
                                 "us_per_tile": round(per_tile, 3), "fixed_us": round(t[0][0] - per_tile * t[0][1], 2)})
            if status.cpu().tolist() != [0, 0, 0, 0]:
                raise SystemExit("device status %s" % status.cpu().tolist())
    finally:
        B.set_max_clusters(0)
        B.set_block_tokens(0)
        clocks = sampler.stop()
    for r in rows:
        if clocks.get("sm_mhz"):
            r["cycles_per_tile"] = int(round(r["us_per_tile"] * clocks["sm_mhz"]))
    print(json.dumps({"tile_sweep": rows, "block_tokens": block_t, "config": {"workload": args.config},
                      "clocks": clocks, "note": "time per 256-feature x 224-token tile of one CTA pair: (t(16 tiles) - t(8 tiles)) / 8"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="gpusq", choices=["gpusq", "reference"])
    ap.add_argument("--config", default="deit_base_b64", choices=inputs.config_names())
    ap.add_argument("--patch", default=None, choices=list(inputs.PATCH_CONFIGS),
                    help="measure a patch-embedding workload instead of a block of linear layers")
    ap.add_argument("--launch", default="graph", choices=["graph", "eager"])
    ap.add_argument("--ref-rows", type=int, default=8192,
                    help="token rows per layer the CPU oracle is timed on with all host cores (a quarter of them on one core)")
    ap.add_argument("--ref-rows-reference", type=int, default=0,
                    help="token rows per step for --impl reference (0 = size from a calibration run)")
    ap.add_argument("--tile-sweep", action="store_true",
                    help="time per output tile of one CTA pair on 9 pairs and on all of them (measurement aid, not a throughput figure)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    cfg = inputs.CONFIGS[args.config]
    if args.tile_sweep and args.impl == "gpusq":
        run_tile_sweep(args, cfg)
        return
    if args.patch is not None and args.impl == "gpusq":
        run_patch_embed(args, inputs.PATCH_CONFIGS[args.patch])
        return
    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) != 0:
            return
        args.ref_rows = args.ref_rows_reference
        run_reference(args, cfg)
    else:
        run_gpusq(args, cfg)


if __name__ == "__main__":
    main()
