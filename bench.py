#!/usr/bin/env python
"""Benchmark of the LQER / L2QER inference linear layer on B200.

One step = one pass of the whole hot path over the LLaMA-7B-shaped decoder linear stack
(32 layers x {q,k,v,o: 4096x4096; gate,up: 4096x11008; down: 11008x4096}, MXINT4 weights,
MXINT8 activations, block 16, rank 32): the 224 linears at M=1 (decode) and then at M=2048
(prefill), back to back on one stream through lqer_linear_batched.  Weights, factors and
activations are seeded synthetic draws of the paper's shapes and value structure.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--layers L]

Prints ONE JSON line (rank 0).  `value` is the whole-job TFLOP/s of the timed steps
(algorithmic flops 2 M [(K + k) N + K k] per linear); the decode and prefill legs of the same
steps are reported separately, as are the end-to-end figure through host buffers, the
roofline of the dominant kernel and the CPU oracle timed on a bounded sample.
"""
from __future__ import annotations

import argparse
import dataclasses
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import lqer_inputs as gen

METRIC = "fused W4A8+low-rank linear: prefill TOPS & % MMA peak; decode us/layer & HBM GB/s"
WORKLOAD = ("LLaMA-7B-shaped decoder linear stack: 32 layers x {q,k,v,o 4096x4096; gate,up 4096x11008; "
            "down 11008x4096}, MXINT4/MXINT8 block 16, rank 32, M=1 then M=2048 back to back on one stream")
M_DECODE, M_PREFILL = 1, 2048

# DRAM traffic of one launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum
# from an ncu capture) per shape, valid only for the kernel sources whose hash is given.
TRAFFIC = {"sources_sha256": "50984f2c583415ea", "bytes_per_launch": 737.0e6,
           "note": "644.9 MB measured on one launch of the seven linears of a decoder layer, scaled to the eight linears "
                   "of a bench launch (profiles/gemm_tc2_kernel_7b_layer.md)"}
DOMINANT_SOURCES = ["paper_2402_02446_b200/csrc/lqer_gemm_tc2.cu", "paper_2402_02446_b200/csrc/lqer_tc_ptx.cuh"]


def sources_hash(sources=None) -> str:
    h = hashlib.sha256()
    for rel in (DOMINANT_SOURCES if sources is None else sources):
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


# The same for the HBM-bound kernels: measured DRAM bytes over algorithmic bytes of the captured launch (the traffic
# grows in proportion to the bytes a launch streams), valid for the sources whose hash is given.
TRAFFIC_RATIO = {
    "decode": {"sources": ["paper_2402_02446_b200/csrc/lqer_decode_cols.cu", "paper_2402_02446_b200/csrc/lqer_common.cuh"],
               "sha256": "9934eeedd710cc07", "ratio": 254.9 / 250.5, "note": "profiles/decode_cols_kernel_7b_layer.md"},
    "prologue": {"sources": ["paper_2402_02446_b200/csrc/lqer_prologue_tc.cu", "paper_2402_02446_b200/csrc/lqer_common.cuh"],
                 "sha256": "a2bf7fc29e22ad24", "ratio": 411.6 / 438.2, "note": "profiles/prologue_tc_kernel_7b_layer.md"},
}


def traffic_of(kernel: str, algorithmic_bytes_per_launch: float):
    t = TRAFFIC_RATIO[kernel]
    if t["ratio"] is None or t["sha256"] != sources_hash(t["sources"]):
        return None
    return t["ratio"] * algorithmic_bytes_per_launch


def layer_flops(M: int, K: int, N: int, k: int) -> float:
    return 2.0 * M * ((K + k) * N + K * k)


W_BITS = 4          # mantissa bits of W_q of this run (--w-bits)


def layer_weight_bytes(K: int, N: int, k: int) -> float:
    """Algorithmic bytes of the stored operands: w_bits + 1 exponent byte per 16 for W_q,
    8-bit + 1 exponent byte per 16 for A_k and B_k (rank padded to a multiple of 16)."""
    k_pad = (k + 15) // 16 * 16
    return (W_BITS / 8.0 + 0.0625) * K * N + 1.0625 * (k * K + k_pad * N)


def measured_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled every 100 ms while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device: int):
        self.proc = None
        try:
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.proc = subprocess.Popen(["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, pw = [], [], []
        reasons = set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); pw.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(pw), "samples": len(sm),
                "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ reference arm
def oracle_sample(rows: int, a_bits: int = 8, w_bits: int = 4, rank=None):
    """The bounded sample the oracle is timed on: layer 0's q, gate and down linears, `rows` tokens
    of the M=2048 batch.  Returns (callable running the sample once, flops of one run, description)."""
    from oracle import lqer as olqer
    work = []
    flops = 0.0
    for which in (0, 4, 6):
        spec = gen.config_stack(0, which, M_PREFILL)
        if rank is not None:
            spec = dataclasses.replace(spec, k=rank)
        W = gen.make_weight(spec)
        A, B = gen.make_random_factors(spec)
        P = olqer.prepare_weights(W, A, B, w_bits=w_bits)
        X = gen.make_activations(spec, M=rows)
        work.append((X, P, W, A, B))
        flops += layer_flops(rows, spec.K, spec.N, spec.k)
    def run():
        return [olqer.forward(X, P, w_bits=w_bits, a_bits=a_bits) for X, P, _, _, _ in work]
    run.work = work
    return run, flops, f"layer 0 q, gate, down linears, {rows} rows of the M={M_PREFILL} batch"


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [int(p.get("num_threads", 1)) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def time_oracle(steps: int, warmup: int, rows: int, a_bits: int = 8, check=None, w_bits: int = 4, rank=None):
    """TFLOP/s and milliseconds per run of the oracle on its bounded sample.  check(work, results), if given, is
    called with the sample's inputs and the oracle's results of the last run (the GPU arm compares its own
    output on the same inputs with them)."""
    run, flops, what = oracle_sample(rows, a_bits, w_bits, rank)
    for _ in range(warmup):
        run()
    t0 = time.perf_counter()
    res = None
    for _ in range(steps):
        res = run()
    dt = (time.perf_counter() - t0) / max(steps, 1)
    extra = check(run.work, res) if check is not None else None
    return flops / dt / 1e12, dt * 1e3, what, extra


def run_reference(args) -> None:
    if int(os.environ.get("RANK", "0")) != 0:
        return
    steps, warmup = max(args.steps, 1), max(args.warmup, 0)
    tflops, ms, what, _ = time_oracle(steps, warmup, rows=args.oracle_rows, a_bits=args.a_bits, w_bits=args.w_bits, rank=args.rank)
    cores = blas_threads()
    line = {"impl": "reference", "metric": METRIC, "value": tflops, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": what},
            "cpu_baseline": {"value": tflops, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": what},
            "e2e": {"value": tflops, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def max_over_ranks(values, dist, device):
    """Element-wise maximum of per-rank timings over all ranks (the job is as slow as its slowest rank);
    the values themselves when the job has one rank (dist is None)."""
    if dist is None:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_value(flops_per_rank_step: float, ms_per_step: float, world: int) -> float:
    """TFLOP/s of the whole job: every rank runs its own replica of the step (weak scaling)."""
    return world * flops_per_rank_step / (ms_per_step * 1e-3) / 1e12



# ------------------------------------------------------------------------------------------ the other workloads
def time_calls(fn, iters: int, warmup: int = 3) -> float:
    """Microseconds per call of fn(i), i = 0 .. iters - 1, timed with CUDA events on the current stream."""
    stream = torch.cuda.current_stream()
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(iters):
        fn(i)
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / iters


def one_launch_per_call_us(L, calls, ws, iters: int, x_t=torch.float32, y_t=torch.float32) -> float:
    """Microseconds for one pass over `calls` (decode-sized) with every call a launch of its own, in stream order, as a
    decoder must run layers that depend on one another.  The loop over the calls runs inside the library, so the
    figure is the device's, not the Python interpreter's."""
    from paper_2402_02446_b200 import binding
    L.set_path(binding.PATH_DECODE)
    try:
        return time_calls(lambda i: L.linear_batched_ex(calls, ws, x_t, y_t), iters)
    finally:
        L.set_path(binding.PATH_AUTO)


def packed_copies(L, spec, cfg, dev, min_bytes: float, k: int | None = None):
    """Distinct packed buffers of one layer (the same numbers at different addresses), at least min_bytes together."""
    W = gen.make_weight_device(spec, dev)
    kk = spec.k if k is None else k
    A = B = None
    if kk > 0:
        sp = gen.LayerSpec(spec.name, spec.M, spec.K, spec.N, kk, spec.calib_rows, spec.outlier_frac, spec.outlier_scale,
                           spec.weight_law, spec.seed)
        A, B = gen.make_random_factors_device(sp, dev)
    out = [L.prepare_weights(W, A, B, cfg)]
    while sum(p.buf.numel() for p in out) < min_bytes:
        out.append(L.prepare_weights(W, A, B, cfg))
    torch.cuda.synchronize()
    return out


def run_other_configs(L, cfg, dev, peaks, quick: bool) -> dict:
    """Driver-run figures for the decode-shaped layer, the two prefill MLP layers and the 13B-shaped rank sweep
    (weights rotated through more than L2 where a layer alone would stay resident)."""
    out = {}
    rot = 272e6                                             # bytes of distinct packed copies a timing loop walks
    hbm, hbm_nom = peaks["hbm_gbs"], 8000.0

    # ---- decode-shaped layer: 4096 x 4096, rank 32, M in {1, 4, 16}
    dec = {}
    for M in (1, 4, 16):
        spec = gen.config_decode(M)
        copies = packed_copies(L, spec, cfg, dev, rot)
        n = len(copies)
        X = gen.make_activations_device(spec, dev)
        Ys = [torch.empty((M, spec.N), dtype=torch.float32, device=dev) for _ in range(n)]
        ws = L.new_workspace(M, copies[0])
        nbytes = layer_weight_bytes(spec.K, spec.N, spec.k) + 4.0 * M * (spec.K + spec.N)
        calls = L.make_calls([(X, c, y) for c, y in zip(copies, Ys)])
        wsb = torch.zeros(max(L.batched_workspace_bytes(calls), ws.numel()), dtype=torch.uint8, device=dev)
        us_lone = one_launch_per_call_us(L, calls, wsb, 4) / n
        us_shared = time_calls(lambda i: L.linear_batched(calls, wsb), 8) / n
        dec[f"M{M}"] = {
            "bytes": nbytes, "copies": n,
            "lone_call": {"us": us_lone, "gbs": nbytes / us_lone * 1e-3, "frac_of_measured_hbm": nbytes / us_lone * 1e-3 / hbm,
                          "frac_of_8tbs": nbytes / us_lone * 1e-3 / hbm_nom},
            "shared_launches": {"us_per_layer": us_shared, "gbs": nbytes / us_shared * 1e-3,
                                "frac_of_measured_hbm": nbytes / us_shared * 1e-3 / hbm,
                                "frac_of_8tbs": nbytes / us_shared * 1e-3 / hbm_nom, "independent_layers": n},
        }
        for c in copies:
            c.release()
        del copies, Ys, ws, wsb
    out["decode_layer_4096x4096_k32"] = dec

    # ---- prefill MLP layers alone: M = 2048, 4096 x 11008 and 11008 x 4096, rank 32
    pre = {}
    for transposed in (False, True):
        spec = gen.config_prefill(transposed)
        copies = packed_copies(L, spec, cfg, dev, 0)
        Xs = [gen.make_activations_device(spec, dev) for _ in range(2)]
        Y = torch.empty((spec.M, spec.N), dtype=torch.float32, device=dev)
        ws = L.new_workspace(spec.M, copies[0])
        us = time_calls(lambda i: L.linear(Xs[i & 1], copies[0], ws, Y), 20)
        fl = layer_flops(spec.M, spec.K, spec.N, spec.k)
        pre[spec.name] = {"K": spec.K, "N": spec.N, "M": spec.M, "us": us, "tflops": fl / us * 1e-6,
                          "frac_of_measured_bf16_burst": fl / us * 1e-6 / peaks["bf16_tflops"],
                          "frac_of_measured_bf16_sustained": fl / us * 1e-6 / peaks["bf16_tflops_sustained"]}
        copies[0].release()
        del copies, Xs, Y, ws
    out["prefill_mlp_M2048_k32"] = pre

    # ---- 13B-shaped sweep: K = 5120, low-rank overhead against rank
    sweep = []
    Ns = gen.SWEEP_N
    Ms = (1, 512) if quick else gen.SWEEP_M
    for N in Ns:
        for M in Ms:
            base_us = None
            for k in (0,) + gen.SWEEP_K_RANK:
                spec = gen.config_sweep(N, M, gen.SWEEP_K_RANK[0] if k == 0 else k)
                copies = packed_copies(L, spec, cfg, dev, rot if M <= 64 else 0, k=k)
                n = len(copies)
                X = gen.make_activations_device(spec, dev)
                Y = torch.empty((M, N), dtype=torch.float32, device=dev)
                ws = L.new_workspace(M, copies[0])
                if M <= 16:
                    calls = L.make_calls([(X, c, Y) for c in copies])
                    us = one_launch_per_call_us(L, calls, ws, 3) / n
                else:
                    iters = max(8, 2 * n) if M <= 64 else (12 if M <= 512 else 6)
                    us = time_calls(lambda i: L.linear(X, copies[i % n], ws, Y), iters)
                if k == 0:
                    base_us = us
                K = spec.K
                row = {"N": N, "M": M, "k": k, "us": us, "overhead_vs_k0": us / base_us - 1.0,
                       "analytic_flop_overhead": k * (K + N) / (K * N),
                       "analytic_byte_overhead": 1.0625 * ((k + 15) // 16 * 16) * (K + N) / (0.5625 * K * N)}
                if M >= 512:
                    row["tflops"] = layer_flops(M, K, N, k) / us * 1e-6
                else:
                    nb = layer_weight_bytes(K, N, k) + 4.0 * M * (K + N)
                    row["gbs"] = nb / us * 1e-3
                    row["roofline_us"] = max(nb / (hbm * 1e3), layer_flops(M, K, N, k) / (peaks["bf16_tflops"] * 1e6))
                sweep.append(row)
                for c in copies:
                    c.release()
                del copies, X, Y, ws
    out["sweep_13b_K5120"] = sweep
    return out


# ------------------------------------------------------------------------------------------ GPU arm
def run_ours(args) -> None:
    import paper_2402_02446_b200 as L

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # ---- build the stack (untimed): one packed buffer per linear, its own activations
    layers = args.layers
    cfg = L.default_config()
    cfg.a_bits = args.a_bits
    cfg.w_bits = args.w_bits
    packed, shapes = [], []
    for layer in range(layers):
        for which in range(len(gen.STACK_LINEARS)):
            spec = gen.config_stack(layer, which, M_PREFILL)
            if args.rank is not None:
                spec = dataclasses.replace(spec, k=args.rank)
            W = gen.make_weight_device(spec, dev)
            A, B = gen.make_random_factors_device(spec, dev)
            packed.append(L.prepare_weights(W, A, B, cfg))
            shapes.append((spec.K, spec.N, spec.k, spec))
            del W, A, B
    torch.cuda.synchronize()
    n_lin = len(packed)
    Kmax = max(s[0] for s in shapes)
    ws_bytes = max(L.workspace_bytes(M_PREFILL, K, N, k) for K, N, k, _ in shapes)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    L.lib().lqer_workspace_init(ws.data_ptr(), ws_bytes, int(torch.cuda.current_stream().cuda_stream))

    # element types at the boundary: X fp32 or bf16; Y fp32, bf16, or re-quantised to MXINT8 (17 bytes per 16 elements)
    x_t = torch.float32 if args.io == "f32" else L.MXINT8 if args.io == "mxint8" else torch.bfloat16
    y_t = torch.float32 if args.io == "f32" else torch.bfloat16 if args.io == "bf16" else L.MXINT8
    x_b = 4.0 if args.io == "f32" else 17.0 / 16.0 if args.io == "mxint8" else 2.0
    y_b = 4.0 if args.io == "f32" else 2.0 if args.io == "bf16" else 17.0 / 16.0

    def as_x(Xf):
        """An fp32 activation tensor in the element type of the run (MXINT8: quantised by the library's own routine)."""
        if x_t == L.MXINT8:
            Xm, Xe = L.quantize_activations(Xf if Xf.is_cuda else Xf.to(dev), cfg)
            buf = L.to_mxint8(Xm, Xe)
            return buf if Xf.is_cuda else buf.cpu()
        return Xf.to(x_t)

    def new_y(M, N, device=dev):
        if y_t == L.MXINT8:
            return torch.empty(L.mxint8_bytes(M, N), dtype=torch.uint8, device=device)
        return torch.empty((M, N), dtype=y_t, device=device)

    X1 = [as_x(gen.make_activations_device(s[3], dev, M=M_DECODE)) for s in shapes]
    X2 = [as_x(gen.make_activations_device(s[3], dev, M=M_PREFILL)) for s in shapes]
    # outputs: one buffer per linear type and M (write-only; each is larger than a tile's reuse window)
    Y1 = [new_y(M_DECODE, N) for _, N, _, _ in shapes]
    Y2_by_type = [new_y(M_PREFILL, gen.STACK_LINEARS[w][2]) for w in range(len(gen.STACK_LINEARS))]
    Y2 = [Y2_by_type[j % len(gen.STACK_LINEARS)] for j in range(n_lin)]
    decode_calls = L.make_calls(zip(X1, packed, Y1), x_t, y_t)
    prefill_calls = L.make_calls(zip(X2, packed, Y2), x_t, y_t)
    # room for the shared launches of same-shape neighbours (one Xcat slice per layer of a group)
    ws_bytes = max(ws_bytes, L.batched_workspace_bytes(decode_calls), L.batched_workspace_bytes(prefill_calls))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    L.lib().lqer_workspace_init(ws.data_ptr(), ws_bytes, int(torch.cuda.current_stream().cuda_stream))

    flops_decode = sum(layer_flops(M_DECODE, K, N, k) for K, N, k, _ in shapes)
    flops_prefill = sum(layer_flops(M_PREFILL, K, N, k) for K, N, k, _ in shapes)
    bytes_decode = sum(layer_weight_bytes(K, N, k) + (x_b * K + y_b * N) * M_DECODE for K, N, k, _ in shapes)

    stream = torch.cuda.current_stream()

    def step(mid_event=None):
        L.linear_batched_ex(decode_calls, ws, x_t, y_t)
        if mid_event is not None:
            mid_event.record(stream)
        L.linear_batched_ex(prefill_calls, ws, x_t, y_t)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    if L.poll_status(ws) != 0:
        raise SystemExit("device-side error during warm-up")

    # ---- timed region: exactly K steps, events on the launching stream
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = L.launch_count()
    barrier()
    t_start = torch.cuda.Event(enable_timing=True)
    t_stop = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for e0, e1, e2 in ev:
        e0.record(stream)
        step(e1)
        e2.record(stream)
    t_stop.record(stream)
    barrier()
    launches = L.launch_count() - launches0
    clocks = sampler.stop() if sampler is not None else None
    total_ms = t_start.elapsed_time(t_stop)
    decode_ms = [e0.elapsed_time(e1) for e0, e1, _ in ev]
    prefill_ms = [e1.elapsed_time(e2) for _, e1, e2 in ev]
    total_ms, dec_ms, pre_ms = max_over_ranks([total_ms, statistics.median(decode_ms), statistics.median(prefill_ms)], dist, dev)
    if L.poll_status(ws) != 0:
        raise SystemExit("device-side error during the timed region")
    ms_per_step = total_ms / args.steps
    value = whole_job_value(flops_decode + flops_prefill, ms_per_step, world)

    # ---- roofline of the dominant kernel: one more step with an event pair around every launch
    peaks = measured_peaks()
    L.profile_enable(True)
    step()
    torch.cuda.synchronize()
    fam = L.profile_collect()
    L.profile_enable(False)
    fam_total = sum(ms for _, ms in fam.values())
    dominant = max(fam, key=lambda n: fam[n][1])
    dom_launches, dom_ms = fam[dominant]
    roofline = None
    if dominant.startswith("gemm"):
        # every M=2048 linear goes through this kernel, up to eight neighbours in one launch;
        # algorithmic flops per launch = all of them / the launches counted
        flops_per_launch = sum(2.0 * M_PREFILL * (K + k) * N for K, N, k, _ in shapes) / dom_launches
        achieved = flops_per_launch / (dom_ms / dom_launches * 1e-3) / 1e12
        peak = peaks["bf16_tflops_sustained"]
        traffic = TRAFFIC["bytes_per_launch"] if TRAFFIC["sources_sha256"] == sources_hash() else None
        roofline = {"bound": "tensor", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                    "frac": achieved / peak, "peak_source": f"bf16 cuBLAS sustained, {peaks['source']}",
                    "frac_of_burst_peak": achieved / peaks["bf16_tflops"], "frac_of_nominal_2250": achieved / 2250.0,
                    "traffic": traffic, "avg_launch_us": dom_ms / dom_launches * 1e3, "launches": dom_launches,
                    "share_of_kernel_time": dom_ms / fam_total}
    kernels = {n: {"launches": c, "ms": round(ms, 4), "share": round(ms / fam_total, 4)} for n, (c, ms) in fam.items()}
    # one entry per bound: the tensor-bound GEMM above, the HBM-bound decode kernels and the HBM-bound activation prologue
    rooflines = {"tensor_gemm": roofline}
    if "decode" in fam:
        c, ms = fam["decode"]
        ach = bytes_decode / (ms * 1e-3) / 1e9
        rooflines["hbm_decode"] = {"bound": "hbm", "kernel": "decode (column-owner kernel, 16 layers per launch, + activations ahead)",
                                   "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                                   "frac_of_8tbs": ach / 8000.0, "peak_source": f"copy bandwidth, {peaks['source']}",
                                   "launches": c, "avg_launch_us": ms / c * 1e3,
                                   "traffic": traffic_of("decode", bytes_decode / c)}
    if "prologue" in fam:
        c, ms = fam["prologue"]
        pb = sum(float(x_b) * M_PREFILL * K + 2.0 * M_PREFILL * ((K + 63) // 64 * 64 + (k + 15) // 16 * 16) for K, N, k, _ in shapes)
        ach = pb / (ms * 1e-3) / 1e9
        rooflines["hbm_prologue"] = {"bound": "hbm", "kernel": "prologue (activation quantisation + low-rank projection)",
                                     "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                                     "frac_of_8tbs": ach / 8000.0, "peak_source": f"copy bandwidth, {peaks['source']}",
                                     "launches": c, "avg_launch_us": ms / c * 1e3, "traffic": traffic_of("prologue", pb / c)}

    # ---- the decode leg with every linear a launch of its own (stream order, as layers that depend on one another run)
    dep_us = one_launch_per_call_us(L, decode_calls, ws, max(2, min(args.steps, 5)), x_t, y_t)
    (dep_us,) = max_over_ranks([dep_us], dist, dev)
    decode_dependent = {"us_per_linear": dep_us / n_lin, "us_per_decoder_layer": dep_us / layers,
                        "hbm_gbs": bytes_decode / dep_us * 1e-3,
                        "frac_of_measured_hbm": bytes_decode / dep_us * 1e-3 / peaks["hbm_gbs"],
                        "what": "224 linears at M=1, one launch per linear in stream order (no sharing of launches)"}

    # ---- the other workloads (one GPU, rank 0's figures)
    other = None
    if not args.no_configs:
        other = run_other_configs(L, cfg, dev, peaks, quick=args.quick_configs)

    # ---- end to end through host buffers (pinned), copies inside the timed region
    e2e = None
    if not args.no_e2e:
        types = len(gen.STACK_LINEARS)
        hx1 = [as_x(torch.randn((M_DECODE, gen.STACK_LINEARS[w][1]))).pin_memory() for w in range(types)]
        hx2 = [as_x(torch.randn((M_PREFILL, gen.STACK_LINEARS[w][1]))).pin_memory() for w in range(types)]
        hy1 = [new_y(M_DECODE, gen.STACK_LINEARS[w][2], "cpu").pin_memory() for w in range(types)]
        hy2 = [new_y(M_PREFILL, gen.STACK_LINEARS[w][2], "cpu").pin_memory() for w in range(types)]
        calls1 = L.make_host_calls([(hx1[j % types], packed[j], hy1[j % types]) for j in range(n_lin)], x_t, y_t)
        calls2 = L.make_host_calls([(hx2[j % types], packed[j], hy2[j % types]) for j in range(n_lin)], x_t, y_t)
        ws_h = torch.empty(max(L.linear_host_batched_bytes(calls1), L.linear_host_batched_bytes(calls2)),
                           dtype=torch.uint8, device=dev)
        L.lib().lqer_workspace_init(ws_h.data_ptr(), ws_h.numel(), int(stream.cuda_stream))

        def e2e_step():
            # every layer's X goes host -> device and its Y device -> host inside the call; the copies of
            # neighbouring layers overlap the layer that is running
            L.linear_host_batched_ex(calls1, ws_h, x_t, y_t, stream)
            L.linear_host_batched_ex(calls2, ws_h, x_t, y_t, stream)

        e2e_step()
        barrier()
        e_steps = max(1, min(args.steps, 2))
        t0 = time.perf_counter()
        for _ in range(e_steps):
            e2e_step()
        barrier()
        e_ms = (time.perf_counter() - t0) * 1e3 / e_steps
        (e_ms,) = max_over_ranks([e_ms], dist, dev)
        h2d = int(sum(x_b * (M_DECODE + M_PREFILL) * K for K, _, _, _ in shapes))
        d2h = int(sum(y_b * (M_DECODE + M_PREFILL) * N for _, N, _, _ in shapes))
        e2e = {"value": world * (flops_decode + flops_prefill) / (e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
               "ms_per_step": e_ms, "steps": e_steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "api": "lqer_linear_host_batched (224 layers per call, M=1 then M=2048), pinned host X and Y, "
                      "copies pipelined with the layers"}

    # ---- the oracle on the host cores (rank 0, N = 1 only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        def gpu_against_oracle(work, results):
            # the same sample through the library: observed max |Y_gpu - Y_oracle| / tol (the parity bound is 1)
            worst = 0.0
            for (X, P, W, A, B), ref in zip(work, results):
                Pg = L.prepare_weights(torch.from_numpy(W).to(dev), torch.from_numpy(A).to(dev), torch.from_numpy(B).to(dev), cfg)
                wsg = L.new_workspace(X.shape[0], Pg)
                Y = L.linear(torch.from_numpy(X).to(dev), Pg, wsg).cpu().numpy().astype(np.float64)
                worst = max(worst, float(np.max(np.abs(Y - ref.Y) / ref.tol)))
                Pg.release()
            return worst
        tflops, ms, what, worst = time_oracle(1, 0, rows=args.oracle_rows, a_bits=args.a_bits, check=gpu_against_oracle,
                                              w_bits=args.w_bits, rank=args.rank)
        cpu = {"value": tflops, "unit": "TFLOP/s", "cores": blas_threads(), "kind": "oracle", "sample": what,
               "seconds": ms / 1e3, "gpu_max_abs_err_over_tol": worst}

    # ---- weight preparation from W and a calibration batch alone: the GPU's against the oracle's (one 4096 x 4096 layer)
    prep = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import lqer as olqer
        spec = gen.config_decode(1)
        Wn = gen.make_weight(spec)
        cal = gen.make_calibration(spec)
        Wd, cald = torch.from_numpy(Wn).to(dev), [torch.from_numpy(x).to(dev) for x in cal]
        for _ in range(2):
            Pp, _, _, code = L.prepare_from_calibration(Wd, cald, spec.k, cfg=cfg, seed=1)
            Pp.release()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        Pp, _, _, code = L.prepare_from_calibration(Wd, cald, spec.k, cfg=cfg, seed=1)
        torch.cuda.synchronize()
        gpu_s = time.perf_counter() - t0
        Pp.release()
        t0 = time.perf_counter()
        Wm, We = olqer.quantize_weight(Wn, w_bits=args.w_bits)
        E = olqer.quantization_error(Wn, Wm, We, w_bits=args.w_bits)
        sv = olqer.calibration_scale(cal)
        Ao, Bo, _ = olqer.lqer_factors(E, spec.k, sv, method="subspace", rng=np.random.default_rng(1))
        olqer.prepare_weights(Wn, Ao.astype(np.float32), Bo.astype(np.float32), w_bits=args.w_bits)
        cpu_s = time.perf_counter() - t0
        prep = {"what": "W_q, calibration scale, rank-32 factors by subspace iteration, quantise and pack: one 4096 x 4096 layer, "
                        "512 calibration rows", "gpu_ms": gpu_s * 1e3, "oracle_s": cpu_s, "device_status": code,
                "includes": "workspace allocation and the draw of the test matrix on the GPU side"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16 operands (exact MXINT values), fp32 accumulate", "data": "synthetic",
            "config": {"workload": (WORKLOAD if layers == 32 else WORKLOAD + f" [reduced to {layers} layers]") +
                                   ("" if args.a_bits == 8 else f" [activations MXINT{args.a_bits}]") +
                                   ("" if args.w_bits == 4 else f" [weights MXINT{args.w_bits}]") + ("" if args.io == "f32" else " [bf16 X and Y]" if args.io == "bf16" else " [bf16 X, MXINT8 Y]" if args.io == "bf16-mxint8" else " [MXINT8 X and Y]") +
                                   ("" if args.rank is None else f" [rank {args.rank}]"),
                       "linears": n_lin, "M_decode": M_DECODE, "M_prefill": M_PREFILL, "rank": 32 if args.rank is None else args.rank,
                       "a_bits": args.a_bits, "w_bits": args.w_bits, "io": args.io,
                       "shared_launches": "lqer_linear_batched runs consecutive independent calls together: up to 16 "
                                          "decode calls as one launch that divides the SMs among the layers (their "
                                          "activations quantised ahead by one kernel per 64 calls), up to 8 prefill "
                                          "calls as one prologue per layer and one GEMM launch over the tiles of all "
                                          "of them",
                       "l2": "inputs larger than L2: every linear has its own packed weights and activations "
                             f"({sum(p.buf.numel() for p in packed) / 1e9:.2f} GB of weights per step)",
                       "parallelism": "replicas (independent token batches)" if world > 1 else "1 GPU"},
            "prefill": {"tflops": world * flops_prefill / (pre_ms * 1e-3) / 1e12, "ms": pre_ms,
                        "frac_of_measured_bf16_sustained": flops_prefill / (pre_ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                        "us_per_linear": pre_ms * 1e3 / n_lin},
            "decode": {"us_per_linear": dec_ms * 1e3 / n_lin, "us_per_decoder_layer": dec_ms * 1e3 / layers,
                       "hbm_gbs": bytes_decode / (dec_ms * 1e-3) / 1e9,
                       "frac_of_measured_hbm": bytes_decode / (dec_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                       "frac_of_8tbs": bytes_decode / (dec_ms * 1e-3) / 1e9 / 8000.0, "ms": dec_ms,
                       "what": "224 independent linears at M=1, up to 16 per launch",
                       "dependent_order": decode_dependent},
            "roofline": roofline, "rooflines": rooflines, "configs": other, "prepare": prep, "kernels": kernels, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": int(launches), "clocks": clocks, "peaks": peaks,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--layers", type=int, default=32, help="decoder layers of the stack (32 = the full workload)")
    ap.add_argument("--oracle-rows", type=int, default=2048, help="token rows of the oracle's bounded sample")
    ap.add_argument("--a-bits", type=int, default=8, help="mantissa bits of the activations: 8 (W4A8, the workload) or 6 (W4A6)")
    ap.add_argument("--w-bits", type=int, default=4, help="mantissa bits of the weights: 4 (the workload) or 2 (W2A8, Section 4.4)")
    ap.add_argument("--rank", type=int, default=None, help="rank of the correction of every linear (default 32, the workload)")
    ap.add_argument("--io", choices=["f32", "bf16", "bf16-mxint8", "mxint8"], default="f32",
                    help="element types of X and Y at the layer's boundary: f32 (the workload), bf16 (16-bit activations, "
                         "Section 2.1), bf16 X with Y re-quantised to MXINT8 by the epilogue, or MXINT8 both ways (w&a setting: "
                         "17 bytes per 16 activations)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the decode-layer, prefill-MLP and rank-sweep legs")
    ap.add_argument("--quick-configs", action="store_true", help="rank sweep at M = 1 and 512 only")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    global W_BITS
    W_BITS = args.w_bits
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
