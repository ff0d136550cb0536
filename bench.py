#!/usr/bin/env python
"""Benchmark of the format-disaggregated quantized linear layer on B200.

One step = one pass of the serving hot path over one batch of synthetic input on
one packed layer: dq_prefill_quantize + dq_prefill_gemm (NVFP4 prefill linear for
M tokens) followed by dq_decode_linear (LUT3 decode, batch 1).  Packing is a
load-time operation; it is timed once and reported as `pack_ms`.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs an
independent replica of the same workload; there is no data-path collective.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

import numpy as np
import torch

import dq_inputs

METRIC = "NVFP4 prefill GEMM TFLOP/s & LUT3 decode GEMV GB/s, % of B200 roofline"
DEFAULT_WORKLOAD = "c3_gate_up27b"
L2_BYTES = 126 * 1024 * 1024

# DRAM bytes per launch measured with ncu (dram__bytes_read.sum + dram__bytes_write.sum) on the kernel named in the
# roofline object of the same line.  None = not captured for that workload.
NCU_TRAFFIC_BYTES = {
    ("gemm", "c3_gate_up27b"): 80.95e6 + 239.5e6,     # gemm_nvfp4_pair_kernel, full size (one-pass launch list)
    ("gemv", "c3_gate_up27b"): 39.04e6,               # gemv_lut_kernel<3, 640, 1, 1, true>, full size, batch 1 (reads; writes are 35 KB)
    ("gemv_nvfp4", "c3_gate_up27b"): 50.19e6,         # gemv_nvfp4_mma_kernel<640, 3>, full size (one-pass launch list)
}
NOMINAL_FP4_TFLOPS = 9000.0                            # dense FP4, 4 x the 2250 TFLOP/s bf16 figure
NOMINAL_HBM_GBS = 8000.0


def load_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_burst": float(d["bf16_tflops"]),
                "bf16_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs."""

    def __init__(self, device_index: int, period_s: float = 0.001):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        self.h = None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            props = torch.cuda.get_device_properties(device_index)
            h = None
            uuid = getattr(props, "uuid", None)
            if uuid is not None:
                try:
                    h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
                except Exception:
                    h = None
            if h is None:
                vis = os.environ.get("CUDA_VISIBLE_DEVICES")
                phys = int(vis.split(",")[device_index]) if vis and vis.split(",")[device_index].isdigit() else device_index
                h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.h = h
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.h = None

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def oracle_sample_run(cfg, W_f32, ref, A_f32, sa, X_f32, rows):
    """One bounded pass of the oracle: `rows` prefill tokens + one decode token."""
    import oracle
    t0 = time.perf_counter()
    oracle.prefill_linear(A_f32[:rows], sa, ref["nvfp4_codes"], ref["nvfp4_scales"], ref["s"])
    t1 = time.perf_counter()
    oracle.decode_linear(X_f32, ref["lut3_planes"], ref["lut3_scales"], ref["s"])
    t2 = time.perf_counter()
    return t1 - t0, t2 - t1


def run_reference(args, cfg):
    """--impl reference: the CPU oracle as it stands, on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    # rows per step: about half a second of oracle work, so that the default 200 steps end within minutes
    rows = args.ref_rows or max(16, min(cfg.M, int(0.5 * 0.05e12 / (2.0 * cfg.N * cfg.K)) // 16 * 16))
    W = dq_inputs.make_weight(cfg)
    W_f32 = dq_inputs.bf16_to_f32_numpy(W)
    A = dq_inputs.make_activations(cfg, rows)
    sa = dq_inputs.static_act_scale(A)
    A_f32 = dq_inputs.bf16_to_f32_numpy(A)
    X_f32 = dq_inputs.bf16_to_f32_numpy(dq_inputs.make_activations(cfg, 1, salt=2))
    ref = oracle.pack_weights(W_f32)
    for _ in range(min(args.warmup, 2)):
        oracle_sample_run(cfg, W_f32, ref, A_f32, sa, X_f32, rows)
    tp = td = 0.0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        a, b = oracle_sample_run(cfg, W_f32, ref, A_f32, sa, X_f32, rows)
        tp += a
        td += b
    total = time.perf_counter() - t0
    tflops = 2.0 * rows * cfg.N * cfg.K * args.steps / tp / 1e12
    dec_bytes = 0.4375 * cfg.N * cfg.K + 2 * cfg.K + 2 * cfg.N + 4
    sample = (f"{rows} of {cfg.M} prefill rows (oracle quantise + dequantise of activations and of the whole N x K layer, "
              f"then numpy's fp64 dgemm: oracle.matmul_nt_lib) + 1 decode token per step")
    line = {
        "impl": "reference", "metric": METRIC, "value": tflops, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "N": cfg.N, "K": cfg.K, "M": cfg.M, "decode_batch": 1, "sample": sample},
        "cpu_baseline": {"value": tflops, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "decode": {"value": dec_bytes * args.steps / td / 1e9, "unit": "GB/s"},
        "e2e": {"value": tflops, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def run_stack(args):
    """--workload c4_stack27b: the 64-layer 27B-class linear stack (fused qkv, o, fused gate/up, down per
    layer; 23.15 G weights).  One step = one prefill pass of M = 4096 tokens through all 256 matrices
    (activation quantiser + FP4 GEMM each; fresh N(0,1) input per matrix shape, no attention or
    non-linearity in between) plus one decode token step over the same stack, replayed from one CUDA
    graph as the paper measured decode (App. C.2).  Weights are drawn on the GPU (seeded) one matrix at a
    time and packed immediately; the 23 GB packed stack is far larger than L2."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    import __graft_entry__ as g
    if rank == 0:
        g.build()
    if world > 1:
        dist.barrier()
    import paper_2609_26333_b200 as dq
    from paper_2609_26333_b200 import replicas
    peaks = load_peaks()
    M, B = dq_inputs.C4_PREFILL_M, args.decode_batch
    layers = args.layers or dq_inputs.C4_LAYERS
    gen = torch.Generator(device=dev)
    stack = []
    t0 = time.perf_counter()
    for layer in range(layers):
        for cfg in dq_inputs.c4_fused_layer(layer):
            gen.manual_seed(dq_inputs.seed_of(cfg, layer))
            W = (torch.randn(cfg.N, cfg.K, generator=gen, device=dev, dtype=torch.float32) * cfg.w_std).to(torch.bfloat16)
            stack.append((cfg, dq.pack_weights(W)))
            del W
    torch.cuda.synchronize()
    pack_s = time.perf_counter() - t0
    Ks = sorted({c.K for c, _ in stack})
    Ns = sorted({c.N for c, _ in stack})
    gen.manual_seed(4242)
    A = {k: torch.randn(M, k, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16) for k in Ks}
    X = {k: torch.randn(B, k, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16) for k in Ks}
    sa = {k: dq_inputs.static_act_scale(A[k]) for k in Ks}
    Y = {n: torch.empty(M, n, dtype=torch.bfloat16, device=dev) for n in Ns}
    Yd = {n: torch.empty(B, n, dtype=torch.bfloat16, device=dev) for n in Ns}
    ws_bytes = max(dq.prefill_workspace_bytes(w, M) for _, w in stack)
    workspace = dq.alloc_workspace(ws_bytes, dev)

    def prefill_pass():
        for cfg, w in stack:
            dq.prefill_quantize(w, A[cfg.K], sa[cfg.K], workspace)
            dq.prefill_gemm(w, M, sa[cfg.K], Y[cfg.N], workspace)

    def decode_pass():
        for cfg, w in stack:
            dq.decode_linear(w, X[cfg.K], out=Yd[cfg.N])

    decode_pass()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        decode_pass()
    for _ in range(max(3, args.warmup)):
        prefill_pass()
        graph.replay()
    torch.cuda.synchronize()
    steps = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    sampler = ClockSampler(local_rank)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    for i in range(steps):
        ev[i][0].record()
        prefill_pass()
        ev[i][1].record()
        graph.replay()
        ev[i][2].record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if world > 1:
        dist.barrier()
    st, det = dq.get_status()
    if st != 0:
        raise RuntimeError(f"device status {dq.status_string(st)} (detail {det})")
    p_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev]))
    d_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in ev]))
    # token after token (how decode runs in serving): the token step of the timed region follows 50 ms of FP4 GEMMs and
    # runs at the SM clock the power cap leaves then; ten consecutive token steps, after a pause, run at the decode
    # phase's own clock
    time.sleep(0.5)
    graph.replay()
    torch.cuda.synchronize()
    l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler2 = ClockSampler(local_rank)
    sampler2.start()
    l0.record()
    for _ in range(10):
        graph.replay()
    l1.record()
    torch.cuda.synchronize()
    clocks_loop = sampler2.stop()
    d_loop_ms = l0.elapsed_time(l1) / 10
    # the same prefill pass with every layer's gate/up -> down pair chained through the gated epilogue (the gate/up GEMM
    # gates and quantises for the down projection; the M x 2F bf16 matrix and the down projection's quantiser pass
    # are gone); random weights stand for interleaved rows as well as for any other order.  Outside `value`; timed
    # alternately with the plain pass, because both run under the power cap.
    ws_h = dq.alloc_workspace(max(dq.prefill_workspace_bytes(w, M) for c, w in stack if c.name.endswith("_down")), dev)
    sh = 1.0 / 2688.0

    def prefill_pass_gated():
        for i, (cfg, w) in enumerate(stack):
            if cfg.name.endswith("_gate_up"):
                dq.prefill_quantize(w, A[cfg.K], sa[cfg.K], workspace)
                dq.prefill_gemm_silu_mul_quantize(w, M, sa[cfg.K], workspace, stack[i + 1][1], sh, ws_h)
            elif cfg.name.endswith("_down"):
                dq.prefill_gemm(w, M, sh, Y[cfg.N], ws_h)
            else:
                dq.prefill_quantize(w, A[cfg.K], sa[cfg.K], workspace)
                dq.prefill_gemm(w, M, sa[cfg.K], Y[cfg.N], workspace)

    prefill_pass_gated()
    torch.cuda.synchronize()
    g_ev = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
    g_ev[0].record()
    prefill_pass()
    g_ev[1].record()
    prefill_pass_gated()
    g_ev[2].record()
    prefill_pass()
    g_ev[3].record()
    prefill_pass_gated()
    g_ev[4].record()
    torch.cuda.synchronize()
    st, det = dq.get_status()
    if st != 0:
        raise RuntimeError(f"device status {dq.status_string(st)} (detail {det}) after the gated prefill pass")
    pg_plain = 0.5 * (g_ev[0].elapsed_time(g_ev[1]) + g_ev[2].elapsed_time(g_ev[3]))
    pg_gated = 0.5 * (g_ev[1].elapsed_time(g_ev[2]) + g_ev[3].elapsed_time(g_ev[4]))
    p_ms, d_ms, d_loop_ms, pg_plain, pg_gated = replicas.max_over_ranks([p_ms, d_ms, d_loop_ms, pg_plain, pg_gated], device=dev)
    weights = float(sum(c.N * c.K for c, _ in stack))
    flops = 2.0 * M * weights
    dec_bytes = 0.4375 * weights + sum(2.0 * B * (c.K + c.N) + 4 for c, _ in stack)
    tflops = replicas.whole_job_rate(flops, world, p_ms) / 1e12
    gbs = replicas.whole_job_rate(dec_bytes, world, d_ms) / 1e9
    passes = (B + 1) // 2
    line = {
        "metric": METRIC, "value": tflops, "unit": "TFLOP/s", "n_gpus": world, "steps": steps, "warmup": max(3, args.warmup),
        "ms_per_step": p_ms + d_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "nvfp4",
        "data": "synthetic",
        "config": {"workload": "c4_stack27b", "layers": layers, "matrices": len(stack), "weights": weights, "M": M,
                   "decode_batch": B, "parallelism": f"replicas x{world}",
                   "l2": f"inputs larger than L2: packed stack {sum(w.packed.numel() for _, w in stack) / 1e9:.1f} GB",
                   "step": "prefill pass (quantise + GEMM per matrix) + decode token step (one CUDA graph)"},
        "clocks": clocks, "gpu_launches": steps * len(stack) * (2 + passes),
        "prefill": {"ms": p_ms, "linear_tflops_per_gpu": tflops / world,
                    "gated_ffn_pass_ms": pg_gated, "plain_pass_beside_it_ms": pg_plain,
                    "gated_ffn_pass_tflops_per_gpu": flops / (pg_gated * 1e-3) / 1e12},
        "decode": {"ms": d_ms, "value": gbs, "unit": "GB/s", "batch": B, "frac_of_measured_hbm": gbs / world / peaks["hbm_gbs"],
                   "token_loop_ms": d_loop_ms, "token_loop_gbs": dec_bytes / (d_loop_ms * 1e-3) / 1e9,
                   "token_loop_frac_of_measured_hbm": dec_bytes / (d_loop_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                   "token_loop_clocks": clocks_loop},
        "pack_s": pack_s,
        "roofline": {"kernel": "gemm_nvfp4_pair_kernel (+ quant_act_kernel)", "bound": "tensor", "achieved": tflops / world,
                     "peak": 4.0 * peaks["bf16_sustained"], "unit": "TFLOP/s",
                     "frac": tflops / world / (4.0 * peaks["bf16_sustained"]), "traffic": None},
    }
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(dq_inputs.CONFIGS) + ["c4_stack27b"])
    ap.add_argument("--layers", type=int, default=0, help="c4_stack27b only: number of layers (0 = all 64)")
    ap.add_argument("--mnk", default=None, help="M,N,K of an ad-hoc Gaussian layer (profiling small cases)")
    ap.add_argument("--impl", default="dq", choices=["dq", "reference"])
    ap.add_argument("--decode-batch", type=int, default=1)
    ap.add_argument("--copies", type=int, default=0, help="rotating packed-weight copies (0 = enough to exceed 2x L2)")
    ap.add_argument("--ref-rows", type=int, default=0,
                    help="prefill rows per oracle pass (0 = 2048 for cpu_baseline; sized to a ~3 minute run for --impl reference)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-b2b", action="store_true", help="skip the back-to-back decode loops (short profiling runs)")
    ap.add_argument("--no-ffn", action="store_true", help="skip the gated FFN chain (gate/up, SiLU*up, down) measurement")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # asked for N GPUs outside a launcher: start N ranks (one per GPU) of this same command
        from paper_2609_26333_b200 import replicas
        os.execvp(sys.executable, replicas.spawn_command(args.gpus, [str(Path(__file__).resolve())] + sys.argv[1:]))
    args.warmup = max(args.warmup, 3) if args.impl == "dq" else args.warmup
    if args.workload == "c4_stack27b":
        if args.impl == "reference":
            print(json.dumps({"impl": "reference", "unavailable": "the stack workload is timed on the GPU arm only"}))
            return
        if args.steps == 200:
            args.steps = 5
        run_stack(args)
        return
    cfg = dq_inputs.CONFIGS[args.workload]
    if args.mnk:
        m, n, k = (int(v) for v in args.mnk.split(","))
        cfg = dq_inputs.LayerConfig(f"adhoc_{m}x{n}x{k}", N=n, K=k, M=m, cfg_id=9)

    if args.impl == "reference":
        run_reference(args, cfg)
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    import __graft_entry__ as g
    if rank == 0:
        g.build()
    if world > 1:
        dist.barrier()
    import paper_2609_26333_b200 as dq
    dq.lib()

    peaks = load_peaks()
    M, N, K, B = cfg.M, cfg.N, cfg.K, args.decode_batch

    # ---- inputs (seeded, CPU-drawn, same bytes the oracle would see) ----
    W = dq_inputs.make_weight(cfg).to(dev)
    A_host = dq_inputs.make_activations(cfg, M).pin_memory()
    X_host = dq_inputs.make_activations(cfg, B, salt=2).pin_memory()
    sa = dq_inputs.static_act_scale(A_host)
    A = A_host.to(dev)
    X = X_host.to(dev)

    FORMATS = dq.FMT_NVFP4 | dq.FMT_LUT3 | dq.FMT_LUT2
    packed_bytes = dq.packed_bytes(N, K, FORMATS)
    copies = args.copies or max(2, int(np.ceil(2.5 * L2_BYTES / (0.4375 * N * K))))
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ws = []
    for c in range(copies):
        if c == 1:
            e0.record()
        ws.append(dq.pack_weights(W, formats=FORMATS))
        if c == 1:
            e1.record()
    torch.cuda.synchronize()
    pack_ms = e0.elapsed_time(e1) if copies > 1 else None
    del W

    workspace = dq.alloc_workspace(dq.prefill_workspace_bytes(ws[0], M), dev)
    Y = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
    Yd = torch.empty(B, N, dtype=torch.bfloat16, device=dev)

    def step(i, ev=None):
        w = ws[i % copies]
        if ev is not None:
            ev[0].record()
        dq.prefill_quantize(w, A, sa, workspace)
        if ev is not None:
            ev[1].record()
        dq.prefill_gemm(w, M, sa, Y, workspace)
        if ev is not None:
            ev[2].record()
        dq.decode_linear(w, X, out=Yd)
        if ev is not None:
            ev[3].record()

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    st, det = dq.get_status()
    if st != 0:
        raise RuntimeError(f"device status {dq.status_string(st)} (detail {det}) after warm-up")

    # ---- timed region: exactly K steps ----
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    t_start.record()
    for i in range(args.steps):
        step(args.warmup + i, evs[i])
    t_end.record()
    torch.cuda.synchronize()
    # the last GEMM launch of the timed region as its own first CTA saw it: SM cycles and global-timer nanoseconds
    gemm_cycles, gemm_ns = dq.bench_gemm_clocks() if M > 128 else (0, 0)
    clocks = sampler.stop()
    if world > 1:
        dist.barrier()
    total_ms = t_start.elapsed_time(t_end)
    q_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
    g_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    d_ms = float(np.mean([e[2].elapsed_time(e[3]) for e in evs]))
    st, det = dq.get_status()
    if st != 0:
        raise RuntimeError(f"device status {dq.status_string(st)} (detail {det}) after the timed region")

    # ---- decode launches back to back (token after token, rotating weight copies): the events of the
    #      step loop separate the launches, which hides the overlap of one launch's set-up with the tail
    #      of the launch before it (programmatic dependent launch); this loop shows it.  The token loop is
    #      captured into one CUDA graph and replayed (how the paper times decode, App. C.2), so that the
    #      host's launch rate is not what is measured.
    nb2b = 2 if args.no_b2b else max(50, 3 * copies)
    b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def token_loop_ms(fn, X=X, Yd=Yd):
        for i in range(copies):
            fn(ws[i], X, out=Yd)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(nb2b):
                fn(ws[i % copies], X, out=Yd)
        g.replay()
        torch.cuda.synchronize()
        reps = 3
        b0.record()
        for _ in range(reps):
            g.replay()
        b1.record()
        torch.cuda.synchronize()
        return b0.elapsed_time(b1) / (reps * nb2b)

    d_b2b_ms = token_loop_ms(dq.decode_linear)
    # the same token loop on the NVFP4 view (weight-only NVFP4A16 decode, 0.5625 byte per weight)
    d_nv_ms = token_loop_ms(dq.decode_linear_nvfp4)
    # and on the LUT2 weights (2.5 bit per weight)
    d_l2_ms = token_loop_ms(dq.decode_linear_lut2)
    # LUT3 decode at larger batches (skinny GEMM on the same weights): back-to-back launches, ms per launch
    d_batches = {}
    if not args.no_b2b:
        for bb in (2, 4, 8, 16, 32, 64):
            Xb = torch.randn(bb, K, dtype=torch.float32, device=dev).to(torch.bfloat16)
            Yb = torch.empty(bb, N, dtype=torch.bfloat16, device=dev)
            d_batches[str(bb)] = token_loop_ms(dq.decode_linear, Xb, Yb)
    # the tcgen05 variant of the LUT3 decode (levels through tensor memory; not what dq_decode_linear launches), where its
    # shared-memory layout takes the row length and the batch is 1
    d_tc_ms = None
    if B == 1 and K <= 12288 and not args.no_b2b:
        d_tc_ms = token_loop_ms(lambda w, X, out: dq.test_decode_linear(w, dq.FMT_LUT3, X, out=out, variant=3))

    # ---- measured ceilings (outside the timed region): the GEMM kernel's MMA issue sequence alone, and a
    #      read-only 128-bit streaming pass over the packed copies
    fp4_probe_tflops = stream_read_gbs = None
    if M > 128 and not args.no_b2b:
        for _ in range(3):
            dq.bench_gemm_mma_only(ws[0], M, Y, workspace)
        torch.cuda.synchronize()
        b0.record()
        for _ in range(10):
            dq.bench_gemm_mma_only(ws[0], M, Y, workspace)
        b1.record()
        torch.cuda.synchronize()
        fp4_probe_tflops = 2.0 * M * N * K / (b0.elapsed_time(b1) / 10 * 1e-3) / 1e12
    if not args.no_b2b:
        scratch = torch.zeros(8, dtype=torch.uint8, device=dev)
        bufs = [w.packed for w in ws]
        for t in bufs:
            dq.bench_stream_read(t[: t.numel() // 16 * 16], scratch)
        torch.cuda.synchronize()
        b0.record()
        for t in bufs:
            dq.bench_stream_read(t[: t.numel() // 16 * 16], scratch)
        b1.record()
        torch.cuda.synchronize()
        stream_read_gbs = sum(t.numel() // 16 * 16 for t in bufs) / (b0.elapsed_time(b1) * 1e-3) / 1e9
        st, det = dq.get_status()
        if st != 0:
            raise RuntimeError(f"device status {dq.status_string(st)} (detail {det}) after the measurement hooks")

    # ---- the activation stage fused with the operator in front of it (outside the timed region): the stand-alone
    #      quantiser against RMSNorm + quantiser in one kernel (K wide) and, for the stage in front of a down
    #      projection of this width, SiLU(gate)*up + quantiser on a [gate | up] matrix of 2K columns
    fused = None
    if not args.no_b2b:
        def timed(fn, n=10):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            b0.record()
            for _ in range(n):
                fn()
            b1.record()
            torch.cuda.synchronize()
            return b0.elapsed_time(b1) / n
        gamma = torch.ones(K, dtype=torch.bfloat16, device=dev)
        Mf = min(M, 4096)
        GU = torch.randn(Mf, 2 * K, generator=torch.Generator(device=dev).manual_seed(5), device=dev, dtype=torch.float32).to(torch.bfloat16)
        q_only = timed(lambda: dq.prefill_quantize(ws[0], A, sa, workspace))
        n_q = timed(lambda: dq.prefill_rmsnorm_quantize(ws[0], A, gamma, 1e-6, sa, workspace))
        s_q = timed(lambda: dq.prefill_silu_mul_quantize(ws[0], GU, sa, workspace))
        fused = {"quantize_ms": q_only, "rmsnorm_quantize_ms": n_q, "rmsnorm_quantize_gbs": 2.5625 * M * K / (n_q * 1e-3) / 1e9,
                 "silu_mul_quantize_ms": s_q, "silu_mul_rows": Mf, "silu_mul_quantize_gbs": 4.5625 * Mf * K / (s_q * 1e-3) / 1e9,
                 "note": "unfused, the bf16 intermediate costs a write and a read of 2 bytes per element (4 of the 6.56 "
                         "bytes per element of norm + quantiser) that the fused kernels do not make"}
        del GU

    # ---- the gated FFN this matrix belongs to (outside the timed region): fused gate/up projection (2N x K, rows
    #      interleaved for the gated epilogue), SiLU(gate)*up, down projection (K x N), once with the bf16 gate/up
    #      matrix written and read back (three calls) and once with the gating and the quantiser in the GEMM's
    #      epilogue (two calls); the activation quantiser in front is the same in both and is included
    ffn = None
    if not args.no_b2b and not args.no_ffn and N % 128 == 0:
        gen = torch.Generator(device=dev).manual_seed(6)
        Wgu = (torch.randn(2 * N, K, generator=gen, device=dev, dtype=torch.float32) * 0.02).to(torch.bfloat16)
        w_gu = dq.pack_weights(Wgu, formats=dq.FMT_NVFP4)
        del Wgu
        Wd = (torch.randn(K, N, generator=gen, device=dev, dtype=torch.float32) * 0.02).to(torch.bfloat16)
        w_dn = dq.pack_weights(Wd, formats=dq.FMT_NVFP4)
        del Wd
        ws_in = dq.alloc_workspace(dq.prefill_workspace_bytes(w_gu, M), dev)
        ws_h = dq.alloc_workspace(dq.prefill_workspace_bytes(w_dn, M), dev)
        GU = torch.empty(M, 2 * N, dtype=torch.bfloat16, device=dev)
        Yf = torch.empty(M, K, dtype=torch.bfloat16, device=dev)
        sh = 1.0 / 2688.0

        def ffn_unfused():
            dq.prefill_quantize(w_gu, A, sa, ws_in)
            dq.prefill_gemm(w_gu, M, sa, GU, ws_in)
            dq.prefill_silu_mul_quantize(w_dn, GU, sh, ws_h)
            dq.prefill_gemm(w_dn, M, sh, Yf, ws_h)

        def ffn_fused():
            dq.prefill_quantize(w_gu, A, sa, ws_in)
            dq.prefill_gemm_silu_mul_quantize(w_gu, M, sa, ws_in, w_dn, sh, ws_h)
            dq.prefill_gemm(w_dn, M, sh, Yf, ws_h)

        t_un, t_fu = timed(ffn_unfused), timed(ffn_fused)
        t_g = timed(lambda: dq.prefill_gemm(w_gu, M, sa, GU, ws_in))
        t_gg = timed(lambda: dq.prefill_gemm_silu_mul_quantize(w_gu, M, sa, ws_in, w_dn, sh, ws_h))
        t_s = timed(lambda: dq.prefill_silu_mul_quantize(w_dn, GU, sh, ws_h))
        t_d = timed(lambda: dq.prefill_gemm(w_dn, M, sh, Yf, ws_h))
        fl = 2.0 * M * (2 * N) * K + 2.0 * M * K * N
        ffn = {"M": M, "hidden": K, "features": N, "three_call_ms": t_un, "gated_epilogue_ms": t_fu,
               "three_call_tflops": fl / (t_un * 1e-3) / 1e12, "gated_epilogue_tflops": fl / (t_fu * 1e-3) / 1e12,
               "gate_up_gemm_ms": t_g, "gate_up_gemm_gated_ms": t_gg, "silu_mul_quantize_ms": t_s, "down_gemm_ms": t_d,
               "bf16_intermediate_bytes_avoided": 2 * 2 * M * 2 * N}
        st, det = dq.get_status()
        if st != 0:
            raise RuntimeError(f"device status {dq.status_string(st)} (detail {det}) after the FFN chain")
        del GU, Yf, ws_in, ws_h, w_gu, w_dn

    # ---- end to end: pinned host buffers, copies inside the timed region ----
    e2e = None
    if not args.no_e2e:
        Y_host = torch.empty(M, N, dtype=torch.bfloat16).pin_memory()
        Yd_host = torch.empty(B, N, dtype=torch.bfloat16).pin_memory()
        staging = dq.alloc_workspace(dq.prefill_host_staging_bytes(ws[0], M), dev)

        def e2e_step(i, ev=None):
            # the C-ABI calls on host buffers: copies in both directions are inside the calls
            w = ws[i % copies]
            if ev is not None:
                ev[0].record()
            dq.prefill_linear_host(w, A_host, sa, Y_host, staging)
            if ev is not None:
                ev[1].record()
            dq.decode_linear_host(w, X_host, Yd_host, staging)
            if ev is not None:
                ev[2].record()

        for i in range(3):
            e2e_step(i)
        torch.cuda.synchronize()
        n_e2e = max(3, min(args.steps, 10))
        ee = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_e2e)]
        for i in range(n_e2e):
            e2e_step(i, ee[i])
        torch.cuda.synchronize()
        p_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ee]))
        dd_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in ee]))
        e2e = {"prefill_ms": p_ms, "decode_ms": dd_ms, "steps": n_e2e}

    # ---- max over ranks ----
    from paper_2609_26333_b200 import replicas
    total_ms, q_ms, g_ms, d_ms, e2e_p_ms, e2e_d_ms, d_b2b_ms, d_nv_ms, d_l2_ms = replicas.max_over_ranks(
        [total_ms, q_ms, g_ms, d_ms, e2e["prefill_ms"] if e2e else 0.0, e2e["decode_ms"] if e2e else 0.0, d_b2b_ms,
         d_nv_ms, d_l2_ms], device=dev)

    flops = 2.0 * M * N * K
    dec_bytes = 0.4375 * N * K + 2.0 * B * K + 2.0 * B * N + 4
    quant_bytes = 2.5625 * M * K
    prefill_tflops = replicas.whole_job_rate(flops, world, q_ms + g_ms) / 1e12
    gemm_tflops = flops / (g_ms * 1e-3) / 1e12
    decode_gbs = dec_bytes / (d_ms * 1e-3) / 1e9
    quant_gbs = quant_bytes / (q_ms * 1e-3) / 1e9
    # FP4 tensor peak "of measured": 4 x the measured bf16 cuBLAS rate (nominal ratio fp4 : bf16), the burst figure
    # when the whole timed region is shorter than a second (the clocks never settle under the power cap in that
    # time), the sustained figure otherwise
    burst = total_ms < 1000.0
    fp4_peak = 4.0 * (peaks["bf16_burst"] if burst else peaks["bf16_sustained"])
    sm_mhz = clocks.get("sm_mhz")
    in_kernel = None
    if gemm_cycles and gemm_ns:
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        per_clk = 2.0 * M * N * K / (gemm_cycles * sms)
        in_kernel = {"sm_cycles": gemm_cycles, "us": gemm_ns / 1e3, "sm_mhz": gemm_cycles / gemm_ns * 1e3,
                     "flop_per_clk_per_sm": per_clk, "frac_of_tensor_pipe_per_clock": per_clk / 32768.0,
                     "note": "last GEMM launch of the timed region, clock64 and globaltimer on its first CTA's SM; 32768 "
                             "FLOP per clock and SM = one 128x256x64 FP4 MMA per 128 clocks, the rate the MMA issue "
                             "sequence reaches between accumulator hand-offs"}

    line = {
        "metric": METRIC, "value": prefill_tflops, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "nvfp4", "data": "synthetic",
        "config": {"workload": cfg.name, "N": N, "K": K, "M": M, "decode_batch": B, "parallelism": f"replicas x{world}",
                   "l2": f"inputs larger than L2: {copies} rotating packed-weight copies "
                         f"({copies * packed_bytes / 1e6:.0f} MB), A {2 * M * K / 1e6:.0f} MB, Y {2 * M * N / 1e6:.0f} MB",
                   "step": "dq_prefill_quantize + dq_prefill_gemm + dq_decode_linear"},
        "clocks": clocks,
        "gpu_launches": 3 * args.steps,
        "prefill": {"quant_ms": q_ms, "gemm_ms": g_ms, "gemm_tflops": gemm_tflops,
                    "linear_tflops_per_gpu": prefill_tflops / world, "quant_gbs": quant_gbs,
                    "quant_frac_of_hbm": quant_gbs / peaks["hbm_gbs"]},
        "decode": {"ms": d_ms, "value": world * decode_gbs, "unit": "GB/s", "batch": B,
                   "frac_of_measured_hbm": decode_gbs / peaks["hbm_gbs"], "frac_of_8tbs": decode_gbs / 8000.0,
                   "back_to_back_ms": d_b2b_ms, "back_to_back_gbs": world * dec_bytes / (d_b2b_ms * 1e-3) / 1e9,
                   "back_to_back_frac_of_measured_hbm": dec_bytes / (d_b2b_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "decode_nvfp4a16": {"back_to_back_ms": d_nv_ms, "unit": "GB/s",
                            "value": world * (0.5625 * N * K + 2.0 * B * (K + N)) / (d_nv_ms * 1e-3) / 1e9,
                            "frac_of_measured_hbm": (0.5625 * N * K + 2.0 * B * (K + N)) / (d_nv_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "pack_ms": pack_ms,
        "roofline": {"kernel": "gemm_nvfp4_pair_kernel" if M > 128 else "gemm_nvfp4_kernel", "bound": "tensor",
                     "achieved": gemm_tflops, "peak": fp4_peak,
                     "unit": "TFLOP/s", "frac": gemm_tflops / fp4_peak,
                     "traffic": NCU_TRAFFIC_BYTES.get(("gemm", cfg.name)),
                     "peak_source": f"4 x {peaks['source']} bf16 cuBLAS, {'burst' if burst else 'sustained'} figure "
                                    f"({peaks['bf16_burst'] if burst else peaks['bf16_sustained']} TFLOP/s): the timed region "
                                    f"lasted {total_ms:.0f} ms",
                     "frac_of_4x_burst_bf16": gemm_tflops / (4.0 * peaks["bf16_burst"]),
                     "frac_of_4x_sustained_bf16": gemm_tflops / (4.0 * peaks["bf16_sustained"]),
                     "frac_of_nominal_fp4": gemm_tflops / NOMINAL_FP4_TFLOPS,
                     "fp4_probe_tflops": fp4_probe_tflops,
                     "frac_of_probe": gemm_tflops / fp4_probe_tflops if fp4_probe_tflops else None,
                     "gemm_ms_x_sm_mhz": g_ms * sm_mhz if sm_mhz else None,
                     "in_kernel": in_kernel},
        "roofline_decode": {"kernel": "gemv_lut_kernel<3>", "bound": "hbm", "achieved": decode_gbs,
                            "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": decode_gbs / peaks["hbm_gbs"],
                            "traffic": NCU_TRAFFIC_BYTES.get(("gemv", cfg.name)) if B == 1 else None,
                            "peak_source": f"{peaks['source']} copy bandwidth",
                            "timing": "inside the step, between the GEMM and the next step's quantiser",
                            "frac_of_nominal_8tbs": decode_gbs / NOMINAL_HBM_GBS,
                            "stream_read_gbs": stream_read_gbs,
                            "decode_ms_x_sm_mhz": d_ms * sm_mhz if sm_mhz else None},
    }
    nv_bytes = 0.5625 * N * K + 2.0 * B * (K + N)
    line["roofline_decode_nvfp4a16"] = {"kernel": "gemv_nvfp4_mma_kernel", "bound": "hbm",
                                        "achieved": nv_bytes / (d_nv_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                        "frac": nv_bytes / (d_nv_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                        "traffic": NCU_TRAFFIC_BYTES.get(("gemv_nvfp4", cfg.name)),
                                        "timing": "back-to-back launches replayed from one CUDA graph", "peak_source": f"{peaks['source']} copy bandwidth"}
    line["roofline_decode"]["back_to_back"] = {"achieved": dec_bytes / (d_b2b_ms * 1e-3) / 1e9,
                                               "frac": dec_bytes / (d_b2b_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                               "frac_of_stream_read": dec_bytes / (d_b2b_ms * 1e-3) / 1e9 / stream_read_gbs
                                               if stream_read_gbs else None}
    l2_bytes = 0.3125 * N * K + 2.0 * B * (K + N) + 4
    line["roofline_decode_lut2"] = {"kernel": "gemv_lut_kernel<2>", "bound": "hbm", "achieved": l2_bytes / (d_l2_ms * 1e-3) / 1e9,
                                    "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                    "frac": l2_bytes / (d_l2_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None,
                                    "ms": d_l2_ms, "timing": "back-to-back launches replayed from one CUDA graph",
                                    "peak_source": f"{peaks['source']} copy bandwidth"}
    if d_batches:
        line["decode"]["back_to_back_ms_by_batch"] = d_batches
    if d_tc_ms:
        line["roofline_decode"]["tcgen05_variant"] = {"kernel": "gemv_lut_tc_kernel<3>", "ms": d_tc_ms,
                                                      "achieved": dec_bytes / (d_tc_ms * 1e-3) / 1e9,
                                                      "frac": dec_bytes / (d_tc_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                                      "timing": "back-to-back launches replayed from one CUDA graph (test hook)"}
    if fused:
        line["fused_activation_stage"] = fused
    if ffn:
        line["gated_ffn"] = ffn
    if e2e:
        line["e2e"] = {"value": world * flops / (e2e_p_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                       "h2d_bytes_per_step": int(2 * M * K + 2 * B * K), "d2h_bytes_per_step": int(2 * M * N + 2 * B * N),
                       "prefill_ms": e2e_p_ms, "decode_ms": e2e_d_ms,
                       "decode_gbs": world * dec_bytes / (e2e_d_ms * 1e-3) / 1e9}

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        rows = min(M, args.ref_rows or 8192)
        W_f32 = dq_inputs.bf16_to_f32_numpy(dq_inputs.make_weight(cfg))
        A_f32 = dq_inputs.bf16_to_f32_numpy(A_host[:rows])
        X_f32 = dq_inputs.bf16_to_f32_numpy(X_host)
        ref = oracle.pack_weights(W_f32)
        tp = td = 0.0
        passes = 0
        t_all = time.perf_counter()
        while passes < 2 or (time.perf_counter() - t_all < 12.0 and passes < 16):    # about 10-20 s of oracle work
            a, b = oracle_sample_run(cfg, W_f32, ref, A_f32, sa, X_f32, rows)
            tp, td, passes = tp + a, td + b, passes + 1
        tp, td = tp / passes, td / passes
        line["cpu_baseline"] = {"value": 2.0 * rows * N * K / tp / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(),
                                "kind": "oracle",
                                "sample": f"{passes} passes of {rows} of {M} prefill rows against the whole {N}x{K} layer "
                                          f"(oracle quantise + dequantise, then numpy's fp64 dgemm (oracle.matmul_nt_lib), "
                                          f"{tp:.1f} s each) and 1 decode token ({td:.1f} s each)",
                                "decode_gbs": (0.4375 * N * K + 2 * K + 2 * N + 4) / td / 1e9}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
