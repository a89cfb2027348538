#!/usr/bin/env python
"""Benchmark of the fake-quantization hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = one pass of the whole path over one batch: the quantization-aware linear layer with
MXFP4 weights and activations, forward plus straight-through backward (dX and dW), on
X [8192,4096], W [12288,4096], dY [8192,12288] — i.e. two quantize-dequantize passes over W and X
(forward, and again in the backward, since the fake-quantized copies are transient; the backward's pass over X
rides inside the dX matmul launch) and three BF16 tensor-core matmuls. Prints ONE JSON line (rank 0). Multi-GPU runs are independent replicas of
the same workload (the path has no exchange step): weak scaling, no data-path collective. With
``--gpus N`` (N > 1) and no torchrun environment the script starts the N ranks itself.

Beside the headline the line carries: the matmul's roofline record (with the SM clock the kernel itself
measured), a sustained run of at least two seconds, the quantizer bandwidths, the end-to-end figure with host
buffers, the CPU oracle's rate, and the other named workloads (``other_workloads``).

`--impl reference` times the CPU oracle (the only other place this file may execute `oracle/`).
"""
from __future__ import annotations

import argparse
import json
import os
import re
import socket
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

M, N, K = 8192, 12288, 4096
WORKLOAD = "mxfp4_w4a4_linear_fwd_bwd_8192x4096x12288"
FLOP_PER_GEMM = 2.0 * M * N * K
FLOP_PER_STEP = 3.0 * FLOP_PER_GEMM
SECTIONS = ("roofline", "sustained", "qdq", "e2e", "cpu", "configs")
DATASHEET_TFLOPS = 2250.0            # dense BF16, nominal
TENSOR_FLOP_PER_CLK_PER_SM = 8192    # dense BF16 multiply-adds x 2 per SM per clock (2250e12 / 148 / 1.86e9)
NUM_SMS = 148


def _set_shape(spec: str):
    """--shape M,N,K: a smaller case of the same workload, for profiler captures only."""
    global M, N, K, WORKLOAD, FLOP_PER_GEMM, FLOP_PER_STEP
    M, N, K = (int(v) for v in spec.split(","))
    WORKLOAD = f"mxfp4_w4a4_linear_fwd_bwd_{M}x{K}x{N}"
    FLOP_PER_GEMM = 2.0 * M * N * K
    FLOP_PER_STEP = 3.0 * FLOP_PER_GEMM
KERNELS_PER_STEP = 6          # fwd: qdq(W), qdq(X), gemm; bwd: qdq(W), gemm (dX, with qdq(X) as its side job), gemm (dW)


def _peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"], "bf16_sustained": d["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


def _profiled_traffic(m: int, n: int, k: int):
    """Mean DRAM bytes per matmul launch of a step, as the committed ncu summary of that shape records it
    (a line ``traffic_bytes_per_launch M=.. N=.. K=..: <bytes>``); None when no capture of this shape is on file."""
    p = ROOT / "profiles" / "gemm_pair_kernel_mxfp4_linear.md"
    if not p.exists():
        return None
    pat = re.compile(r"traffic_bytes_per_launch\s+M=(\d+)\s+N=(\d+)\s+K=(\d+):\s*([0-9.eE+]+)")
    for mm in pat.finditer(p.read_text()):
        if (int(mm.group(1)), int(mm.group(2)), int(mm.group(3))) == (m, n, k):
            return float(mm.group(4))
    return None


class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML while the timed region runs (read-only), about once
    per millisecond."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                 "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for n, bit in names.items():
                    if r & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(0.001)

    def __enter__(self):
        if self.nv:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_min_mhz": s[0] if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def _physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# -------------------------------------------------------------------------------------------------
# launcher: --gpus N without a torchrun environment starts N ranks
# -------------------------------------------------------------------------------------------------

def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n: int, argv: list[str]) -> int:
    """Re-runs this script as n ranks under torch.distributed.run (one process per GPU, rendezvous on 127.0.0.1)
    and returns its exit code. Rank 0 of the children prints the JSON line."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), str(Path(__file__).resolve()), *argv]
    return subprocess.call(cmd)


def run_dry(args):
    """The launch and timing protocol alone, with no GPU: ranks rendezvous over gloo, "run" steps that only sleep,
    take the max time over ranks and print the line. What the CPU tests use to check `--gpus N`."""
    from paper_2609_39223_b200 import replicas
    world, rank, _ = replicas.world()
    replicas.init("gloo")
    replicas.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(0.002 * (1 + rank))
    ms = replicas.max_over_ranks((time.perf_counter() - t0) * 1e3)
    replicas.barrier()
    if rank == 0:
        print(json.dumps({"dry_run": True, "impl": args.impl, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                          "ms_per_step": ms / max(1, args.steps), "scaling": "weak"}))
    replicas.finish()


# -------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on a bounded slice of the same workload
# -------------------------------------------------------------------------------------------------

def _oracle_slice(m_rows: int, n_rows: int, seed: int = 0):
    """fwd + dX + dW of the MXFP4 W4A4 layer on an [m_rows, K] x [n_rows, K] slice; returns (seconds, flop)."""
    import numpy as np
    import oracle
    from paper_2609_39223_b200 import synth
    c = synth.linear_case(m_rows, n_rows, K, seed=seed)
    import torch
    to_bits = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)
    xb, wb, dyb = to_bits(c.X), to_bits(c.W), to_bits(c.dY)
    t0 = time.perf_counter()
    oracle.fq_linear_fwd(xb, wb, oracle.FMT_MXFP4, oracle.FMT_MXFP4)
    oracle.fq_linear_bwd(dyb, xb, wb, oracle.FMT_MXFP4, oracle.FMT_MXFP4)
    dt = time.perf_counter() - t0
    return dt, 3.0 * 2.0 * m_rows * n_rows * K


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    world = int(os.environ.get("WORLD_SIZE", "1"))
    import oracle
    cores = oracle.num_threads()
    n_rows = 512
    # size the slice so that steps+warmup stay within about two minutes
    dt, fl = _oracle_slice(64, n_rows)
    rate = fl / dt
    budget = 120.0 / max(1, args.steps + args.warmup)
    m_rows = int(max(8, min(512, (rate * budget) / (6.0 * n_rows * K))))
    for _ in range(args.warmup):
        _oracle_slice(m_rows, n_rows)
    t_total, fl_total = 0.0, 0.0
    for i in range(args.steps):
        dt, fl = _oracle_slice(m_rows, n_rows, seed=i)
        t_total += dt
        fl_total += fl
    value = fl_total / t_total / 1e12
    sample = f"fwd+dX+dW on a [{m_rows},{K}] x [{n_rows},{K}] slice per step (QDQ of both slices included)"
    print(json.dumps({
        "impl": "reference", "metric": "fake-quant linear fwd+bwd TFLOPS", "value": value, "unit": "TFLOP/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_total / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# -------------------------------------------------------------------------------------------------
# the other named workloads
# -------------------------------------------------------------------------------------------------

def _time_ms(torch, fn, reps=5, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


def _timed_region(torch, gpu_index, fn, min_seconds=1.0, warm=3, probe=3):
    """ms per call of fn over a region of at least min_seconds, with the clocks sampled during that region."""
    est = _time_ms(torch, fn, reps=probe, warm=warm)
    reps = max(probe, int(min_seconds * 1e3 / max(est, 1e-3)) + 1)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    with ClockSampler(gpu_index) as clk:
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
    return a.elapsed_time(b) / reps, reps, clk.summary()


def _graph(torch, fn):
    fn(); torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()          # replayed as a graph: the Python binding's per-call cost is not GPU time
    with torch.cuda.graph(g):
        fn()
    return g


def measure_other_workloads(torch, api, synth, dev, peaks, gpu_index, which, region_seconds=1.0):
    """The other named workloads; `which` is a subset of {"cfg1", "cfg3", "cfg4", "cfg5"}; timed regions last at least
    region_seconds (0: a handful of repetitions, for profiler captures)."""
    out = {}
    rs = region_seconds
    wsq = api.workspace(api.OP_QDQ, 0, 0, 0, device=dev)
    hbm = peaks["hbm_gbs"]
    rate = lambda nbytes, ms: nbytes / (ms * 1e-3) / 1e9
    bw = lambda g: {"gbs": g, "frac_of_measured_hbm": g / hbm, "frac_of_8000_nominal": g / 8000.0}
    if "cfg1" in which:
        _cfg1(torch, api, synth, dev, gpu_index, out, bw, rate, wsq, rs)
    if "cfg3" in which:
        _cfg3(torch, api, synth, dev, gpu_index, out, bw, rate, wsq, rs)
    if "cfg4" in which:
        _cfg4(torch, api, synth, dev, gpu_index, out, peaks, rs)
    if "cfg5" in which:
        _cfg5(torch, api, synth, dev, gpu_index, out, peaks, rs)
    return out


def _cfg1(torch, api, synth, dev, gpu_index, out, bw, rate, wsq, rs):
    # ---- 1: NVFP4 QDQ of 2048x2048 weights (all outputs, scale derived from the tensor) -----------------
    mats = [synth.weight_with_outliers(2048, 2048, seed=i, device=dev) for i in range(32)]
    o = torch.empty_like(mats[0]); c = torch.empty((2048, 1024), dtype=torch.uint8, device=dev)
    sc = torch.empty((2048, 128), dtype=torch.uint8, device=dev)
    ts1 = torch.empty(1, dtype=torch.float32, device=dev)
    one = lambda m: api.qf_qdq(api.FMT_NVFP4, m, out=o, codes=c, scales=sc, ws=wsq, tensor_scale=None, ts_out=ts1)
    nbytes = 19136516
    g_cold = _graph(torch, lambda: [one(m) for m in mats])              # 32 distinct matrices, 268 MB: more than twice L2
    g_warm = _graph(torch, lambda: [one(mats[0]) for _ in range(32)])   # one matrix, back to back
    batch = api.QdqBatch(api.FMT_NVFP4, mats)
    g_batch = _graph(torch, batch.run)
    g_spec = _graph(torch, lambda: batch.run(api.TENSOR_SCALE_SPECULATIVE))   # guesses = the scales the previous call derived
    cfg1 = {"bytes_per_matrix": nbytes, "outputs": "codes, E4M3 block scales, FP32 tensor scale, BF16 dequantized",
            "note": "every variant replayed as one CUDA graph of 32 matrices; single = qf_qdq per matrix (header memset + amax "
                    "pre-pass + quantize), batched = one qf_qdq_batched call for the 32 matrices"}
    for name, g in (("single_cold_l2", g_cold), ("single_warm_l2", g_warm), ("batched_32", g_batch),
                    ("batched_32_speculated_scales_hit", g_spec)):
        ms, reps, clk = _timed_region(torch, gpu_index, g.replay, min_seconds=0.2 * min(rs, 1.0))
        cfg1[name] = {"us_per_matrix": ms * 1e3 / 32, **bw(rate(32 * nbytes, ms)), "clocks": clk}
    out["nvfp4_qdq_2048x2048"] = cfg1
    del mats, batch, g_cold, g_warm, g_batch, g_spec


def _cfg3(torch, api, synth, dev, gpu_index, out, bw, rate, wsq, rs):
    # ---- 3: Q4_K QDQ over all linear weights of the 32-layer dense decoder, per-layer seeds (14 GB of weights
    # resident; outputs go to one layer's buffers, reused) ------------------------------------------------------
    layers = [[synth.dense_decoder_weight(l, name, device=dev) for name, _, _ in synth.DENSE_DECODER_LAYER]
              for l in range(synth.DENSE_DECODER_LAYERS)]
    outs = [torch.empty_like(w) for w in layers[0]]
    codes = [torch.empty((w.shape[0], w.shape[1] // 2), dtype=torch.uint8, device=dev) for w in layers[0]]
    scs = [torch.empty(api.scales_shape(api.FMT_Q4_K, *w.shape), dtype=torch.uint8, device=dev) for w in layers[0]]

    def q4k_all():
        for layer in layers:
            for w, oo, cc, ss in zip(layer, outs, codes, scs):
                api.qf_qdq(api.FMT_Q4_K, w, out=oo, codes=cc, scales=ss, ws=wsq)
    g3 = _graph(torch, q4k_all)
    ms, reps, clk = _timed_region(torch, gpu_index, g3.replay, min_seconds=0.5 * min(rs, 1.0), warm=1, probe=2)
    elems = synth.dense_decoder_layer_elems() * synth.DENSE_DECODER_LAYERS
    out["q4k_qdq_dense_decoder_32_layers"] = {"ms": ms, "elements": elems, **bw(rate(elems * 4.5625, ms)), "reps": reps, "clocks": clk,
                                              "note": "224 distinct weight tensors (per-layer seeds), one qf_qdq call each, as one CUDA graph"}
    del layers, outs, codes, scs, g3
    torch.cuda.empty_cache()


def _cfg4(torch, api, synth, dev, gpu_index, out, peaks, rs):
    # ---- 4: NVFP4 weight-only linear, one 32K-token sequence, up and down projections, fwd + bwd ---------------
    Mt = 32768
    tot_ms, tot_fl, parts = 0.0, 0.0, {}
    for pname, (Nn, Kk) in (("up", (14336, 4096)), ("down", (4096, 14336))):
        cse = synth.linear_case(Mt, Nn, Kk, seed=4, device=dev, outlier_channels=0)
        ws4 = api.workspace(api.OP_LINEAR_BWD, Mt, Nn, Kk, device=dev)
        Y = torch.empty((Mt, Nn), dtype=torch.bfloat16, device=dev); dX = torch.empty((Mt, Kk), dtype=torch.bfloat16, device=dev)
        dW = torch.empty((Nn, Kk), dtype=torch.float32, device=dev); wts = torch.zeros(1, device=dev)

        def f4():
            api.qf_fq_linear_fwd(cse.X, cse.W, api.FMT_NVFP4, api.FMT_NONE, ws=ws4, Y=Y, w_tscale=wts)
            api.qf_fq_linear_bwd(cse.dY, cse.X, cse.W, api.FMT_NVFP4, api.FMT_NONE, ws=ws4, dX=dX, dW=dW, w_tscale=wts)
        ms, reps, clk = _timed_region(torch, gpu_index, f4, min_seconds=rs, warm=2, probe=2)
        fl = 3 * 2.0 * Mt * Nn * Kk
        mhz = _kernel_clock_mhz(ws4)
        clk["sm_mhz_in_kernel"] = mhz
        parts[pname] = {"ms": ms, "tflops": fl / (ms * 1e-3) / 1e12, "reps": reps, "clocks": clk,
                        "frac_of_tensor_peak_at_kernel_clock": fl / (ms * 1e-3) / (NUM_SMS * TENSOR_FLOP_PER_CLK_PER_SM * mhz * 1e6) if mhz else None}
        tot_ms += ms; tot_fl += fl
        del cse, ws4, Y, dX, dW
    t4 = tot_fl / (tot_ms * 1e-3) / 1e12
    out["nvfp4_weight_only_linear_32k_tokens_up_down"] = {"ms": tot_ms, "tflops": t4, "frac_of_2250_datasheet": t4 / DATASHEET_TFLOPS,
                                                           "frac_of_measured_sustained": t4 / peaks["bf16_sustained"],
                                                           "frac_of_measured_burst": t4 / peaks["bf16_burst"], **parts}


def _cfg5(torch, api, synth, dev, gpu_index, out, peaks, rs):
    # ---- 5: MoE grouped MXFP4 W4A4: 128 experts, top-8 of 16384 tokens, gate + up + down, fwd + bwd. The gate and up
    # projections are stored as one [E, 2F, H] weight, as serving engines keep them: the same products (the quantizer's
    # blocks run along H, so quantizing the concatenation is concatenating the quantized halves), and the routed
    # activations are quantized once for both. ------------------------------------------------------------------------
    tokens, E, top_k, H, F = 16384, 128, 8, 2048, 768
    r = synth.moe_routing(tokens, E, top_k, seed=0)
    rows = int(r.group_offsets[-1]); offs = r.group_offsets.to(dev)
    fmt = api.FMT_MXFP4
    res = {k: [0.0, None] for k in ("default", "reuse", "bf16_dw")}
    for (Nn, Kk) in ((2 * F, H), (H, F)):
        Xp = synth.randn_bf16((rows, Kk), 1.0, 5, device=dev); Xp[(r.token_of_row < 0).to(dev)] = 0
        Wg = synth.randn_bf16((E, Nn, Kk), 0.02, 6, device=dev)
        dYp = synth.randn_bf16((rows, Nn), 1e-3, 7, device=dev); dYp[(r.token_of_row < 0).to(dev)] = 0
        ws5 = api.workspace(api.OP_GROUPED_BWD, rows, Nn, Kk, E, device=dev)
        Y = torch.empty((rows, Nn), dtype=torch.bfloat16, device=dev); dX = torch.empty((rows, Kk), dtype=torch.bfloat16, device=dev)
        dW = torch.empty((E, Nn, Kk), dtype=torch.float32, device=dev)
        dW16 = torch.empty((E, Nn, Kk), dtype=torch.bfloat16, device=dev)

        def f5(dw=dW, flags=0):
            api.qf_fq_grouped_linear_fwd(Xp, Wg, offs, fmt, fmt, ws=ws5, Y=Y)
            api.qf_fq_grouped_linear_bwd(dYp, Xp, Wg, offs, fmt, fmt, ws=ws5, dX=dX, dW=dw, flags=flags)
        for key, fn in (("default", f5), ("reuse", lambda: f5(flags=api.REUSE_W_HAT | api.REUSE_X_HAT)), ("bf16_dw", lambda: f5(dw=dW16))):
            ms, reps, clk = _timed_region(torch, gpu_index, fn, min_seconds=rs if key == "default" else 0.3 * min(rs, 1.0))
            clk["sm_mhz_in_kernel"] = _kernel_clock_mhz(ws5)
            res[key][0] += ms
            res[key][1] = clk
        del Xp, Wg, dYp, ws5, Y, dX, dW, dW16
    fl = 3 * 3 * 2.0 * tokens * top_k * H * F
    tf = lambda ms: fl / (ms * 1e-3) / 1e12
    out["moe_grouped_mxfp4_128_experts"] = {
        "ms": res["default"][0], "tflops": tf(res["default"][0]), "frac_of_2250_datasheet": tf(res["default"][0]) / DATASHEET_TFLOPS,
        "frac_of_measured_sustained": tf(res["default"][0]) / peaks["bf16_sustained"], "clocks": res["default"][1],
        "routed_rows": tokens * top_k, "padded_rows": rows,
        "layout": "gate and up as one [128, 1536, 2048] grouped weight, down [128, 2048, 768]; dW in FP32",
        "ms_reusing_forward_copies": res["reuse"][0], "tflops_reusing_forward_copies": tf(res["reuse"][0]),
        "ms_with_bf16_dw": res["bf16_dw"][0], "tflops_with_bf16_dw": tf(res["bf16_dw"][0])}


# -------------------------------------------------------------------------------------------------
# our arm
# -------------------------------------------------------------------------------------------------

def _kernel_clock_mhz(ws):
    """SM clock the last matmul launch measured for itself: cycles of %clock64 over nanoseconds of %globaltimer,
    both read by the first CTA at its start and end and left in the workspace header."""
    import torch
    cyc, ns = (int(v) for v in ws[48:64].view(torch.int64).tolist())
    return 1e3 * cyc / ns if ns > 0 else None


def _kernel_ms(ws):
    """Duration of the last matmul launch as its first CTA measured it (%globaltimer), in ms."""
    import torch
    return int(ws[56:64].view(torch.int64).item()) * 1e-6


def run_ours(args):
    import torch
    from paper_2609_39223_b200 import api, replicas, synth

    world, rank, local_rank = replicas.world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device — the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    gpu_index = _physical_gpu_index(local_rank)
    replicas.init("nccl", dev)
    api.lib()
    peaks = _peaks()
    fmt = api.FMT_MXFP4

    case = synth.linear_case(M, N, K, seed=rank, device=dev)
    X, W, dY = case.X, case.W, case.dY
    ws = api.workspace(api.OP_LINEAR_BWD, M, N, K, device=dev)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
    dX = torch.empty((M, K), dtype=torch.bfloat16, device=dev)
    dW = torch.empty((N, K), dtype=torch.float32, device=dev)

    step_flags = api.FUSED_QDQ if args.in_kernel_qdq else 0

    def step():
        api.qf_fq_linear_fwd(X, W, fmt, fmt, ws=ws, Y=Y, flags=step_flags)
        api.qf_fq_linear_bwd(dY, X, W, fmt, fmt, ws=ws, dX=dX, dW=dW, flags=step_flags)

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    sections = set(args.sections.split(",")) if args.sections else set()
    # ---- QDQ bandwidth per format (memory-bound kernels; reported beside the headline). Measured first,
    # each kernel on its own, before the long matmul loops pull the clocks down under the power cap. ----
    qdq = {}
    if rank == 0 and "qdq" in sections:
        Wq = synth.randn_bf16((14336, 4096 * 2), 0.02, 7, device=dev)          # 235 MB in, larger than L2
        out = torch.empty_like(Wq)
        codes = torch.empty((Wq.shape[0], Wq.shape[1] // 2), dtype=torch.uint8, device=dev)
        wsq = api.workspace(api.OP_QDQ, 0, 0, 0, device=dev)
        given = torch.full((1,), 1e-4, dtype=torch.float32, device=dev)
        # "nvfp4" derives the tensor scale from the tensor (an extra read of the whole input: the two passes move
        # 6.56 B per element for 4.56 algorithmic, a ceiling of 0.70); "nvfp4_given_scale" is the mode with a
        # tracked / tied tensor scale (QF_TENSOR_SCALE_GIVEN), one pass.
        for name, f, ts in (("nvfp4", api.FMT_NVFP4, None), ("nvfp4_given_scale", api.FMT_NVFP4, given),
                            ("mxfp4", api.FMT_MXFP4, None), ("q4_k", api.FMT_Q4_K, None)):
            sc = torch.empty(api.scales_shape(f, *Wq.shape), dtype=torch.uint8, device=dev)
            for _ in range(3):
                api.qf_qdq(f, Wq, out=out, codes=codes, scales=sc, ws=wsq, tensor_scale=ts)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(10):
                api.qf_qdq(f, Wq, out=out, codes=codes, scales=sc, ws=wsq, tensor_scale=ts)
            b.record(); torch.cuda.synchronize()
            bytes_per_elem = 2 + 2 + 0.5 + (1 / 32 if f == api.FMT_MXFP4 else 1 / 16)
            gbs = Wq.numel() * bytes_per_elem / (a.elapsed_time(b) / 10 * 1e-3) / 1e9
            qdq[name] = {"gbs": round(gbs, 1), "frac_of_measured_hbm": round(gbs / peaks["hbm_gbs"], 4),
                         "frac_of_8000_nominal": round(gbs / 8000.0, 4), "bytes_per_elem": bytes_per_elem}
        # NVFP4 with a speculated tensor scale (QF_TENSOR_SCALE_SPECULATIVE): the scale of the previous call as the guess
        # (the steady state of a weight in training: a hit), and a zeroed guess before every call (a miss every time)
        sc = torch.empty(api.scales_shape(api.FMT_NVFP4, *Wq.shape), dtype=torch.uint8, device=dev)
        carried = torch.zeros(1, dtype=torch.float32, device=dev)

        def spec_hit():
            api.qf_qdq(api.FMT_NVFP4, Wq, out=out, codes=codes, scales=sc, ws=wsq, tensor_scale=carried, flags=api.TENSOR_SCALE_SPECULATIVE)

        def spec_miss():
            carried.zero_()
            spec_hit()
        for name, fn in (("nvfp4_speculated_scale_hit", spec_hit), ("nvfp4_speculated_scale_miss", spec_miss)):
            for _ in range(3):
                fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(10):
                fn()
            b.record(); torch.cuda.synchronize()
            gbs = Wq.numel() * 4.5625 / (a.elapsed_time(b) / 10 * 1e-3) / 1e9
            qdq[name] = {"gbs": round(gbs, 1), "frac_of_measured_hbm": round(gbs / peaks["hbm_gbs"], 4),
                         "frac_of_8000_nominal": round(gbs / 8000.0, 4), "bytes_per_elem": 4.5625}
        del Wq, out, codes

    # ---- headline: K steps, inputs resident in HBM -------------------------------------------------
    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(gpu_index) as clk:
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        barrier()
    ms = replicas.max_over_ranks(e0.elapsed_time(e1), dev)
    status = api.qf_read_status(ws)
    if status != 0:
        raise SystemExit(f"bench.py: device-side status {status} ({api.status_string(status)})")
    value = world * FLOP_PER_STEP * args.steps / (ms * 1e-3) / 1e12
    headline_kernel_mhz = _kernel_clock_mhz(ws)          # what the last launch of the timed region ran at

    # ---- roofline of the dominant kernel (the tcgen05 matmul), timed alone on the same operands ------
    # The three matmuls of a step are launched here on the already fake-quantized operands (format NONE
    # skips the quantizers), each launch bracketed by CUDA events on the launching stream.
    achieved, gemm_ms, gemm_mhz, last_ms_in_kernel = None, None, None, None
    Xh = api.qf_qdq(fmt, X, want_codes=False, want_scales=False)["out"]
    Wh = api.qf_qdq(fmt, W, want_codes=False, want_scales=False)["out"]
    n_rep = max(3, min(args.steps, 20)) if "roofline" in sections else -2
    evs = []

    def timed(f):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); f(); b.record()
        evs.append((a, b))

    for it in range(n_rep + 2):
        if it == 2:
            evs.clear()
        timed(lambda: api.qf_fq_linear_fwd(Xh, Wh, 0, 0, ws=ws, Y=Y))
        timed(lambda: api.qf_fq_linear_bwd(dY, None, Wh, 0, 0, ws=ws, dX=dX, want_dw=False))
        timed(lambda: api.qf_fq_linear_bwd(dY, Xh, None, 0, 0, ws=ws, dW=dW, want_dx=False))
    torch.cuda.synchronize()
    if evs:
        gemm_ms = sum(a.elapsed_time(b) for a, b in evs) / len(evs)
        achieved = FLOP_PER_GEMM / (gemm_ms * 1e-3) / 1e12
        gemm_mhz = _kernel_clock_mhz(ws)
        last_ms_in_kernel = _kernel_ms(ws)
    # the three matmuls alone, back to back for at least two seconds: the figure to hold against the library GEMM's
    # sustained rate (the whole-step sustained figure below also contains the quantize passes)
    gemm_sustained = None
    if "sustained" in sections and evs:
        def three():
            api.qf_fq_linear_fwd(Xh, Wh, 0, 0, ws=ws, Y=Y)
            api.qf_fq_linear_bwd(dY, None, Wh, 0, 0, ws=ws, dX=dX, want_dw=False)
            api.qf_fq_linear_bwd(dY, Xh, None, 0, 0, ws=ws, dW=dW, want_dx=False)
        n3 = int(2000.0 / (3 * gemm_ms)) + 1
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        with ClockSampler(gpu_index) as gclk:
            g0.record()
            for _ in range(n3):
                three()
            g1.record()
            torch.cuda.synchronize()
        gms = g0.elapsed_time(g1)
        gval = 3 * FLOP_PER_GEMM * n3 / (gms * 1e-3) / 1e12
        gmhz = _kernel_clock_mhz(ws)
        gemm_sustained = {"value": gval, "unit": "TFLOP/s", "seconds": gms * 1e-3, "launches": 3 * n3, "clocks": gclk.summary(),
                          "sm_mhz_in_kernel": gmhz, "frac_of_measured_sustained": gval / peaks["bf16_sustained"],
                          "frac_of_2250_datasheet": gval / DATASHEET_TFLOPS,
                          "frac_of_tensor_peak_at_kernel_clock": gval / (NUM_SMS * TENSOR_FLOP_PER_CLK_PER_SM * gmhz * 1e6 / 1e12) if gmhz else None}
    del Xh, Wh

    # ---- sustained: the same step back to back for at least two seconds (the power cap pulls the clock down) ----
    sustained = None
    if "sustained" in sections:
        n_sus = max(args.steps, int(2000.0 / (ms / args.steps)) + 1)
        barrier()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with ClockSampler(gpu_index) as sclk:
            s0.record()
            for _ in range(n_sus):
                step()
            s1.record()
            barrier()
        sms = replicas.max_over_ranks(s0.elapsed_time(s1), dev)
        sval = world * FLOP_PER_STEP * n_sus / (sms * 1e-3) / 1e12
        smhz = _kernel_clock_mhz(ws)
        sustained = {"value": sval, "unit": "TFLOP/s", "steps": n_sus, "seconds": sms * 1e-3, "ms_per_step": sms / n_sus,
                     "clocks": sclk.summary(), "sm_mhz_in_kernel": smhz,
                     "frac_of_measured_sustained": sval / world / peaks["bf16_sustained"],
                     "frac_of_2250_datasheet": sval / world / DATASHEET_TFLOPS,
                     "frac_of_tensor_peak_at_kernel_clock": (sval / world) / (NUM_SMS * TENSOR_FLOP_PER_CLK_PER_SM * smhz * 1e6 / 1e12) if smhz else None}

    # ---- end to end: host buffers, H2D of the inputs and D2H of the results inside the timed region ---
    # Every step copies X, W, dY from pinned host memory, runs the step through the C ABI, and copies
    # Y, dX, dW back to pinned host memory. Copies and compute run on three streams over two sets of
    # device buffers, so step i+1's upload and step i-1's download overlap step i's kernels.
    e2e = None
    if "e2e" in sections:
        hX, hW, hdY = (t.cpu().pin_memory() for t in (X, W, dY))
        hY = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
        hdX = torch.empty((M, K), dtype=torch.bfloat16).pin_memory()
        hdW = torch.empty((N, K), dtype=torch.float32).pin_memory()
        h2d = sum(t.numel() * t.element_size() for t in (hX, hW, hdY))
        d2h = sum(t.numel() * t.element_size() for t in (hY, hdX, hdW))
        bufs = [dict(X=X, W=W, dY=dY, Y=Y, dX=dX, dW=dW),
                dict(X=torch.empty_like(X), W=torch.empty_like(W), dY=torch.empty_like(dY), Y=torch.empty_like(Y),
                     dX=torch.empty_like(dX), dW=torch.empty_like(dW))]
        s_up, s_down, s_main = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()

        def e2e_run(n):
            comp_done, down_done = [None, None], [None, None]
            first = torch.cuda.Event(enable_timing=True)
            last = torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(s_up):
                first.record()
            for i in range(n):
                b = bufs[i % 2]
                with torch.cuda.stream(s_up):
                    if comp_done[i % 2] is not None:
                        s_up.wait_event(comp_done[i % 2])          # inputs of this set were consumed two steps ago
                    b["X"].copy_(hX, non_blocking=True); b["W"].copy_(hW, non_blocking=True); b["dY"].copy_(hdY, non_blocking=True)
                    up = torch.cuda.Event(); up.record()
                s_main.wait_event(up)
                if down_done[i % 2] is not None:
                    s_main.wait_event(down_done[i % 2])            # outputs of this set were downloaded
                api.qf_fq_linear_fwd(b["X"], b["W"], fmt, fmt, ws=ws, Y=b["Y"])
                api.qf_fq_linear_bwd(b["dY"], b["X"], b["W"], fmt, fmt, ws=ws, dX=b["dX"], dW=b["dW"])
                comp_done[i % 2] = torch.cuda.Event(); comp_done[i % 2].record()
                with torch.cuda.stream(s_down):
                    s_down.wait_event(comp_done[i % 2])
                    hY.copy_(b["Y"], non_blocking=True); hdX.copy_(b["dX"], non_blocking=True); hdW.copy_(b["dW"], non_blocking=True)
                    down_done[i % 2] = torch.cuda.Event(); down_done[i % 2].record()
            with torch.cuda.stream(s_down):
                last.record()
            return first, last

        e2e_steps = max(4, min(args.steps, 12))
        e2e_run(3)
        barrier()
        first, last = e2e_run(e2e_steps)
        barrier()
        e2e_ms = replicas.max_over_ranks(first.elapsed_time(last), dev)
        e2e = {"value": world * FLOP_PER_STEP * e2e_steps / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "pcie_gbs_both_directions": (h2d + d2h) * e2e_steps / (e2e_ms * 1e-3) / 1e9,
               "how": "pinned host buffers; upload, kernels and download on three streams, two device buffer sets"}
        del bufs

    # ---- CPU baseline: the oracle on a bounded slice, rank 0 of a 1-GPU run only -----------------------
    cpu = None
    if rank == 0 and world == 1 and "cpu" in sections:
        import oracle
        n_rows = 2048
        dt, fl = _oracle_slice(128, n_rows)                      # calibrate, then aim for about 15 s of CPU work
        m_rows = int(max(128, min(M, 15.0 * (fl / dt) / (6.0 * n_rows * K)))) // 128 * 128
        dt, fl = _oracle_slice(m_rows, n_rows)
        cpu = {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
               "sample": f"fwd+dX+dW on a [{m_rows},{K}] x [{n_rows},{K}] slice of the workload, QDQ of both slices "
                         f"included, {dt:.1f} s"}

    other = None
    which = {"cfg1", "cfg3", "cfg4", "cfg5"} if "configs" in sections else sections & {"cfg1", "cfg3", "cfg4", "cfg5"}
    if rank == 0 and world == 1 and which:
        del X, W, dY, Y, dX, dW, ws
        torch.cuda.empty_cache()
        other = measure_other_workloads(torch, api, synth, dev, peaks, gpu_index, which, args.region_seconds)

    if rank == 0:
        clocks = clk.summary()
        clocks["sm_mhz_in_kernel"] = headline_kernel_mhz
        peak = peaks["bf16_burst"]
        at_clock = NUM_SMS * TENSOR_FLOP_PER_CLK_PER_SM * gemm_mhz * 1e6 / 1e12 if gemm_mhz else None
        line = {
            "metric": "fake-quant linear fwd+bwd TFLOPS", "value": value, "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "wq_fmt": "mxfp4", "aq_fmt": "mxfp4", "M": M, "N": N, "K": K,
                       "outputs": "Y bf16, dX bf16, dW f32", "parallelism": f"replicas x{world}",
                       "qdq": "inside the matmul kernel (QF_FUSED_QDQ)" if args.in_kernel_qdq else "materialised in the workspace (default)",
                       "l2": "inputs (369 MB) larger than L2; no flush"},
            "clocks": clocks,
            "e2e": e2e,
            "gpu_launches": (3 if args.in_kernel_qdq else KERNELS_PER_STEP) * args.steps,
            "roofline": {"bound": "tensor", "kernel": "gemm_pair_kernel (tcgen05 cta_group::2 BF16, 256x256x64 tiles per CTA pair)", "achieved": achieved,
                         "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak if achieved else None,
                         # mean dram__bytes_read.sum + dram__bytes_write.sum per launch over the three matmuls of a
                         # step, read from the committed ncu summary of this shape (None for other shapes)
                         "traffic": _profiled_traffic(M, N, K),
                         "algorithmic_bytes": (2.0 * (M * K + N * K) + 2.0 * M * N + 2.0 * (M * N + N * K) + 2.0 * M * K
                                               + 2.0 * (M * N + M * K) + 4.0 * N * K) / 3.0,
                         "peak_source": f"{peaks['source']} cuBLAS bf16 burst", "ms_per_launch": gemm_ms,
                         "ms_per_launch_note": "CUDA events around the call: the 256-byte header memset and the launch",
                         "last_launch_ms_in_kernel": last_ms_in_kernel, "sustained_matmul_only": gemm_sustained,
                         "sm_mhz_in_kernel": gemm_mhz,
                         "frac_of_tensor_peak_at_kernel_clock": achieved / at_clock if achieved and at_clock else None,
                         "frac_of_sustained": achieved / peaks["bf16_sustained"] if achieved else None,
                         "frac_of_2250_datasheet": achieved / DATASHEET_TFLOPS if achieved else None,
                         "step_frac_of_burst": value / world / peak,
                         "step_frac_of_2250_datasheet": value / world / DATASHEET_TFLOPS},
            "sustained": sustained,
            "cpu_baseline": cpu,
            "qdq_gbs": qdq,
        }
        if other is not None:
            line["other_workloads"] = other
        print(json.dumps(line))
    replicas.finish()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sections", default=",".join(SECTIONS),
                    help="measurements beside the headline: roofline, sustained, qdq, e2e, cpu, configs (the other named "
                         "workloads; cfg1 / cfg3 / cfg4 / cfg5 pick single ones); all by default (empty string: none)")
    ap.add_argument("--region-seconds", type=float, default=1.0,
                    help="minimum length of the timed regions of the other named workloads (0 for profiler captures)")
    ap.add_argument("--shape", default=None, help="M,N,K of a smaller case (profiler captures only)")
    ap.add_argument("--in-kernel-qdq", action="store_true",
                    help="run the step with QF_FUSED_QDQ (quantize the staged tiles inside the matmul kernel) instead of the default path")
    ap.add_argument("--dry-run", action="store_true",
                    help="launch and timing protocol only (gloo ranks that sleep; no GPU): checks that --gpus N starts N ranks")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not under torchrun: start the ranks ourselves, one per GPU
        raise SystemExit(spawn_ranks(args.gpus, sys.argv[1:]))
    if args.shape:
        _set_shape(args.shape)
    if args.dry_run:
        run_dry(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
