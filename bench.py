#!/usr/bin/env python
"""Benchmark of the UE5M3-FP4 per-linear hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic input shaped like the
8B-hybrid linears: tokens M = 8192, in-features K = 4096, out-features N = 16384, BF16:
    quantize X (1D rows and 1D columns, RNE, both from one read), W (2D tiles + transposed copy, RNE), dY (1D rows, SR),
    dY (1D columns, SR);  GEMMs fprop Y = X W^T, dgrad dX = dY W, wgrad dW = dY^T X;
    tensor maxima are sampled at step 0 and held (re-sampled every 50 steps).
The reported value is the whole-step rate in TFLOP/s (GEMM flops only: 3 * 2 M K N per step, the
quantization time is inside the step).  The roofline object covers the dominant kernel (the GEMM);
the `quantizer` object reports the streaming kernels against the HBM roofline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--sweep]

With N > 1 (launched by torchrun) every rank runs the same workload on its own tokens: the path
shards over tokens without any exchange, so scaling is "weak" and no collective is on the data path.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
`--sweep` prints the quantizer bandwidth sweep (2^20 .. 2^30 elements) instead of the step benchmark.
`--stack` times every eligible linear of one 8B-hybrid-shaped layer stack at 16384 tokens.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

M_TOK, K_IN, N_OUT = 8192, 4096, 16384
WORKLOAD = "linear fwd+bwd M=8192 K=4096 N=16384 bf16 (fprop+dgrad+wgrad, 5 quantized operands from 4 launches, SR on dY)"
METRIC = "fwd+bwd block-scaled linear throughput (quantize + 3 GEMMs)"
UNIT = "TFLOP/s"
FLOPS_PER_STEP = 3 * 2 * M_TOK * K_IN * N_OUT


def set_shape(m, k, n):
    """Profiling aid: run the same step on another linear shape (the JSON line then names it)."""
    global M_TOK, K_IN, N_OUT, WORKLOAD, FLOPS_PER_STEP, GEMM_FLOPS, KERNEL_BYTES
    M_TOK, K_IN, N_OUT = m, k, n
    WORKLOAD = f"NON-DEFAULT profiling shape: linear fwd+bwd M={m} K={k} N={n} bf16"
    FLOPS_PER_STEP = 3 * 2 * m * k * n
    GEMM_FLOPS = 2 * m * k * n
    KERNEL_BYTES = kernel_bytes()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------------------------------------
# CPU oracle arm (the benchmark's cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------
SAMPLE_M, SAMPLE_N = 512, 1024
SAMPLE_DESC = (f"same linear cut to M={SAMPLE_M} tokens, K={K_IN}, N={SAMPLE_N}: 5 oracle quantizations + 3 exact "
               "oracle GEMMs, all host threads")


def oracle_sample_inputs():
    import synth_inputs as si
    X = si.to_numpy_bits(si.channel_scaled_activation(SAMPLE_M, K_IN, seed=1))
    W = si.to_numpy_bits(si.weight(SAMPLE_N, K_IN, seed=2))
    dY = si.to_numpy_bits(si.heavy_tailed_gradient(SAMPLE_M, SAMPLE_N, seed=3))
    return X, W, dY


def oracle_step(X, W, dY, g, seed):
    import oracle
    qx = oracle.quantize(X, 0, 0, g[0])
    qw = oracle.quantize(W, 2, 0, g[1], want_t=True)
    qg = oracle.quantize(dY, 0, 1, g[2], seed=4 * seed)
    qgt = oracle.quantize(dY, 1, 1, g[2], seed=4 * seed + 1)
    qxt = oracle.quantize(X, 1, 0, g[0])
    oracle.gemm(qx["payload"], qx["scales"], False, qx["decode"], qw["payload"], qw["scales"], True, qw["decode"])
    oracle.gemm(qg["payload"], qg["scales"], False, qg["decode"], qw["payload_t"], qw["scales_t"], True, qw["decode"])
    oracle.gemm(qgt["payload"], qgt["scales"], False, qgt["decode"], qxt["payload"], qxt["scales"], False, qxt["decode"])


def time_oracle(steps: int, warmup: int):
    import oracle
    X, W, dY = oracle_sample_inputs()
    g = (oracle.amax(X), oracle.amax(W), oracle.amax(dY))
    for s in range(warmup):
        oracle_step(X, W, dY, g, s)
    t0 = time.perf_counter()
    for s in range(steps):
        oracle_step(X, W, dY, g, warmup + s)
    dt = (time.perf_counter() - t0) / steps
    flops = 3 * 2 * SAMPLE_M * K_IN * SAMPLE_N
    return flops / dt / 1e12, dt, oracle.num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, min(args.steps, 3))
    warmup = min(args.warmup, 1)
    val, dt, cores = time_oracle(steps, warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int128 exact sum / f32 stepwise quantizer", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": SAMPLE_DESC},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": SAMPLE_DESC},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi clock / throttle-reason samples of this rank's GPU while a region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device):
        import torch
        self.proc = None
        self.path = None
        try:
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            self.gpu_id = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            self.gpu_id = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            cmd = ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "25"]
            if self.gpu_id:
                cmd += ["-i", self.gpu_id]
            self.proc = subprocess.Popen(cmd, stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def wait_first_sample(self, timeout=20.0):
        t0 = time.time()
        while self.proc is not None and time.time() - t0 < timeout:
            try:
                if os.path.getsize(self.path) > 0:
                    return
            except OSError:
                return
            time.sleep(0.05)

    def mark(self):
        """Samples written before this point (warm-up) are not counted."""
        try:
            with open(self.path) as f:
                self.skip = sum(1 for _ in f)
        except Exception:
            self.skip = 0

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        try:
            with open(self.path) as f:
                for line in f:
                    c = [v.strip() for v in line.split(",")]
                    if len(c) < 7:
                        continue
                    try:
                        rows.append((float(c[0]), float(c[1]), float(c[2]), c[3:7]))
                    except ValueError:
                        continue
            os.unlink(self.path)
        except Exception:
            pass
        skip = getattr(self, "skip", 0)
        # a timed region shorter than the sampling interval may hold no sample: then the last samples of the warm-up
        # (the same launch sequence, directly before the region) stand in, and the record says so
        picked = rows[skip:]
        if not picked and rows:
            picked = rows[-3:]
            out["note"] = "no sample fell inside the timed region; these are the last samples of the warm-up before it"
        sm, mx, pw, reasons = [], [], [], set()
        for a, b, c_, flags in picked:
            sm.append(a); mx.append(b); pw.append(c_)
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), flags):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), power_w_max=max(pw), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


class LinearStep:
    """Pre-allocated buffers and the launch sequence of one fwd+bwd step."""
    KERNELS = ("q_x_dual", "q_w_2d", "gemm_fprop", "q_dy_row_sr", "gemm_dgrad", "q_dy_col_sr", "gemm_wgrad")

    def __init__(self, device, seed=0, scale_layout=0, gemm_path="auto"):
        import torch
        import paper_2609_02846_b200 as lib
        import synth_inputs as si
        self.torch, self.lib, self.dev = torch, lib, device
        self.X = si.channel_scaled_activation(M_TOK, K_IN, seed=seed * 3 + 1, device=device)
        self.W = si.weight(N_OUT, K_IN, seed=seed * 3 + 2, device=device)
        self.dY = si.heavy_tailed_gradient(M_TOK, N_OUT, seed=seed * 3 + 3, device=device)
        self.cx, self.cw, self.cg = lib.AmaxCache(50), lib.AmaxCache(50), lib.AmaxCache(50)
        self.scale_layout = scale_layout
        self.q = {}
        self.Y = torch.empty((M_TOK, N_OUT), dtype=torch.bfloat16, device=device)
        self.dX = torch.empty((M_TOK, K_IN), dtype=torch.bfloat16, device=device)
        self.dW = torch.empty((N_OUT, K_IN), dtype=torch.bfloat16, device=device)
        self.launches = 0
        # auto: ue5m3_gemm (scale preparation, native FP4 kernel, FP16 kernel: three launches, one does the product);
        # fp16: ue5m3_gemm_fp16 (the FP16 reconstruction kernel alone)
        self.gemm = lib.gemm if gemm_path == "auto" else lib.gemm_fp16
        self.gemm_launches = 3 if gemm_path == "auto" else 1

    def _timed(self, name, fn, ev):
        if ev is None:
            return fn()
        a, b = self.torch.cuda.Event(enable_timing=True), self.torch.cuda.Event(enable_timing=True)
        a.record()
        r = fn()
        b.record()
        ev.setdefault(name, []).append((a, b))
        return r

    def run(self, step, ev=None, per_kernel=False):
        """One step.  With `ev`, CUDA events bracket every GEMM launch and every GROUP of consecutive quantizer
        launches (names in QUANT_GROUPS), so that the quantizer time of a step has no event gaps inside a group;
        `per_kernel=True` brackets every quantizer launch separately instead (breakdown pass, not the timed region)."""
        lib = self.lib
        refresh = self.cx.refreshes_at(step)
        gx, gw, gg = self.cx.get(self.X, step), self.cw.get(self.W, step), self.cg.get(self.dY, step)
        self.launches += 3 if refresh else 0
        sl = self.scale_layout
        q = self.q
        evk = ev if per_kernel else None
        evg = None if per_kernel else ev

        def fwd_quant():
            # X is needed along K (fprop) and along the tokens (wgrad): both operands come from ONE read of X
            q["x"], q["xt"] = self._timed("q_x_dual", lambda: lib.quantize_dual(
                self.X, lib.ROUND_RNE, gx, 448.0, 448.0, scale_layout=sl,
                out=(q["x"], q["xt"]) if "x" in q else None), evk)
            q["w"] = self._timed("q_w_2d", lambda: lib.quantize(self.W, lib.LAYOUT_2D, lib.ROUND_RNE, gw, 448.0,
                                                                want_transpose=True, out=q.get("w")), evk)

        def dgrad_quant():
            q["g"] = self._timed("q_dy_row_sr", lambda: lib.quantize(self.dY, lib.LAYOUT_1D_ROW, lib.ROUND_SR, gg, 448.0,
                                                                     seed=4 * step, scale_layout=sl, out=q.get("g")), evk)

        def wgrad_quant():
            q["gt"] = self._timed("q_dy_col_sr", lambda: lib.quantize(self.dY, lib.LAYOUT_1D_COL, lib.ROUND_SR, gg, 448.0,
                                                                      seed=4 * step + 1, scale_layout=sl, out=q.get("gt")), evk)

        self._timed("quant_fwd", fwd_quant, evg)
        self._timed("gemm_fprop", lambda: self.gemm(lib.FPROP, q["x"], q["w"], out=self.Y), ev)
        self._timed("quant_dgrad", dgrad_quant, evg)
        self._timed("gemm_dgrad", lambda: self.gemm(lib.DGRAD, q["g"], q["w"].transposed(), out=self.dX), ev)
        self._timed("quant_wgrad", wgrad_quant, evg)
        self._timed("gemm_wgrad", lambda: self.gemm(lib.WGRAD, q["gt"], q["xt"], out=self.dW), ev)
        self.launches += 4 + 3 * self.gemm_launches


    def gemm_kernels(self):
        """Which kernel ue5m3_gemm uses for each of the three products of the step just run: ue5m3_gemm_native says in its
        workspace whether every scale row of the two operands had a window (then it did the product)."""
        lib, q, torch = self.lib, self.q, self.torch
        out = {}
        for name, a, b, c in (("gemm_fprop", q["x"], q["w"], self.Y), ("gemm_dgrad", q["g"], q["w"].transposed(), self.dX),
                              ("gemm_wgrad", q["gt"], q["xt"], self.dW)):
            if self.gemm_launches == 1 or a.Kc % 256:
                out[name] = "gemm_kernel"
                continue
            ws = lib.gemm_native_workspace(a, b)
            lib.gemm_native(lib.FPROP, a, b, out=c, workspace=ws)
            torch.cuda.synchronize()
            ok = lib.native_windows(ws, a, b)[0]
            out[name] = "gemm_native_kernel" if ok else "gemm_kernel"
        return out


QUANT_GROUPS = {"quant_fwd": ("q_x_dual", "q_w_2d"), "quant_dgrad": ("q_dy_row_sr",), "quant_wgrad": ("q_dy_col_sr",)}
NOMINAL_HBM_GBS, NOMINAL_BF16_TFLOPS = 8000.0, 2250.0


# algorithmic bytes of each streaming kernel per launch (BF16 in, payload + scales out)
def _quant_bytes(rows, cols, layout, transposed_copy=False):
    n = rows * cols
    if layout == 2:
        return n * 2 + n // 2 * (2 if transposed_copy else 1) + n // 256 * (2 if transposed_copy else 1)
    return n * 2 + n // 2 + n // 16


def kernel_bytes():
    nx = M_TOK * K_IN
    return {
        "q_x_dual": nx * 2 + 2 * (nx // 2 + nx // 16),          # one read of X, row and column operand out
        "q_w_2d": _quant_bytes(N_OUT, K_IN, 2, True),
        "q_dy_row_sr": _quant_bytes(M_TOK, N_OUT, 0), "q_dy_col_sr": _quant_bytes(M_TOK, N_OUT, 1),
    }


KERNEL_BYTES = kernel_bytes()
GEMM_FLOPS = 2 * M_TOK * K_IN * N_OUT
# dram__bytes_read.sum + dram__bytes_write.sum per GEMM launch of the default workload (mean of fprop, dgrad, wgrad;
# one ncu pass each; summaries in profiles/gemm_kernel_M9472_K4096_N1024_ncu_full.txt and
# profiles/gemm_native_kernel_linear_M8192_K4096_N16384_ncu_full.txt).  Algorithmic bytes: 238 MB per launch.
GEMM_DRAM_TRAFFIC_BYTES = {"gemm_kernel": (150.3e6 + 220.9e6 + 195.0e6 + 48.0e6 + 100.7e6 + 99.1e6) / 3,
                           "gemm_native_kernel": (167.7e6 + 221.7e6 + 219.4e6 + 51.6e6 + 100.3e6 + 101.6e6) / 3}
NOMINAL_FP4_OVER_BF16 = 4.0      # dense tensor peaks of the part: 9 PFLOP/s FP4, 2.25 PFLOP/s BF16


def max_over_ranks(ms: float, world: int, device=None) -> float:
    """Step time of the job = the slowest rank's (MAX all-reduce of one number; no data-path collective)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(ms_per_step: float, world: int) -> float:
    """Whole-job TFLOP/s: every rank runs the same per-rank workload on its own tokens (weak scaling)."""
    return world * FLOPS_PER_STEP / (ms_per_step * 1e-3) / 1e12


def run_ours(args):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    import paper_2609_02846_b200 as lib
    if not os.path.exists(lib.library_path()):
        if local == 0:
            from paper_2609_02846_b200.build import build_library
            build_library()                     # build product missing (fresh tree): compile it once per node
        if world > 1:
            dist.barrier()
    peaks = measured_peaks()
    step = LinearStep(dev, seed=rank, scale_layout=args.scale_layout, gemm_path=args.gemm_path)
    K, Wm = args.steps, max(args.warmup, 3)

    sampler = ClockSampler(dev)
    if rank == 0:
        sampler.start()      # started before the warm-up: its own start-up must not fall into the timed region
        sampler.wait_first_sample()
    for s in range(Wm):
        step.run(s)
    barrier()
    launches0 = step.launches
    sampler.mark()
    ev = {}
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t0.record()
    for s in range(K):
        step.run(Wm + s, ev)
    t1.record()
    barrier()
    clocks = sampler.stop()
    total_ms = t0.elapsed_time(t1)
    status = lib.last_device_status()
    if status != 0:
        raise SystemExit(f"device status {lib.status_string(status)}")
    total_ms = max_over_ranks(total_ms, world, dev)
    ms_per_step = total_ms / K
    value = job_value(ms_per_step, world)
    gpu_launches = step.launches - launches0
    gemm_kernels = step.gemm_kernels()          # after the timed region: it launches each product once more

    per_kernel = {k: statistics.mean(a.elapsed_time(b) for a, b in v) for k, v in ev.items()}
    gemm_ms = statistics.mean(per_kernel[k] for k in ("gemm_fprop", "gemm_dgrad", "gemm_wgrad"))
    gemm_tflops = GEMM_FLOPS / (gemm_ms * 1e-3) / 1e12
    # quantizers inside the timed region: one event pair per group of consecutive quantizer launches
    qbytes = float(sum(KERNEL_BYTES.values()))
    qms = sum(per_kernel[g] for g in QUANT_GROUPS)
    quant = {"timing": "inside the timed region: one CUDA-event pair around each group of consecutive quantizer launches "
                       "(no event between the launches of a group)",
             "groups": {g: {"kernels": list(ks), "ms": round(per_kernel[g], 4),
                            "GB/s": round(sum(KERNEL_BYTES[k] for k in ks) / (per_kernel[g] * 1e-3) / 1e9, 1)}
                        for g, ks in QUANT_GROUPS.items()},
             "all": {"ms": round(qms, 4), "GB/s": round(qbytes / (qms * 1e-3) / 1e9, 1),
                     "frac_of_measured_hbm": round(qbytes / (qms * 1e-3) / 1e9 / peaks["hbm_gbs"], 3),
                     "frac_of_nominal_8TBs": round(qbytes / (qms * 1e-3) / 1e9 / NOMINAL_HBM_GBS, 3),
                     "share_of_step": round(qms / ms_per_step, 3)}}

    # ---- breakdown pass (outside the timed region): every quantizer launch with its own event pair ----
    evb = {}
    for s_ in range(min(K, 20)):
        step.run(Wm + K + s_, evb, per_kernel=True)
    torch.cuda.synchronize()
    pk = {}
    for k, nbytes in KERNEL_BYTES.items():
        ms = statistics.mean(a.elapsed_time(b) for a, b in evb[k])
        gbs = nbytes / (ms * 1e-3) / 1e9
        pk[k] = {"ms": round(ms, 4), "GB/s": round(gbs, 1), "frac_of_measured_hbm": round(gbs / peaks["hbm_gbs"], 3)}
    quant["per_kernel"] = pk
    quant["per_kernel_timing"] = ("separate pass after the timed region, one event pair per launch: each figure includes the "
                                  "launch gap of a single short kernel (a few microseconds)")

    # ---- sustained leg: at least two seconds of back-to-back steps under the power cap ----
    sustained = None
    if rank == 0 and world == 1 and not args.no_sustained:
        sampler2 = ClockSampler(dev)
        sampler2.start()
        sampler2.wait_first_sample()
        n_sus = max(50, int(2200.0 / ms_per_step))
        for s_ in range(20):
            step.run(Wm + K + 20 + s_)
        torch.cuda.synchronize()
        sampler2.mark()
        evs = {}
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for s_ in range(n_sus):
            step.run(Wm + K + 40 + s_, evs)
        s1.record()
        torch.cuda.synchronize()
        clk2 = sampler2.stop()
        sus_ms = s0.elapsed_time(s1) / n_sus
        sus_gemm_ms = statistics.mean(a.elapsed_time(b) for k in ("gemm_fprop", "gemm_dgrad", "gemm_wgrad") for a, b in evs[k])
        sus_gemm = GEMM_FLOPS / (sus_gemm_ms * 1e-3) / 1e12
        sustained = {"seconds": round(sus_ms * n_sus * 1e-3, 2), "steps": n_sus, "ms_per_step": round(sus_ms, 4),
                     "tflops_per_step": round(FLOPS_PER_STEP / (sus_ms * 1e-3) / 1e12, 1),
                     "gemm_tflops_per_launch": round(sus_gemm, 1), "gemm_avg_launch_ms": round(sus_gemm_ms, 4),
                     "gemm_over_bf16_sustained_peak": round(sus_gemm / peaks["bf16_tflops_sustained"], 3),
                     "gemm_over_bf16_burst_peak": round(sus_gemm / peaks["bf16_tflops"], 3),
                     "gemm_over_bf16_nominal_2250": round(sus_gemm / NOMINAL_BF16_TFLOPS, 3),
                     "gemm_frac_of_own_pipe_sustained": round(sus_gemm / (peaks["bf16_tflops_sustained"] * (
                         NOMINAL_FP4_OVER_BF16 if all(v == "gemm_native_kernel" for v in gemm_kernels.values()) else 1.0)), 3),
                     "clocks": clk2,
                     "gemm_launch_ms_x_sm_mhz": None if not clk2.get("sm_mhz") else round(sus_gemm_ms * clk2["sm_mhz"], 1)}

    # ---- end to end: host buffers in, results back to the host, every step ----
    # Three streams and two sets of device buffers: the copy-in of step s+1 and the copy-out of step s-1 run under
    # the compute of step s, as a training pipeline would; every step still moves all of its inputs and outputs.
    e2e = None
    if rank == 0 or world > 1:
        Xh, Wh, dYh = (t.cpu().pin_memory() for t in (step.X, step.W, step.dY))
        Yh, dXh, dWh = (torch.empty_like(t, device="cpu").pin_memory() for t in (step.Y, step.dX, step.dW))
        names = ("X", "W", "dY", "Y", "dX", "dW")
        bufs = [tuple(getattr(step, n) for n in names), tuple(torch.empty_like(getattr(step, n)) for n in names)]
        s_in, s_out, main = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev), torch.cuda.current_stream()
        in_done, comp_done, out_done = [None, None], [None, None], [None, None]
        n_e2e = max(2, min(K, 50))        # long enough that filling and draining the three-stage pipeline is amortised

        def e2e_step(s):
            b_ = s & 1
            X_, W_, dY_, Y_, dX_, dW_ = bufs[b_]
            with torch.cuda.stream(s_in):
                if comp_done[b_] is not None:
                    s_in.wait_event(comp_done[b_])             # the step that last read these input buffers
                X_.copy_(Xh, non_blocking=True); W_.copy_(Wh, non_blocking=True); dY_.copy_(dYh, non_blocking=True)
                in_done[b_] = torch.cuda.Event(); in_done[b_].record(s_in)
            main.wait_event(in_done[b_])
            if out_done[b_] is not None:
                main.wait_event(out_done[b_])                  # the copy-out that last read these output buffers
            for n, t in zip(names, bufs[b_]):
                setattr(step, n, t)
            step.run(s)
            comp_done[b_] = torch.cuda.Event(); comp_done[b_].record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(comp_done[b_])
                Yh.copy_(Y_, non_blocking=True); dXh.copy_(dX_, non_blocking=True); dWh.copy_(dW_, non_blocking=True)
                out_done[b_] = torch.cuda.Event(); out_done[b_].record(s_out)

        for s in range(2):
            e2e_step(Wm + K + 100000 + s)
        main.wait_stream(s_out)
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for s in range(n_e2e):
            e2e_step(Wm + K + 100002 + s)
        main.wait_stream(s_in); main.wait_stream(s_out)
        b.record()
        barrier()
        e_ms = max_over_ranks(a.elapsed_time(b), world, dev) / n_e2e
        h2d = sum(t.numel() * t.element_size() for t in (Xh, Wh, dYh))
        d2h = sum(t.numel() * t.element_size() for t in (Yh, dXh, dWh))
        e2e = {"value": job_value(e_ms, world), "unit": UNIT, "ms_per_step": e_ms, "steps": n_e2e,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "schedule": "copy-in, compute and copy-out of consecutive steps overlap on three streams"}

    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            v, dt, cores = time_oracle(1, 0)
            cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": SAMPLE_DESC, "seconds": round(dt, 2)}
        # Denominator from this run's own clock record: a short region at full clocks is compared with the burst
        # figure of the measured cuBLAS BF16 peak, a long or power-capped one with the sustained figure.  When the three
        # products ran on the native FP4 kernel the peak is that of its own pipe: the measured BF16 figure times the
        # nominal dense FP4 : BF16 ratio (9 : 2.25 PFLOP/s).
        region_s = total_ms * 1e-3
        capped = "sw_power_cap" in (clocks.get("reasons") or [])
        use_burst = region_s < 1.0 and not capped
        native = all(v == "gemm_native_kernel" for v in gemm_kernels.values())
        ratio = NOMINAL_FP4_OVER_BF16 if native else 1.0
        peak = ratio * (peaks["bf16_tflops"] if use_burst else peaks["bf16_tflops_sustained"])
        kernel = "gemm_native_kernel" if native else "gemm_kernel"
        roofline = {"bound": "tensor", "kernel": kernel, "kernel_per_gemm": gemm_kernels,
                    "achieved": gemm_tflops, "peak": peak, "unit": "TFLOP/s", "frac": gemm_tflops / peak,
                    "peak_source": peaks["source"] + " cuBLAS BF16" + (" x 4 (nominal dense FP4 : BF16), " if native else ", ") +
                                   ("burst: timed region %.3f s, no power cap seen" % region_s if use_burst
                                    else "sustained: timed region %.3f s%s" % (region_s, ", sw_power_cap seen" if capped else "")),
                    "achieved_over_bf16_burst_peak": gemm_tflops / peaks["bf16_tflops"],
                    "achieved_over_bf16_sustained_peak": gemm_tflops / peaks["bf16_tflops_sustained"],
                    "achieved_over_bf16_nominal_2250": gemm_tflops / NOMINAL_BF16_TFLOPS,
                    "achieved_over_fp4_nominal_9000": gemm_tflops / (NOMINAL_BF16_TFLOPS * NOMINAL_FP4_OVER_BF16),
                    "avg_launch_ms": gemm_ms,
                    "avg_launch_ms_note": "one ue5m3_gemm call: with --gemm-path auto that is the kernel that prepares the scales, the kernel "
                                          "that does the product and the other kernel's immediate return",
                    "avg_launch_ms_x_sm_mhz": None if not clocks.get("sm_mhz") else round(gemm_ms * clocks["sm_mhz"], 1),
                    "traffic": GEMM_DRAM_TRAFFIC_BYTES.get(kernel) if (M_TOK, K_IN, N_OUT) == (8192, 4096, 16384) else None,
                    "traffic_unit": "bytes of DRAM read+write per launch (ncu, mean of the three GEMMs)",
                    "per_gemm_ms": {k: round(per_kernel[k], 4) for k in ("gemm_fprop", "gemm_dgrad", "gemm_wgrad")}}
        sweep = None
        if world == 1 and not args.no_sweep:
            sweep = quantizer_sweep_cells(dev, peaks)
        # A region of a few hundred milliseconds holds a handful of samples, and the power-cap flag is not up in every one
        # of them while the clock is already down; the sustained leg that follows runs the same steps for two seconds.
        if (clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and clocks["sm_mhz"] < 0.97 * clocks["sm_max_mhz"]
                and not clocks.get("reasons") and sustained and sustained["clocks"].get("reasons")):
            clocks["note"] = ("median clock below the maximum with no reason flagged in this region's %d samples; the sustained leg "
                              "after it (the same steps for %.1f s) records %s at up to %.0f W" % (
                                  clocks.get("samples", 0), sustained["seconds"], "+".join(sustained["clocks"]["reasons"]),
                                  sustained["clocks"].get("power_w_max") or 0.0))
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "fp4 (e2m1 operands, 8-bit block scales, f32 accumulate)" if native else "f16 (exact reconstruction of e2m1 x ue5m3, f32 accumulate)",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "gemm_path": args.gemm_path, "tokens_per_gpu": M_TOK, "l2": f"inputs ({2 * (M_TOK * K_IN + N_OUT * K_IN + M_TOK * N_OUT) >> 20} MiB per step) exceed the 126 MB L2",
                       "scale_layout": "tiled" if args.scale_layout else "rowmajor", "amax": "sampled at step 0, held 50 steps"},
            "roofline": roofline,
            "quantizer": quant, "sustained": sustained, "quantizer_sweep": sweep,
            "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": gpu_launches, "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_stack(args):
    """One 8B-hybrid-shaped layer stack at 16384 tokens: every eligible linear fwd+bwd, per-linear and aggregate TFLOP/s."""
    import torch
    import paper_2609_02846_b200 as lib
    import synth_inputs as si
    dev = torch.device("cuda", 0)
    tokens, out, total_flops, total_ms = 16384, {}, 0.0, 0.0
    for name, k, n in si.LAYER_STACK:
        set_shape(tokens, k, n)
        step = LinearStep(dev, seed=7)
        for s in range(3):
            step.run(s)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        iters = max(5, args.steps // 10)
        a.record()
        for s in range(iters):
            step.run(3 + s)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / iters
        out[name] = {"in": k, "out": n, "ms": round(ms, 4), "TFLOP/s": round(FLOPS_PER_STEP / (ms * 1e-3) / 1e12, 1)}
        total_flops += FLOPS_PER_STEP
        total_ms += ms
        del step
        torch.cuda.empty_cache()
    status = lib.last_device_status()
    print(json.dumps({"workload": "layer stack fwd+bwd, 16384 tokens, six linears", "linears": out, "total_flop": total_flops,
                      "ms": round(total_ms, 4), "TFLOP/s": round(total_flops / (total_ms * 1e-3) / 1e12, 1),
                      "device_status": status}), flush=True)


# FP32 lanes per SM per clock and directed-rounding additions per output cell and 64-product group
# (6 for the exactness interval of the four block sums, 1 toward zero into the running total).
PROBE_FP32_LANES_PER_SM, PROBE_ADDS_PER_GROUP = 128, 7


def run_probe(args):
    """The three GEMMs of the benchmark linear under the output model of Section 6.2 (ue5m3_gemm_probe_matched),
    each timed alone on the quantized operands of one step; the oracle's model GEMM timed beside it on a sample."""
    import torch
    import paper_2609_02846_b200 as lib
    dev = torch.device("cuda", 0)
    step = LinearStep(dev, seed=7)
    step.run(0)
    q = step.q
    props = torch.cuda.get_device_properties(dev)
    sampler = ClockSampler(dev)
    sampler.start()
    sampler.wait_first_sample()
    jobs = (("fprop", lib.FPROP, q["x"], q["w"], step.Y), ("dgrad", lib.DGRAD, q["g"], q["w"].transposed(), step.dX),
            ("wgrad", lib.WGRAD, q["gt"], q["xt"], step.dW))
    iters = max(3, args.steps // 20)
    per_op, total_ms = {}, 0.0
    for name, op, a, b, out in jobs:
        for _ in range(max(3, args.warmup)):
            lib.gemm_probe_matched(op, a, b, out=out)
        torch.cuda.synchronize()
        if name == "fprop":
            sampler.mark()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            lib.gemm_probe_matched(op, a, b, out=out)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / iters
        per_op[name] = {"ms": round(ms, 4), "TFLOP/s": round(2.0 * M_TOK * K_IN * N_OUT / (ms * 1e-3) / 1e12, 1)}
        total_ms += ms
    clocks = sampler.stop()
    status = lib.last_device_status()
    tflops = 3 * 2.0 * M_TOK * K_IN * N_OUT / (total_ms * 1e-3) / 1e12
    sm_hz = (clocks.get("sm_max_mhz") or 1965.0) * 1e6
    peak = props.multi_processor_count * PROBE_FP32_LANES_PER_SM * sm_hz / PROBE_ADDS_PER_GROUP * 128 / 1e12
    line = {"metric": "probe_matched_gemm_tflops", "value": round(tflops, 1), "unit": "TFLOP/s", "n_gpus": 1,
            "dtype": "e2m1 x ue5m3 operands, exact 64-product partials, f32 toward-zero accumulation",
            "config": {"workload": f"fprop, dgrad, wgrad of linear M={M_TOK} K={K_IN} N={N_OUT} under the Section 6.2 output model, "
                                   "grid 1/1024, operands from one quantized step", "launches_timed_per_gemm": iters},
            "per_gemm": per_op,
            "roofline": {"bound": "alu", "achieved": round(tflops, 1), "peak": round(peak, 1), "unit": "TFLOP/s",
                         "frac": round(tflops / peak, 3), "traffic": None,
                         "peak_derivation": f"{props.multi_processor_count} SMs x {PROBE_FP32_LANES_PER_SM} FP32 lanes x max SM clock / "
                                            f"{PROBE_ADDS_PER_GROUP} directed-rounding adds per cell and 64-group x 128 flop per cell and group"},
            "device_status": status, "clocks": clocks}
    if not args.no_cpu_baseline:
        import oracle
        qa, qb = q["x"], q["w"]
        rows, cols = 64, 64
        ap, asc = qa.payload[:rows].cpu().numpy(), qa.scales[:rows].cpu().numpy()
        bp, bsc = qb.payload[:cols].cpu().numpy(), qb.scales[:cols // 16].cpu().numpy()
        t0 = time.perf_counter()
        reps = 0
        while time.perf_counter() - t0 < 10.0:
            oracle.gemm_probe(ap, asc, False, float(qa.decode.item()), bp, bsc, True, float(qb.decode.item()), grid_d=1024)
            reps += 1
        dt = (time.perf_counter() - t0) / reps
        line["cpu_baseline"] = {"value": round(2.0 * rows * cols * K_IN / dt / 1e12, 6), "unit": "TFLOP/s", "cores": oracle.num_threads(),
                                "kind": "oracle", "sample": f"fprop cut to {rows} x {cols} outputs, K={K_IN}, about 10 s"}
    print(json.dumps(line), flush=True)


def run_current(args):
    """The per-batch (D = 1) reference policy: tensor maximum + quantization of X- and dY-sized tensors, as two calls and
    as the one ue5m3_quantize_current call (the second pass directly behind the first on the same stream)."""
    import torch
    import paper_2609_02846_b200 as lib
    import synth_inputs as si
    dev = torch.device("cuda", 0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    out = {}
    for name, rows, cols in (("X", M_TOK, K_IN), ("dY", M_TOK, N_OUT)):
        x = si.channel_scaled_activation(rows, cols, seed=3, device=dev)
        g = lib.sample_amax(x)
        q = lib.quantize(x, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, g)
        res = {}
        for label, fn in (("amax", lambda: lib.sample_amax(x, g)),
                          ("quantize", lambda: lib.quantize(x, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, g, out=q)),
                          ("quantize_current", lambda: lib.quantize_current(x, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, amax_out=g, out=q))):
            ts = []
            for _ in range(max(5, args.steps // 10)):
                flush.fill_(1)                                   # start every measurement with x out of L2
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); fn(); b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b) * 1e3)
            res[label] = round(statistics.median(ts), 1)
        res["MiB"] = rows * cols * 2 >> 20
        out[name] = res
    print(json.dumps({"workload": "per-batch reference policy, BF16, 1D rows, RNE; microseconds, L2 flushed before each measurement",
                      "tensors": out}), flush=True)


def _graph_time(torch, fn, flush, nbytes, warmup, iters, use_graph=True):
    """Median and best time (ms) of one launch replayed from a CUDA graph; L2 flushed before each replay when the
    tensor would otherwise fit in it.  `use_graph=False` launches directly (for captures under a profiler)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    # one launch captured in a CUDA graph: the replay keeps the Python/ctypes call (5-10 us of host time)
    # out of the device timeline, which matters for the small tensors
    graph = None
    if use_graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            fn()
    ts = []
    for _ in range(iters):
        if nbytes < (256 << 20):
            flush.zero_()                      # inputs that fit in L2: flush it between timed launches
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        if graph is not None:
            graph.replay()
        else:
            fn()
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    del graph
    return statistics.median(ts), min(ts)


def sweep_row(torch, lib, si, dev, peaks, flush, log2n, warmup, iters, use_graph=True):
    """One size of the quantizer bandwidth sweep: BF16 [rows, 4096]; amax + {1D_ROW, 1D_COL, 2D} x {RNE, SR}, and a plain
    streaming kernel (elementwise int32 add) moving the same number of bytes as a 1D quantization (what any kernel can
    reach at this size under this timing)."""
    rows = (1 << log2n) // 4096
    x = si.row_scaled_tensor(rows, 4096, seed=log2n, device=dev)
    g = lib.sample_amax(x)
    cells = {"amax": (lambda: lib.sample_amax(x, g), rows * 4096 * 2)}
    for lname, layout in (("1d_row", 0), ("1d_col", 1), ("2d", 2)):
        for rname, rnd in (("rne", 0), ("sr", 1)):
            q = lib.quantize(x, layout, rnd, g, seed=1)
            cells[f"{lname}_{rname}"] = ((lambda layout=layout, rnd=rnd, q=q: lib.quantize(x, layout, rnd, g, seed=1, out=q)),
                                         _quant_bytes(rows, 4096, layout))
    half = _quant_bytes(rows, 4096, 0) // 2 // 1024 * 1024
    src = torch.zeros(half // 4, dtype=torch.int32, device=dev)
    dst = torch.empty(half // 4, dtype=torch.int32, device=dev)
    cells["copy_same_bytes"] = (lambda: torch.add(src, 1, out=dst), 2 * half)
    row = {"log2_elements": log2n}
    for name, (fn, nbytes) in cells.items():
        ms, best = _graph_time(torch, fn, flush, rows * 4096 * 2, warmup, iters, use_graph)
        gbs = nbytes / (ms * 1e-3) / 1e9
        row[name] = {"ms": round(ms, 4), "GB/s": round(gbs, 1), "frac_of_measured_hbm": round(gbs / peaks["hbm_gbs"], 3),
                     "frac_of_nominal_8TBs": round(gbs / NOMINAL_HBM_GBS, 3), "best_GB/s": round(nbytes / (best * 1e-3) / 1e9, 1)}
    return row


def quantizer_sweep_cells(dev, peaks, sizes=(25, 27, 29), warmup=20, iters=100):
    """The part of the bandwidth sweep that goes into the default JSON line: the operand sizes of the benchmark linear
    (2^25 = X, 2^27 = dY) and a large one."""
    import torch
    import paper_2609_02846_b200 as lib
    import synth_inputs as si
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    out = {"method": f"CUDA-graph replay of one launch, {warmup} warm-up + {iters} timed, median; L2 flushed before every "
                     "timed launch; copy_same_bytes = a plain streaming kernel (torch int32 add, read half / write half) moving the "
                     "bytes a 1D quantization moves: what any kernel reaches at that size under this timing",
           "sizes": [sweep_row(torch, lib, si, dev, peaks, flush, n, warmup, iters) for n in sizes]}
    del flush
    torch.cuda.empty_cache()
    return out


def run_sweep(args):
    """Quantizer-only bandwidth sweep: BF16 [rows, 4096], 2^20 .. 2^30 elements, {1D, 2D} x {RNE, SR} + amax."""
    import torch
    import paper_2609_02846_b200 as lib
    import synth_inputs as si
    dev = torch.device("cuda", 0)
    peaks = measured_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    out = []
    lo, hi = args.sweep_log2
    for log2n in range(lo, hi + 1, args.sweep_stride):
        row = sweep_row(torch, lib, si, dev, peaks, flush, log2n, args.sweep_warmup, args.sweep_iters, not args.sweep_no_graph)
        out.append(row)
        print(json.dumps(row), flush=True)
    return out


def run_sweep_oracle(args):
    """The oracle's quantizer on the host cores (all cores at 2^24 and 2^26 elements, one core at 2^24), rows x 4096,
    GB/s of the same algorithmic bytes."""
    import oracle
    import synth_inputs as si
    all_cores = oracle.num_threads()
    for log2n, cores in ((24, all_cores), (26, all_cores), (24, 1)):
        rows = (1 << log2n) // 4096
        x = si.to_numpy_bits(si.row_scaled_tensor(rows, 4096, seed=log2n))
        oracle.set_num_threads(cores)
        g = oracle.amax(x)
        row = {"impl": "oracle", "log2_elements": log2n, "cores": cores}
        for lname, layout in (("1d_row", 0), ("1d_col", 1), ("2d", 2)):
            for rname, rnd in (("rne", 0), ("sr", 1)):
                t0 = time.perf_counter()
                oracle.quantize(x, layout, rnd, g, 448.0, 1)
                dt = time.perf_counter() - t0
                row[f"{lname}_{rname}"] = {"ms": round(dt * 1e3, 1), "GB/s": round(_quant_bytes(rows, 4096, layout) / dt / 1e9, 3)}
        t0 = time.perf_counter()
        oracle.amax(x)
        dt = time.perf_counter() - t0
        row["amax"] = {"ms": round(dt * 1e3, 2), "GB/s": round(rows * 4096 * 2 / dt / 1e9, 3)}
        print(json.dumps(row), flush=True)
    oracle.set_num_threads(all_cores)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--scale-layout", type=int, default=0, choices=[0, 1])
    ap.add_argument("--gemm-path", default="auto", choices=["auto", "fp16"],
                    help="auto: ue5m3_gemm picks the native FP4 kernel when the scale codes allow; fp16: the FP16 kernel alone")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the two-second sustained leg")
    ap.add_argument("--no-sweep", action="store_true", help="skip the quantizer sweep cells of the default line")
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--stack", action="store_true", help="time the six linears of the 8B-hybrid-shaped layer stack")
    ap.add_argument("--current", action="store_true", help="time the per-batch (D = 1) reference policy")
    ap.add_argument("--probe", action="store_true", help="time the GEMMs under the Section 6.2 output model")
    ap.add_argument("--sweep-iters", type=int, default=100)
    ap.add_argument("--sweep-warmup", type=int, default=20)
    ap.add_argument("--sweep-stride", type=int, default=1)
    ap.add_argument("--sweep-log2", type=int, nargs=2, default=[20, 30], metavar=("LO", "HI"),
                    help="smallest and largest log2(elements) of --sweep")
    ap.add_argument("--sweep-no-graph", action="store_true", help="--sweep: launch directly instead of replaying CUDA graphs")
    ap.add_argument("--sweep-no-oracle", action="store_true", help="--sweep: skip the oracle rows")
    ap.add_argument("--shape", default=None, help="M,K,N override for profiling runs (not the benchmark workload)")
    args = ap.parse_args()
    if args.shape:
        set_shape(*(int(v) for v in args.shape.split(",")))
    if args.impl == "reference":
        run_reference(args)
    elif args.sweep:
        run_sweep(args)
        if not args.sweep_no_oracle:
            run_sweep_oracle(args)
    elif args.stack:
        run_stack(args)
    elif args.probe:
        run_probe(args)
    elif args.current:
        run_current(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
