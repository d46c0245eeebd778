#!/usr/bin/env python
"""Benchmark of the W4A8 MSQ linear hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference]

A step is one pass of the whole hot path over one batch shaped like the paper's prefill
workload (Qwen2-7B-shaped down-projection, T = 1024 visual + 64 text tokens, K = 18944,
N = 3584, online 128-block Hadamard rotation): AIFS reorder of the [L, 3584] hidden rows,
position / segment remap, fused rotation + MSQ int8 quantizer, W4A8 tensor-core GEMM with the
dequant epilogue.  Calibration and weight packing are offline and untimed.  Inputs are
seeded synthetic tensors; several independent buffer sets are cycled so that every step
reads its operands from HBM rather than L2.

Prints ONE JSON line (rank 0).  `value` is device-resident throughput in TOPS (2*T*K*N
integer operations per step over all ranks / slowest rank's time); `e2e` is the same metric
through the C ABI with host buffers (H2D of the activations, D2H of the output inside the
timed region); `roofline` describes the dominant kernel (the GEMM) against the measured
tensor peak; `cpu_baseline` is the CPU oracle timed on this machine's host cores.
With --impl reference the oracle itself is the timed program.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "w4a8_msq_linear_prefill_throughput"
UNIT = "TOPS"
WORKLOAD = "config2: Qwen2-7B-shaped down_proj, T=1088 (1024 visual + 64 text), K=18944, N=3584, rot_block=128"
T_VIS, T_TXT, K_DIM, N_DIM, ROT, HIDDEN = 1024, 64, 18944, 3584, 128, 3584
SPANS = [(0, 16), (1, 512), (0, 16), (1, 512), (0, 32)]  # original (interleaved) token order


def ops_per_step(T=T_VIS + T_TXT):
    return 2.0 * T * K_DIM * N_DIM


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"],
                "bf16_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _poll(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._poll, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        if self.nv is not None and not self.samples:
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
            except Exception:
                pass
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------ oracle arm
def oracle_sample_rows():
    """Bounded sample of the workload for the CPU arms: 192 visual rows + all 64 text rows."""
    return np.concatenate([np.arange(0, 192), np.arange(T_VIS, T_VIS + T_TXT)])


def time_oracle(case, qw, s_w, s_v, s_t, rows, repeats):
    from oracle import mq_oracle as O
    from paper_2502_00425_b200 import synth
    seg = synth.segments_from_row_modality(case.seg.row_modality(case.T)[rows])
    x = case.x[rows]
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        O.linear_w4a8_msq(x, seg.seg_end, seg.seg_mod, s_v, s_t, case.rot_block, qw, s_w)
        times.append(time.perf_counter() - t0)
    return times


def host_threads():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, info):
    """The CPU oracle as the timed program (rank 0 only)."""
    if not info.is_main:
        return
    from oracle import mq_oracle as O
    from paper_2502_00425_b200 import synth
    case = synth.config2()
    qw, s_w = O.quantize_weight_int4(case.w)
    s_v, s_t = O.calibrate_static_scales(case.x_calib, case.seg_calib.seg_end, case.seg_calib.seg_mod, ROT)
    rows = oracle_sample_rows()
    time_oracle(case, qw, s_w, s_v, s_t, rows, args.warmup)
    times = time_oracle(case, qw, s_w, s_v, s_t, rows, args.steps)
    total = float(np.sum(times))
    value = ops_per_step(len(rows)) * args.steps / total / 1e12
    sample = f"{len(rows)} of 1088 rows (192 visual + 64 text), all K and N, per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8xint4->int32",
            "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ tensor-pipe microbenchmark
def mma_issue_microbenchmark(torch, B, dev, n_sms):
    """tcgen05.mma kind::i8 with fixed operands and no loads (the library's own probe): cycles per
    128 x N x 32 instruction on every SM at once, for the token-tile widths the GEMM uses."""
    out = {}
    n_mma = 4096
    for n_tok in (64, 128, 192, 224, 256):
        cyc = torch.zeros(n_sms, dtype=torch.int64, device=dev)
        st = torch.zeros(2, dtype=torch.int32, device=dev)
        for _ in range(2):
            B.mq_ubench_mma_i8(n_tok, n_mma, 1, 0, n_sms, cyc, st)
        torch.cuda.synchronize()
        per = float(cyc.cpu().double().mean()) / n_mma   # reduced on the host: no library kernel for it
        out["N%d" % n_tok] = {"cycles_per_mma": per, "ops_per_clk_sm": 2.0 * 128 * n_tok * 32 / per,
                              "status_ok": st.cpu().tolist() == [0, 0]}
    return out


def gemm_traffic_record():
    """DRAM bytes of one GEMM launch on the bench workload, from the ncu capture summarised under
    profiles/: valid only while the kernel source is the one that was captured."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "w4a8_gemm_config2_traffic.json")
    src = os.path.join(ROOT, "paper_2502_00425_b200", "csrc", "mq_gemm.cu")
    try:
        with open(path) as f:
            rec = json.load(f)
        with open(src, "rb") as f:
            sha = hashlib.sha256(f.read()).hexdigest()
    except Exception:
        return None, None
    if rec.get("mq_gemm_cu_sha256") != sha:
        return None, dict(rec, stale="mq_gemm.cu has changed since the capture")
    return rec.get("dram_bytes_per_launch"), rec


def variants_timing(torch, B, dev, T, K, N, rot, n_sets=4, reps=10):
    """The neighbouring settings on the config-2 shape, each as rotation + quantizer + GEMM (CUDA-graph
    replays over n_sets rotating copies, larger than L2 in total; random valid weight bytes: timing only,
    parity is covered by the tests): W4A8 per-channel (the hot path), group-wise W4 (g = 128), W8A8, W4A4."""
    g = torch.Generator(device="cpu").manual_seed(14)
    seg = B.Segments.from_host([T - 64, T], [1, 0], dev)
    G = K // 128
    sets = []
    for _ in range(n_sets):
        x = (torch.randn((T, K), generator=g, dtype=torch.float32) * 2).to(torch.bfloat16).to(dev)
        lay4 = torch.randint(0, 256, (B.mq_w4_layout_bytes(N, K),), dtype=torch.uint8, generator=g).to(dev)
        lay8 = torch.randint(0, 256, (B.mq_w8_layout_bytes(N, K),), dtype=torch.uint8, generator=g).to(dev)
        s_w = (torch.rand(N, generator=g) * 0.01 + 0.001).to(dev)
        s_wg = (torch.rand((G, N), generator=g) * 0.01 + 0.001).to(dev)
        y = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
        sets.append({"x": x, "lay4": lay4, "lay8": lay8, "s_w": s_w, "s_wg": s_wg, "y": y,
                     "ws": B.new_workspace(T, K, N, rot), "ws_g": B.new_workspace(T, K, N, rot, group_size=128),
                     "ws_8": B.new_workspace(T, K, N, rot, B.MQ_FLAG_W8), "ws_a4": B.new_workspace(T, K, N, rot, B.MQ_FLAG_A4)})
    fns = {
        "w4a8_per_channel_us": lambda s_: B.mq_w4a8_msq_linear(s_["x"], seg, 0.5, 0.05, s_["lay4"], s_["s_w"], s_["y"], s_["ws"], N, rot_block=rot),
        "w4a8_g128_us": lambda s_: B.mq_w4a8_msq_linear(s_["x"], seg, 0.5, 0.05, s_["lay4"], s_["s_wg"], s_["y"], s_["ws_g"], N, rot_block=rot, group_size=128),
        "w8a8_us": lambda s_: B.mq_w4a8_msq_linear(s_["x"], seg, 0.5, 0.05, s_["lay8"], s_["s_w"], s_["y"], s_["ws_8"], N, rot_block=rot, extra_flags=B.MQ_FLAG_W8),
        "w4a4_us": lambda s_: B.mq_w4a8_msq_linear(s_["x"], seg, 0.5, 0.05, s_["lay4"], s_["s_w"], s_["y"], s_["ws_a4"], N, rot_block=rot, extra_flags=B.MQ_FLAG_A4),
    }
    out = {}
    for name, fn in fns.items():
        for s_ in sets:
            fn(s_)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for s_ in sets:
                fn(s_)
        graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        out[name] = e0.elapsed_time(e1) * 1e3 / (reps * n_sets)
        del graph
    ok = all(B.mq_last_device_status(s_[k])[0] == 0 for s_ in sets for k in ("ws", "ws_g", "ws_8", "ws_a4"))
    ops = 2.0 * T * K * N
    out.update({"workload": "config2 down_proj T=%d K=%d N=%d rot=%d: quantizer + GEMM" % (T, K, N, rot),
                "tops": {k[:-3]: ops / (v * 1e-6) / 1e12 for k, v in out.items() if k.endswith("_us")},
                "status_ok": ok})
    return out


# ------------------------------------------------------------------------------------------ decode sweep
def decode_sweep(torch, B, dev, peaks, n_sets=6, reps=20):
    """Config-5-shaped decode steps: the linears of a 4096 / 13696 SwiGLU MLP (gate, up: 4096 -> 13696;
    down: 13696 -> 4096 behind the 128-block rotation) at T = 1, 2, 4, 8, 32, 128 text tokens.  Each step
    runs rotation + quantizer + W4A8 product per linear (one fused GEMV kernel up to T = 4); n_sets independent copies of the int4
    weights (84 MB each, more than four L2 sizes in all) are cycled so that the weights come from
    HBM.  Two arrangements are timed: the three linears as three calls, and gate and up stored as
    one [27392, 4096] weight (they share their input), i.e. two calls.  Reported per T:
    microseconds per MLP pass and packed-weight bytes per second."""
    hidden, mlp = 4096, 13696
    arrangements = {"three_calls": [(hidden, mlp, 0), (hidden, mlp, 0), (mlp, hidden, 128)],
                    "gate_up_fused": [(hidden, 2 * mlp, 0), (mlp, hidden, 128)]}
    g = torch.Generator(device="cpu").manual_seed(4)
    w_bytes = 3 * hidden * mlp // 2
    out = {}
    seg = B.Segments.from_host([], [], dev)  # no visual rows: every token uses the text scale
    for name, shapes in arrangements.items():
        weights = []
        for _ in range(n_sets):
            per_set = []
            for K, N, _ in shapes:
                lay = torch.randint(0, 256, (B.mq_w4_layout_bytes(N, K),), dtype=torch.uint8, generator=g).to(dev)
                per_set.append((lay, (torch.rand(N, generator=g) * 0.01 + 0.001).to(dev)))
            weights.append(per_set)
        res = {}
        for T in (1, 2, 4, 8, 32, 128):
            xs = [(torch.randn((T, K), generator=g) * 2).to(torch.bfloat16).to(dev) for K, _, _ in shapes]
            ys = [torch.empty((T, N), dtype=torch.bfloat16, device=dev) for _, N, _ in shapes]
            wss = [B.new_workspace(T, K, N, rot) for K, N, rot in shapes]

            def mlp_pass(i):
                for j, (K, N, rot) in enumerate(shapes):
                    lay, s_w = weights[i % n_sets][j]
                    B.mq_w4a8_msq_linear(xs[j], seg, 1.0, 0.05, lay, s_w, ys[j], wss[j], N, rot_block=rot)

            for i in range(n_sets):
                mlp_pass(i)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                for i in range(n_sets):
                    mlp_pass(i)
            graph.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            sec = e0.elapsed_time(e1) * 1e-3 / (reps * n_sets)
            del graph
            # every linear of the arrangement alone (the same call, rotating weight sets)
            per_linear = []
            for j, (K, N, rot) in enumerate(shapes):
                def one(i, j=j, K=K, N=N, rot=rot):
                    lay, s_w = weights[i % n_sets][j]
                    B.mq_w4a8_msq_linear(xs[j], seg, 1.0, 0.05, lay, s_w, ys[j], wss[j], N, rot_block=rot)
                g1 = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g1):
                    for i in range(n_sets):
                        one(i)
                g1.replay()
                torch.cuda.synchronize()
                e0.record()
                for _ in range(reps):
                    g1.replay()
                e1.record()
                torch.cuda.synchronize()
                us = e0.elapsed_time(e1) * 1e3 / (reps * n_sets)
                del g1
                per_linear.append({"K": K, "N": N, "us": us, "weight_gbs": N * K / 2 / us / 1e3})
            status = [B.mq_last_device_status(w)[0] for w in wss]
            gbs = w_bytes / sec / 1e9
            res["T%d" % T] = {"us_per_mlp": sec * 1e6, "weight_gbs": gbs, "frac_of_measured_hbm": gbs / peaks["hbm_gbs"],
                              "frac_of_nominal_8tbs": gbs / 8000.0, "per_linear": per_linear,
                              "kernel": ("w4a8_gemv_kernel (rotation + quantizer + dp4a product in one launch)" if T <= 3 else
                                         "fwht_quant_kernel + w4a8_gemm_kernel (+ splitk_finalize_kernel when K is split)"),
                              "tokens_per_s": T / sec, "status_ok": all(v == 0 for v in status)}
        out[name] = res
        del weights
        torch.cuda.empty_cache()
    out["roofline"] = {"bound": "hbm", "bytes": "packed int4 weights of the three linears: %d B per MLP pass" % w_bytes,
                       "peak_measured_gbs": peaks["hbm_gbs"], "peak_nominal_gbs": 8000.0,
                       "timing": "CUDA-graph replays of %d MLP passes over rotating weight sets, CUDA events" % n_sets}
    out["workload"] = ("config5: 4096/13696 MLP (gate, up, down with 128-block rotation), %d weight sets of %.0f MB "
                       "cycled" % (n_sets, w_bytes / 1e6))
    return out


# ------------------------------------------------------------------------------------------ RMS linear
def rms_linear_timing(torch, B, dev, T, K, N, rot, n_sets=4, reps=10):
    """Rotation magnitude suppression (Sec. 3.2) on the config-2 down-projection: the linear with
    the split product (one launch, second accumulator) against the plain linear of the same
    shape, both as rotation + quantizer + GEMM, CUDA-graph replays over n_sets rotating copies of
    activations and weights (larger than L2 in total).  Random valid weight bytes: timing only,
    parity is covered by the tests."""
    g = torch.Generator(device="cpu").manual_seed(12)
    seg = B.Segments.from_host([T - 64, T], [1, 0], dev)
    side_k = B.mq_rms_side_ld(K, rot)
    sets = []
    for _ in range(n_sets):
        x = (torch.randn((T, K), generator=g, dtype=torch.float32) * 2).to(torch.bfloat16).to(dev)
        lay = torch.randint(0, 256, (B.mq_w4_layout_bytes(N, K),), dtype=torch.uint8, generator=g).to(dev)
        slay = torch.randint(0, 256, (B.mq_w4_layout_bytes(N, side_k),), dtype=torch.uint8, generator=g).to(dev)
        s_w = (torch.rand(N, generator=g) * 0.01 + 0.001).to(dev)
        s_ws = (torch.rand(N, generator=g) * 0.05 + 0.001).to(dev)
        y = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
        sets.append((x, lay, slay, s_w, s_ws, y, B.new_workspace(T, K, N, rot), B.new_rms_workspace(T, K, N, rot)))

    def plain(i):
        x, lay, slay, s_w, s_ws, y, ws, wsr = sets[i % n_sets]
        B.mq_w4a8_msq_linear(x, seg, 0.5, 0.05, lay, s_w, y, ws, N, rot_block=rot)

    def rms(i):
        x, lay, slay, s_w, s_ws, y, ws, wsr = sets[i % n_sets]
        B.mq_w4a8_msq_linear_rms(x, seg, 0.5, 0.05, lay, s_w, slay, s_ws, y, N, rot, wsr)

    out = {}
    for name, fn in (("plain_us", plain), ("rms_us", rms)):
        for i in range(n_sets):
            fn(i)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(n_sets):
                fn(i)
        graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        out[name] = e0.elapsed_time(e1) * 1e3 / (reps * n_sets)
        del graph
    ok = all(B.mq_last_device_status(s_[6])[0] == 0 and B.mq_last_device_status(s_[7])[0] == 0 for s_ in sets)
    out.update({"workload": "config2 down_proj T=%d K=%d N=%d rot=%d: quantizer + GEMM" % (T, K, N, rot),
                "overhead_frac": out["rms_us"] / out["plain_us"] - 1.0,
                "split_k_codes": side_k, "split_macs_frac": (K // rot) / K, "status_ok": ok})
    return out


# ------------------------------------------------------------------------------------------ static vs dynamic A8
def dynamic_linear_timing(torch, B, dev, T, K, N, rot, n_sets=4, reps=10):
    """The comparison the paper's latency table makes (Sec. 4.3): the same linear with per-token
    dynamic activation scales (row abs-max at run time) against MSQ's static per-modality scales.
    Both as rotation + quantizer + GEMM on the config-2 shape, CUDA-graph replays over n_sets
    rotating copies (larger than L2 in total); also the two quantizer kernels alone."""
    g = torch.Generator(device="cpu").manual_seed(13)
    seg = B.Segments.from_host([T - 64, T], [1, 0], dev)
    sets = []
    for _ in range(n_sets):
        x = (torch.randn((T, K), generator=g, dtype=torch.float32) * 2).to(torch.bfloat16).to(dev)
        lay = torch.randint(0, 256, (B.mq_w4_layout_bytes(N, K),), dtype=torch.uint8, generator=g).to(dev)
        s_w = (torch.rand(N, generator=g) * 0.01 + 0.001).to(dev)
        y = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
        q = torch.empty((T, K), dtype=torch.int8, device=dev)
        sr = torch.empty(T, dtype=torch.float32, device=dev)
        sets.append((x, lay, s_w, y, q, sr, B.new_workspace(T, K, N, rot), B.new_dynamic_workspace(T, K, N, rot)))

    fns = {
        "static_linear_us": lambda s_: B.mq_w4a8_msq_linear(s_[0], seg, 0.5, 0.05, s_[1], s_[2], s_[3], s_[6], N, rot_block=rot),
        "dynamic_linear_us": lambda s_: B.mq_w4a8_dynamic_linear(s_[0], s_[1], s_[2], s_[3], s_[7], N, rot_block=rot),
        "static_quant_us": lambda s_: B.mq_fwht_quant_i8(s_[0], seg, 0.5, 0.05, rot, s_[4], None),
        "dynamic_quant_us": lambda s_: B.mq_dynamic_quant_i8(s_[0], rot, s_[4], s_[5]),
    }
    out = {}
    for name, fn in fns.items():
        for s_ in sets:
            fn(s_)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for s_ in sets:
                fn(s_)
        graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        out[name] = e0.elapsed_time(e1) * 1e3 / (reps * n_sets)
        del graph
    ok = all(B.mq_last_device_status(s_[6])[0] == 0 and B.mq_last_device_status(s_[7])[0] == 0 for s_ in sets)
    out.update({"workload": "config2 down_proj T=%d K=%d N=%d rot=%d" % (T, K, N, rot),
                "static_speedup_linear": out["dynamic_linear_us"] / out["static_linear_us"],
                "static_speedup_quantizer": out["dynamic_quant_us"] / out["static_quant_us"], "status_ok": ok})
    return out


# ------------------------------------------------------------------------------------------ layer mode
def layer_mode_timing(torch, dev, name, shape, seqs, reps=5):
    """Configs 3 and 4 as a whole decoder block (layer mode): AIFS, mask / position remap, the seven W4A8
    MSQ linears, the glue kernels (RMSNorm, rotary embedding, SwiGLU, residuals) and attention under the
    unified mask (mq_aifs_attention), all through the C ABI.  Random valid weight bytes, fixed scales: timing
    only (parity of the block is covered by the tests).  Reports tokens per second for the whole block, and
    for context the same block with attention handed to torch's fused causal kernel on un-permuted rows."""
    from paper_2502_00425_b200 import layer as LY
    blk = LY.random_block(shape, 21, dev)
    blk.fuse_groups = True  # q/k/v and gate/up as one stacked weight each: one launch per group (same results)
    for lw in blk.w.values():
        lw.s_vis, lw.s_txt = 0.5, 0.05
    g = torch.Generator(device="cpu").manual_seed(22)
    embs = [(torch.randn((len(s_), shape.hidden), generator=g) * 2).to(torch.bfloat16).to(dev) for s_ in seqs]
    vis = [torch.from_numpy(s_).to(dev) for s_ in seqs]
    tokens = sum(len(s_) for s_ in seqs)

    def timed():
        blk.forward_batch(embs, vis)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launch = "CUDA graph"
        try:  # the block has dozens of small launches: replay it from a graph so that the GPU, not the host, is timed
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                blk.forward_batch(embs, vis)
            graph.replay()
            torch.cuda.synchronize()
            run = graph.replay
        except Exception:
            torch.cuda.synchronize()
            launch = "eager"
            run = lambda: blk.forward_batch(embs, vis)
        e0.record()
        for _ in range(reps):
            run()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e-3 / reps, launch

    blk.cuda_attention = shape.head_dim == 128
    sec, launch = timed()
    own = blk.cuda_attention
    blk.cuda_attention, blk.causal_glue = False, True  # (plain causal mask in the original order: same result, Eq. 5)
    sec_torch, _ = timed()
    return {"workload": name, "tokens": tokens, "us_per_block": sec * 1e6, "tokens_per_s": tokens / sec,
            "attention": "mq_aifs_attention (unified mask, AIFS order)" if own else "torch (head_dim != 128)",
            "glue": "library kernels: RMSNorm, RoPE, SwiGLU, residuals", "launch": launch,
            "with_torch_causal_attention": {"us_per_block": sec_torch * 1e6, "tokens_per_s": tokens / sec_torch},
            "status_ok": blk.device_status_ok()}


def attention_timing(torch, B, dev, peaks, reps=10):
    """mq_aifs_attention alone on the sequences of configs 3 and 4 (one sequence per call) and on a long text-only
    sequence: microseconds and TFLOP/s over the multiply-adds the mask allows (4 * D * allowed pairs * heads), and
    that rate as a fraction of the measured dense bf16 rate (the kernel's products are bf16 tensor-core MMAs)."""
    from paper_2502_00425_b200 import synth as SY
    out = {}
    cases = [("config3 sequence: [img 1024][txt 96] x 3, 28 / 4 heads", SY.interleaved_modality([(1, 1024), (0, 96)] * 3), 28, 4),
             ("config4 sequence: [txt 32][4 x 576 visual][txt 96], 32 / 8 heads", SY.interleaved_modality([(0, 32), (1, 2304), (0, 96)]), 32, 8),
             ("text only, 8192 tokens, 32 / 8 heads", SY.interleaved_modality([(0, 8192)]), 32, 8)]
    g = torch.Generator(device="cpu").manual_seed(31)
    for name, is_visual, hq, hkv in cases:
        L, D = int(is_visual.shape[0]), 128
        q = torch.randn((L, hq * D), generator=g).to(torch.bfloat16).to(dev)
        k = torch.randn((L, hkv * D), generator=g).to(torch.bfloat16).to(dev)
        v = torch.randn((L, hkv * D), generator=g).to(torch.bfloat16).to(dev)
        o = torch.empty_like(q)
        ws = torch.empty(B.mq_aifs_attention_workspace_bytes(L, hkv), dtype=torch.uint8, device=dev)
        status = torch.zeros(2, dtype=torch.int32, device=dev)
        # the permutation comes from the library's own AIFS reorder (of a dummy embedding)
        perm = torch.empty(L, dtype=torch.int32, device=dev)
        dummy = torch.zeros((L, 64), dtype=torch.bfloat16, device=dev)
        B.mq_aifs_reorder(dummy, torch.empty_like(dummy), torch.from_numpy(is_visual).to(dev), None, perm,
                          torch.empty(L, dtype=torch.int32, device=dev), torch.zeros(1, dtype=torch.int32, device=dev), direction=0)
        run = lambda: B.mq_aifs_attention(q, k, v, perm, None, hq, hkv, o, ws, status)
        for _ in range(3):
            run()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            run()
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / reps
        flops = 4.0 * D * hq * (L * (L + 1) / 2)
        out[name] = {"L": L, "us": us, "tflops_allowed_pairs": flops / us / 1e6,
                     "frac_of_measured_bf16_burst": flops / us / 1e6 / peaks["bf16_burst"], "bound": "tensor (bf16)",
                     "status_ok": status.tolist() == [0, 0]}
    return out


# ------------------------------------------------------------------------------------------ layer linear suites
def linear_suite(torch, B, dev, name, T, n_vis_per_seq, n_txt_per_seq, batch, shape, reps=5):
    """The seven W4A8 MSQ linears of one decoder block (configs 3 and 4, linear-suite mode): every
    linear gets its own synthetic activations in AIFS order and runs rotation (down_proj only) +
    quantizer + GEMM through mq_w4a8_msq_linear.  Weight layouts and scales are random valid bytes
    (timing only; parity of these shapes is covered by the tests).  Reports microseconds per
    linear (the linear repeated back to back) and TOPS over the seven in sequence, both as
    CUDA-graph replays."""
    g = torch.Generator(device="cpu").manual_seed(11)
    seg_end, seg_mod, e = [], [], 0
    for _ in range(batch):
        e += n_vis_per_seq
        seg_end.append(e)
        seg_mod.append(1)
        e += n_txt_per_seq
        seg_end.append(e)
        seg_mod.append(0)
    assert e == T
    seg = B.Segments.from_host(seg_end, seg_mod, dev)
    items, total_ops = [], 0.0
    for lname, K, N, rot in shape.linears():
        x = (torch.randn((T, K), generator=g, dtype=torch.float32) * 2).to(torch.bfloat16).to(dev)
        lay = torch.randint(0, 256, (B.mq_w4_layout_bytes(N, K),), dtype=torch.uint8, generator=g).to(dev)
        s_w = (torch.rand(N, generator=g) * 0.01 + 0.001).to(dev)
        y = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
        ws = B.new_workspace(T, K, N, rot)
        items.append((lname, K, N, rot, x, lay, s_w, y, ws))
        total_ops += 2.0 * T * K * N

    def run(it):
        lname, K, N, rot, x, lay, s_w, y, ws = it
        B.mq_w4a8_msq_linear(x, seg, 0.5, 0.05, lay, s_w, y, ws, N, rot_block=rot)

    def timed_graph(body, reps_in_graph):
        """Microseconds per execution of body(), replayed from a CUDA graph (launch cost off the clock)."""
        body()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for _ in range(reps_in_graph):
                body()
        graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(3):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        del graph
        return e0.elapsed_time(e1) * 1e3 / (3 * reps_in_graph)

    per = {it[0]: timed_graph(lambda it=it: run(it), reps) for it in items}
    sec = timed_graph(lambda: [run(it) for it in items], reps) * 1e-6
    ok = all(B.mq_last_device_status(it[8])[0] == 0 for it in items)
    return {"workload": name, "T": T, "us_per_linear": per, "us_all_seven": sec * 1e6, "tops": total_ops / sec / 1e12,
            "tokens_per_s": T / sec, "status_ok": ok}


# ------------------------------------------------------------------------------------------ our arm
class BufferSet:
    """One independent copy of every device buffer a step touches."""

    def __init__(self, B, torch, dev, case, is_vis, emb_bits, w_layout_src, s_w):
        T, K, N = case.T, case.K, case.N
        L = T
        self.x = torch.from_numpy(case.x_bits.astype(np.int16)).to(dev).view(torch.bfloat16)
        self.layout = w_layout_src.clone()
        self.s_w = s_w
        self.ws = B.new_workspace(T, K, N, ROT)
        self.y = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
        self.qx = torch.empty((T, K), dtype=torch.int8, device=dev)
        self.ws_gemm = B.new_workspace(T, K, N, 0, B.MQ_FLAG_X_IS_INT8)
        self.emb = torch.from_numpy(emb_bits.astype(np.int16)).to(dev).view(torch.bfloat16)
        self.emb_u = torch.empty_like(self.emb)
        self.is_vis = torch.from_numpy(is_vis).to(dev)
        self.perm = torch.empty(L, dtype=torch.int32, device=dev)
        self.inv = torch.empty(L, dtype=torch.int32, device=dev)
        self.n_first = torch.empty(1, dtype=torch.int32, device=dev)
        self.pos = torch.empty(L, dtype=torch.int32, device=dev)
        self.seg_end = torch.empty(2, dtype=torch.int32, device=dev)
        self.seg_mod = torch.empty(2, dtype=torch.uint8, device=dev)
        self.seg = B.Segments(self.seg_end, self.seg_mod)

    def bytes(self):
        return sum(t.numel() * t.element_size() for t in (self.x, self.layout, self.ws, self.y, self.emb, self.emb_u))


LAUNCHES_PER_STEP = 4  # fused AIFS index + gather, remap, rotation + quantizer, GEMM


def run_ours(args, info):
    import torch
    from paper_2502_00425_b200 import binding as B
    from paper_2502_00425_b200 import dist as D
    from paper_2502_00425_b200 import synth

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the product path has no CPU fallback")
    B.load(build_if_missing=True)
    torch.cuda.set_device(info.local_rank)
    dev = torch.device("cuda", info.local_rank)
    peaks = read_peaks()
    if args.decode_only:
        if info.is_main:
            print(json.dumps({"decode": decode_sweep(torch, B, dev, peaks, n_sets=4, reps=2)}), flush=True)
        return
    D.init(info)

    case = synth.config2(seed=D.batch_seed(1, info.rank))
    is_vis = synth.interleaved_modality(SPANS)
    assert is_vis.sum() == T_VIS and len(is_vis) == case.T
    emb_bits = synth.to_bf16_bits(synth.embedding_rows(7 + info.rank, case.T, HIDDEN, is_vis))

    # ---- offline, untimed: calibration and weight packing (on the GPU, through the C ABI)
    xc = torch.from_numpy(synth.to_bf16_bits(case.x_calib).astype(np.int16)).to(dev).view(torch.bfloat16)
    state = torch.zeros(2, dtype=torch.int32, device=dev)
    sv, st = torch.zeros(1, device=dev), torch.zeros(1, device=dev)
    B.mq_calibrate_static_scales(xc, B.Segments.from_host(case.seg_calib.seg_end, case.seg_calib.seg_mod, dev), ROT,
                                 state, sv, st)
    s_vis, s_txt = float(sv.item()), float(st.item())
    w = torch.from_numpy(case.w).to(dev)
    s_w = torch.empty(case.N, dtype=torch.float32, device=dev)
    layout = torch.empty(B.mq_w4_layout_bytes(case.N, case.K), dtype=torch.uint8, device=dev)
    B.mq_pack_w4(w, None, s_w, layout)
    del w, xc

    n_sets = args.buffer_sets
    sets = [BufferSet(B, torch, dev, case, is_vis, emb_bits, layout, s_w) for _ in range(n_sets)]
    footprint = sum(s.bytes() for s in sets)

    names = ["aifs_reorder", "mask_remap", "fwht_quant", "gemm"]

    def k_aifs(s):
        B.mq_aifs_reorder(s.emb, s.emb_u, s.is_vis, None, s.perm, s.inv, s.n_first, 0)

    def k_remap(s):
        B.mq_attn_mask_remap(s.perm, None, None, s.n_first, s.pos, s.seg_end, s.seg_mod)

    def k_quant(s):
        B.mq_fwht_quant_i8(s.x, s.seg, s_vis, s_txt, ROT, s.qx, None)

    def k_gemm(s):
        B.mq_w4a8_msq_linear(s.qx, s.seg, s_vis, s_txt, s.layout, s.s_w, s.y, s.ws_gemm, case.N)

    kernels = [k_aifs, k_remap, k_quant, k_gemm]

    branch = torch.cuda.Stream()

    def k_index(s):
        B.mq_aifs_reorder(None, None, s.is_vis, None, s.perm, s.inv, s.n_first, 0, L=case.T)

    def k_gather(s):  # X_out[inv[i]] = X[i], i.e. X_out[j] = X[perm[j]]: the gather, from the finished index arrays
        B.mq_aifs_reorder(s.emb, s.emb_u, None, None, s.inv, None, None, 1)

    def step(s, events=None):
        """One pass of the hot path.  The linear is issued as its two kernels (the quantizer into
        a caller-owned code buffer, then the GEMM on the codes), which is exactly what
        mq_w4a8_msq_linear does with its workspace, so that events can sit between them.
        Dependencies: the quantizer reads the segment table that the remap writes, and the remap
        reads the permutation; the row gather of the embeddings needs the permutation only.  The
        timed step therefore issues index -> remap -> quantizer -> GEMM in line and the row gather
        as a second branch behind the index kernel (fork and join with events; in a captured graph
        a parallel branch).  With timing events between the kernels (or --serial-step) the fused
        index + gather kernel runs in line instead: four launches."""
        if events is not None or args.serial_step:
            for i, k in enumerate(kernels):
                if events is not None:
                    events[i].record()
                k(s)
            if events is not None:
                events[len(kernels)].record()
            return
        main = torch.cuda.current_stream()
        k_index(s)
        branch.wait_stream(main)
        with torch.cuda.stream(branch):
            k_gather(s)
        k_remap(s)
        k_quant(s)
        k_gemm(s)
        main.wait_stream(branch)

    # ---- CUDA graphs: one per buffer set, so that the host only replays.  A second family of
    # graphs of the same step carries timing events recorded as graph nodes ("external" events)
    # around every kernel; it is replayed after the timed region for the per-kernel durations
    # (event nodes between kernels would keep them from overlapping their launch with the
    # predecessor's tail, so the timed graphs have none).
    graphs, ev_graphs, set_events = None, None, None
    launch_mode = "eager"
    if not args.no_graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                for s in sets:
                    step(s)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            try:
                set_events = [[torch.cuda.Event(enable_timing=True, external=True) for _ in range(len(kernels) + 1)]
                              for _ in sets]
            except TypeError:
                set_events = None
            graphs = []
            for i, s in enumerate(sets):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    step(s)
                graphs.append(g)
            if set_events is not None:
                ev_graphs = []
                for i, s in enumerate(sets):
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g):
                        step(s, set_events[i])
                    ev_graphs.append(g)
            launch_mode = "cuda_graph"
        except Exception as e:  # capture unavailable: time eager launches instead
            graphs, ev_graphs, set_events = None, None, None
            launch_mode = "eager (graph capture failed: %s)" % type(e).__name__
            torch.cuda.synchronize()

    # Steps are independent batches on their own buffer sets.  With --steps-in-flight 2 (the default) they are
    # issued alternately on two streams, so the small kernels at the head of one step (index, remap, quantizer)
    # can run while the GEMM of the step before occupies the tensor cores; every kernel of a step still waits
    # for the kernels it depends on (stream order within the step).  A buffer set comes round again on the
    # stream it was used on before (n_sets is even), so its reuse is ordered.
    in_flight = max(1, min(args.steps_in_flight, 2))
    if n_sets % 2:
        in_flight = 1
    lanes = [torch.cuda.Stream() for _ in range(in_flight)] if in_flight > 1 else None

    def run_step(i):
        if lanes is not None:
            with torch.cuda.stream(lanes[i % in_flight]):
                if graphs is not None:
                    graphs[i % n_sets].replay()
                else:
                    step(sets[i % n_sets])
            return
        if graphs is not None:
            graphs[i % n_sets].replay()
        else:
            step(sets[i % n_sets])

    def fork_lanes():
        if lanes is not None:
            for l_ in lanes:
                l_.wait_stream(torch.cuda.current_stream())

    def join_lanes():
        if lanes is not None:
            for l_ in lanes:
                torch.cuda.current_stream().wait_stream(l_)

    fork_lanes()
    for i in range(max(args.warmup, 3)):
        run_step(i)
    join_lanes()
    torch.cuda.synchronize()

    # ---- timed region: exactly K steps, device-resident inputs
    sampler = ClockSampler(info.local_rank)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    D.barrier(dev)
    torch.cuda.synchronize()
    sampler.start()
    e0.record()
    fork_lanes()
    for i in range(args.steps):
        run_step(i)
    join_lanes()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    D.barrier(dev)
    secs = e0.elapsed_time(e1) * 1e-3
    value_ops, t_max = D.aggregate_throughput(ops_per_step() * args.steps, secs, dev)

    # ---- per-kernel durations.  (1) Inside the step: the same K steps replayed from the graphs
    # that carry event nodes; samples are read every n_sets steps (one per buffer set).
    in_step = None
    if ev_graphs is not None:
        try:
            acc = {n: [] for n in names}
            for i in range(min(args.steps, 200)):
                ev_graphs[i % n_sets].replay()
                if i % n_sets == n_sets - 1:
                    torch.cuda.synchronize()
                    for ev in set_events:
                        for j, n in enumerate(names):
                            acc[n].append(ev[j].elapsed_time(ev[j + 1]) * 1e-3)
            torch.cuda.synchronize()
            if all(acc[n] for n in names):
                in_step = {n: float(np.mean(acc[n])) for n in names}
        except Exception:
            in_step = None
    # (2) Each kernel alone, launched back to back over the rotating buffer sets (one graph of
    # n_sets launches, replayed), timed with events on the launching stream.
    kern = {}
    reps = max(1, min(args.steps, 200) // n_sets)
    for n, k in zip(names, kernels):
        for s in sets:
            k(s)
        torch.cuda.synchronize()
        g = None
        if graphs is not None:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for s in sets:
                    k(s)
            g.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            if g is not None:
                g.replay()
            else:
                for s in sets:
                    k(s)
        e1.record()
        torch.cuda.synchronize()
        kern[n] = e0.elapsed_time(e1) * 1e-3 / (reps * n_sets)
    timing_kind = "CUDA event nodes around the kernel inside graphs of the whole step, replayed after the timed region"
    if in_step is None:
        in_step = dict(kern)
        timing_kind = "kernel alone, launched back to back over the rotating buffer sets"
    status = B.mq_last_device_status(sets[0].ws_gemm)

    # ---- end to end through the C ABI with host buffers
    x_host = torch.from_numpy(case.x_bits.astype(np.int16)).view(torch.bfloat16).pin_memory()
    y_host = torch.empty((case.T, case.N), dtype=torch.bfloat16).pin_memory()
    e2e_steps = max(3, min(args.steps, 50))

    # Three streams: copy-in, compute, copy-out.  Every step still moves its own input from pinned
    # host memory and its own result back; the copies of neighbouring steps overlap with compute,
    # ordered per buffer set with events (a set is refilled only after its result has left).
    st_in, st_comp, st_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(n_sets)]
    ev_comp = [torch.cuda.Event() for _ in range(n_sets)]
    ev_out = [torch.cuda.Event() for _ in range(n_sets)]

    def e2e_step(i):
        j = i % n_sets
        s = sets[j]
        with torch.cuda.stream(st_in):
            st_in.wait_event(ev_out[j])      # the previous result of this set has been read back
            s.x.copy_(x_host, non_blocking=True)
            ev_in[j].record(st_in)
        with torch.cuda.stream(st_comp):
            st_comp.wait_event(ev_in[j])
            k_aifs(s)
            k_remap(s)
            B.mq_w4a8_msq_linear(s.x, s.seg, s_vis, s_txt, s.layout, s.s_w, s.y, s.ws, case.N, rot_block=ROT)
            ev_comp[j].record(st_comp)
        with torch.cuda.stream(st_out):
            st_out.wait_event(ev_comp[j])
            y_host.copy_(s.y, non_blocking=True)
            ev_out[j].record(st_out)

    def e2e_join():
        cur = torch.cuda.current_stream()
        cur.wait_stream(st_in)
        cur.wait_stream(st_comp)
        cur.wait_stream(st_out)

    torch.cuda.synchronize()
    for i in range(3):
        e2e_step(i)
    e2e_join()
    torch.cuda.synchronize()
    D.barrier(dev)
    for st_ in (st_in, st_comp, st_out):
        st_.wait_stream(torch.cuda.current_stream())
    e0.record()
    for st_ in (st_in, st_comp, st_out):
        st_.wait_event(e0)
    for i in range(e2e_steps):
        e2e_step(i)
    e2e_join()
    e1.record()
    torch.cuda.synchronize()
    D.barrier(dev)
    e2e_ops, _ = D.aggregate_throughput(ops_per_step() * e2e_steps, e0.elapsed_time(e1) * 1e-3, dev)

    # ---- decode-shaped sweep (rank 0, N = 1 only): the HBM-bound regime of the same path
    decode, suites, rms_timing, dyn_timing, layers, var_timing, attn_timing = None, None, None, None, None, None, None
    n_sms = torch.cuda.get_device_properties(dev).multi_processor_count
    ubench = None
    if info.is_main:
        try:
            ubench = mma_issue_microbenchmark(torch, B, dev, n_sms)
        except Exception:
            ubench = None
    if info.is_main and info.world == 1 and not args.no_decode:
        del graphs, ev_graphs
        decode = decode_sweep(torch, B, dev, peaks)
        del sets
        torch.cuda.empty_cache()
        suites = [linear_suite(torch, B, dev, "config3: Qwen2-7B-shaped block, 3 x (1024 visual + 96 text) in AIFS order",
                               3360, 3072, 288, 1, synth.QWEN2_7B),
                  linear_suite(torch, B, dev, "config4: 8B-shaped block, 4 sequences x (2304 visual + 128 text)",
                               9728, 2304, 128, 4, synth.LLAMA_8B)]
        rms_timing = rms_linear_timing(torch, B, dev, case.T, case.K, case.N, ROT)
        dyn_timing = dynamic_linear_timing(torch, B, dev, case.T, case.K, case.N, ROT)
        torch.cuda.empty_cache()
        var_timing = variants_timing(torch, B, dev, case.T, case.K, case.N, ROT)
        torch.cuda.empty_cache()
        layers = [layer_mode_timing(torch, dev, "config3: Qwen2-7B-shaped block, one sequence of 3360 tokens",
                                    synth.QWEN2_7B, [synth.config3_sequence()]),
                  layer_mode_timing(torch, dev, "config4: 8B-shaped block, 4 sequences of 2432 tokens",
                                    synth.LLAMA_8B, [synth.config4_sequence()] * 4)]
        torch.cuda.empty_cache()
        attn_timing = attention_timing(torch, B, dev, peaks)

    # ---- CPU baseline: the oracle on this host (rank 0, N = 1 only)
    cpu = None
    if info.is_main and info.world == 1 and not args.no_cpu_baseline:
        from oracle import mq_oracle as O
        qw, sw_ref = O.quantize_weight_int4(case.w)
        o_v, o_t = O.calibrate_static_scales(case.x_calib, case.seg_calib.seg_end, case.seg_calib.seg_mod, ROT)
        rows = np.arange(case.T)
        times = time_oracle(case, qw, sw_ref, o_v, o_t, rows, 3)
        cpu = {"value": ops_per_step() / float(np.median(times)) / 1e12, "unit": UNIT, "cores": host_threads(),
               "kind": "oracle", "sample": "the full config-2 workload (1088 rows), median of 3 passes",
               "seconds_per_pass": float(np.median(times))}
        try:  # the same oracle confined to one thread, on a 64-row sample (the library matmul is its only threaded step)
            from threadpoolctl import threadpool_limits
            sample = oracle_sample_rows()[::4]
            with threadpool_limits(limits=1):
                t1 = time_oracle(case, qw, sw_ref, o_v, o_t, sample, 2)
            cpu["single_thread"] = {"value": ops_per_step(len(sample)) / float(np.min(t1)) / 1e12, "unit": UNIT, "cores": 1,
                                    "sample": "%d of 1088 rows, best of 2 passes" % len(sample)}
        except Exception:
            pass
        # the reading of x / s (multiply by the float32 reciprocal) against Eq. 2's literal division, on this batch
        r_rot = O.fwht_blocks(case.x, ROT, np.float32)
        s_rows = O.row_scales(case.T, case.seg.seg_end, case.seg.seg_mod, o_v, o_t)
        differ = int((O.quantize_act_int8(r_rot, s_rows) != O.quantize_act_int8_divide(r_rot, s_rows)).sum())
        cpu["codes_differing_reciprocal_vs_division"] = {"differ": differ, "codes": int(r_rot.size)}

    if info.is_main:
        gemm_tops = ops_per_step() / kern["gemm"] / 1e12
        linear_tops = ops_per_step() / (kern["gemm"] + kern["fwht_quant"]) / 1e12
        timed_s = t_max
        sustained = timed_s > 1.0
        peak = 2.0 * (peaks["bf16_sustained"] if sustained else peaks["bf16_burst"])
        quant_bytes = case.T * case.K * 3
        traffic, traffic_rec = gemm_traffic_record()
        # the tensor pipe's own rate on this machine: the issue-only microbenchmark at the widest tile, at
        # the SM clock sampled during the timed region and at the maximum clock
        sm_mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0
        sm_max = clocks.get("sm_max_mhz") or 1965.0
        ub = ubench["N256"]["ops_per_clk_sm"] if ubench else None
        ub_sampled = ub * n_sms * sm_mhz * 1e6 / 1e12 if ub else None
        ub_max = ub * n_sms * sm_max * 1e6 / 1e12 if ub else None
        denominators = {
            "measured_bf16_burst_x2": 2.0 * peaks["bf16_burst"], "measured_bf16_sustained_x2": 2.0 * peaks["bf16_sustained"],
            "nominal_dense_int8": 4500.0, "mma_microbenchmark_at_sampled_clock": ub_sampled,
            "mma_microbenchmark_at_max_clock": ub_max,
            "ncu_tensor_pipe_pct_of_elapsed": (traffic_rec or {}).get("sm__pipe_tensor_cycles_active_pct_of_elapsed")}
        fracs = lambda tops: {k: (tops / v if v else None) for k, v in denominators.items() if k != "ncu_tensor_pipe_pct_of_elapsed"}
        line = {
            "metric": METRIC, "value": value_ops / 1e12, "unit": UNIT, "n_gpus": info.world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": 1e3 * t_max / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8xint4->int32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "launch": launch_mode,
                       "l2": "inputs larger than L2: %d buffer sets, %.0f MB cycled" % (n_sets, footprint / 1e6),
                       "step": "aifs_reorder + mask_remap + fwht_quant_i8 + w4a8 gemm"
                               + ("" if args.serial_step else " (index -> remap -> quantizer -> GEMM in line, the row "
                                  "gather as a parallel branch behind the index kernel)"),
                       "steps_in_flight": in_flight,
                       "tokens_per_s": (T_VIS + T_TXT) * args.steps * info.world / t_max},
            "clocks": clocks,
            "e2e": {"value": e2e_ops / 1e12, "unit": UNIT, "h2d_bytes_per_step": case.T * case.K * 2,
                    "d2h_bytes_per_step": case.T * case.N * 2, "steps": e2e_steps,
                    "overlap": "copy-in, compute and copy-out of neighbouring steps on three streams"},
            "gpu_launches": (LAUNCHES_PER_STEP if args.serial_step else LAUNCHES_PER_STEP + 1) * args.steps,
            "roofline": {"bound": "tensor", "kernel": "w4a8_gemm_kernel", "achieved": gemm_tops, "peak": peak,
                         "unit": "TOP/s", "frac": gemm_tops / peak,
                         "peak_kind": "2 x measured bf16 %s (%s)" % ("sustained" if sustained else "burst",
                                                                      peaks["source"]),
                         "denominators_tops": denominators, "frac_by_denominator": fracs(gemm_tops),
                         "linear": {"what": "fwht_quant_kernel + w4a8_gemm_kernel (the prefill W4A8 MSQ linear)",
                                    "achieved": linear_tops, "frac_by_denominator": fracs(linear_tops)},
                         "step": {"what": "the whole timed step", "achieved": value_ops / 1e12 / info.world,
                                  "frac_by_denominator": fracs(value_ops / 1e12 / info.world)},
                         "mma_microbenchmark": ubench,
                         "traffic": traffic, "traffic_unit": "bytes per launch (ncu, profiles/)",
                         "traffic_record": traffic_rec,
                         "algorithmic_bytes": case.T * case.K + case.N * case.K // 2 + 4 * case.N
                         + 2 * case.T * case.N,
                         "avg_kernel_us": kern["gemm"] * 1e6,
                         "timing": "average over back-to-back launches of the kernel alone on the rotating "
                                   "(L2-cold) buffer sets, CUDA events on the launching stream",
                         "in_step_us": in_step["gemm"] * 1e6, "in_step_timing": timing_kind},
            "kernels_us": {n: kern[n] * 1e6 for n in names},
            "kernels_in_step_us": {n: in_step[n] * 1e6 for n in names},
            "fwht_quant_hbm": {"achieved_gbs": quant_bytes / kern["fwht_quant"] / 1e9,
                               "peak_gbs": peaks["hbm_gbs"],
                               "frac": quant_bytes / kern["fwht_quant"] / 1e9 / peaks["hbm_gbs"]},
            "decode": decode,
            "layer_linear_suites": suites,
            "rms_linear": rms_timing,
            "static_vs_dynamic_a8": dyn_timing,
            "variants": var_timing,
            "layer_mode": layers,
            "attention": attn_timing,
            "device_status": list(status),
            "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    D.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--buffer-sets", type=int, default=4)
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--steps-in-flight", type=int, default=2,
                    help="independent steps issued concurrently (1: one stream; 2: alternate streams)")
    ap.add_argument("--serial-step", action="store_true",
                    help="issue the four kernels of a step in one line instead of two parallel branches")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--decode-only", action="store_true",
                    help="run only the decode-shaped sweep and print it (used for profiler captures)")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 5 if args.impl == "reference" else 2000
    if args.impl == "reference":
        args.warmup = min(args.warmup, 3)
    from paper_2502_00425_b200 import dist as D
    info = D.rank_info_from_env()
    if args.impl == "reference":
        run_reference(args, info)
    else:
        run_ours(args, info)


if __name__ == "__main__":
    main()
