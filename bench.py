#!/usr/bin/env python
"""Benchmark of the E0M4 weight-only FP4 matmul on B200.

One "step" is one decode token's worth of matmuls: every matrix of every layer of the 14B-class
stack (40 layers x 4 matrices, M = 1, each with its own activations; 6.7 GB of packed weights, the
largest configuration) multiplied once.  The headline runs the step as one tl_e0m4_matmul_batch
call (the matrices of the synthetic stack are independent problems; one persistent kernel per 192
problems); `per_call` gives the same step as one tl_e0m4_matmul call per matrix.  Both are replayed
as CUDA graphs.  The packed weights are far larger than L2, so every step streams them from HBM.

Prints ONE JSON line (rank 0).  `value` is algorithmic GB/s over all GPUs:
(packed codes + scales + x + y bytes of a step) / step time.  Further keys: `roofline` (decode
kernel against the measured HBM copy bandwidth), `sustained` (the same step launched back to back
for more than a second, with the SM clock sampled inside the region and the rate binned by clock),
`e2e` (the same metric through the host-buffer entry point, copies timed), `sweeps` (the M sweeps of
the ChatGLM2-6B-shaped and the 14B-class stack: microseconds, GB/s, TFLOP/s and t_roof / t per
point, with the bound named), `prefill`, `quantize`/`dequant`, the objects of the widened rows,
`cpu_baseline` (the numpy oracle timed on this host's cores on a bounded sample) and, as the LAST
key, `summary`: the few figures that matter, short enough to survive a truncated log.

`--impl reference` times the CPU oracle instead (rank 0 only).  `--gpus N` without a torchrun
environment starts N ranks itself (one independent replica of the stack per GPU).
"""

from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# dram__bytes_read.sum + dram__bytes_write.sum per LAYER of one launch of the decode list kernel at
# M = 1, from the ncu captures summarised under profiles/ (gemv_decode_batch_*_m1.md).  The 14B-class
# figure was captured on 8 of the 40 layers (a capture has to stay small) and is scaled by the layer
# count: a launch's traffic is its weights, read once, so it grows in proportion.  Other workloads
# report null.
DECODE_TRAFFIC_BYTES_PER_LAYER_M1 = {"gemma2b": (1.05985e9 + 6.27e6) / 18, "llm14b": (1.343138e9 + 5.04e6) / 8}

METRIC = "e0m4_decode_gemv_hbm_gbps"
UNIT = "GB/s"
BYTES_PER_WEIGHT = 0.5 + 4.0 / 128.0  # nibble + (fp16 scale + fp16 bias) per 128 weights


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def step_bytes(matrices, layers, M):
    per_layer = sum(K * N * BYTES_PER_WEIGHT + 2 * M * K + 2 * M * N for _, K, N in matrices)
    return per_layer * layers


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

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

    def _once(self):
        nv = self.nv
        self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
        try:
            mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
        except Exception:
            mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
        names = {
            0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
            0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown",
        }
        for bit, name in names.items():
            if mask & bit:
                self.reasons.add(name)

    def _run(self):
        while not self._stop.is_set():
            try:
                self._once()
            except Exception:
                break
            self._stop.wait(0.01)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        """Call while the timed work is still in flight (before the closing synchronize): one more
        sample is taken here, so that even a very short region has one taken under load."""
        if self.nv is not None:
            try:
                self._once()
            except Exception:
                pass
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": []}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


# --------------------------------------------------------------------------- oracle arm
def oracle_sample(stack_name, M, seed=0, max_cols=2048):
    """A bounded sample of the workload for the CPU oracle: layer 0 of the stack with every
    matrix cut to at most `max_cols` output columns.  Returns (matrices, bytes, description)."""
    import numpy as np

    import oracle
    from paper_2403_20041_b200 import workloads

    spec = workloads.STACKS[stack_name]
    items, total = [], 0.0
    for name, K, N in spec["matrices"]:
        Ns = min(N, max_cols)
        w = workloads.weights(K, Ns, workloads.seed_for(stack_name, 0, name, seed))
        codes, d_h, b_h = oracle.quantize(w)
        x = workloads.activations(M, K, workloads.seed_for(stack_name, 0, name, "x", seed))
        items.append((x, codes, d_h, b_h))
        total += K * Ns * BYTES_PER_WEIGHT + 2 * M * K + 2 * M * Ns
    desc = (f"layer 0 of {stack_name}, each matrix cut to <= {max_cols} output columns, "
            f"M={M}: dequantize + fp64 matmul in numpy")
    return items, total, desc


def oracle_pass(items):
    import oracle

    for x, codes, d_h, b_h in items:
        oracle.matmul(x, oracle.dequantize(codes, d_h, b_h))


def time_oracle(stack_name, M, repeats, max_cols=2048):
    items, nbytes, desc = oracle_sample(stack_name, M, max_cols=max_cols)
    oracle_pass(items)  # warm-up
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        oracle_pass(items)
        times.append(time.perf_counter() - t0)
    return nbytes, times, desc


def host_threads():
    try:
        from threadpoolctl import threadpool_info

        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def workload_config(stack, layers, n_matrices, M, nbytes, world):
    """The `config` object both arms print: the workload the metric is quoted on."""
    return {
        "workload": f"{stack}-shaped decode stack: {layers} layers x {n_matrices} E0M4 matmuls, M={M}, group 128",
        "bytes_per_step": nbytes,
        "l2": "inputs larger than L2 (packed stack streamed per step)",
        "launch": "tl_e0m4_matmul_batch over the whole stack (one persistent kernel per 192 "
                  "independent problems), replayed as a CUDA graph",
        "parallelism": f"replicas x{world}",
    }


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy  # noqa: F401

    warm = max(0, min(args.warmup, 2))
    # the sample shrinks with the step count so that the whole run stays within minutes
    max_cols = 2048 if args.steps <= 20 else (512 if args.steps <= 100 else 128)
    nbytes, times, desc = time_oracle(args.stack, args.M, warm + args.steps, max_cols)
    times = times[warm:]
    total = sum(times)
    value = nbytes * len(times) / total / 1e9
    cores = host_threads()
    from paper_2403_20041_b200 import workloads

    spec = workloads.STACKS[args.stack]
    layers = args.layers or spec["layers"]
    config = workload_config(args.stack, layers, len(spec["matrices"]), args.M,
                             step_bytes(spec["matrices"], layers, args.M), args.gpus)
    config["sample"] = desc
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- native arm
def build_stack(binding, workloads, torch, dev, stack_name, layers, M, seed):
    """Quantize every matrix of the stack on the GPU.  Every problem gets its own activations
    (a view of one contiguous x buffer) and its own output (a view of one contiguous y buffer)."""
    spec = workloads.STACKS[stack_name]
    shapes = [(name, K, N) for _ in range(layers) for name, K, N in spec["matrices"]]
    x_all = torch.empty(sum(M * K for _, K, _ in shapes), dtype=torch.float16, device=dev)
    y_all = torch.empty(sum(M * N for _, _, N in shapes), dtype=torch.float16, device=dev)
    problems, xo, yo = [], 0, 0
    for idx, (name, K, N) in enumerate(shapes):
        layer = idx // len(spec["matrices"])
        w = workloads.weights_torch(K, N, workloads.seed_for(stack_name, layer, name, seed), dev)
        packed, scales = binding.tl_e0m4_quantize(w)
        del w
        x = x_all[xo:xo + M * K].view(M, K)
        x.copy_(workloads.activations_torch(M, K, workloads.seed_for(stack_name, layer, name, "x", seed), dev))
        y = y_all[yo:yo + M * N].view(M, N)
        xo += M * K
        yo += M * N
        problems.append({"name": name, "K": K, "N": N, "packed": packed, "scales": scales, "x": x, "y": y})
    torch.cuda.synchronize()
    return problems, x_all, y_all


def make_call_step(binding, torch, problems, M, ws):
    """One tl_e0m4_matmul call per matrix of the stack (arguments marshalled once)."""
    fn = binding.lib().tl_e0m4_matmul
    nbytes = ws.numel()
    calls = [(p["x"].data_ptr(), p["packed"].data_ptr(), p["scales"].data_ptr(), p["y"].data_ptr(),
              M, p["K"], p["N"], 128, ws.data_ptr(), nbytes) for p in problems]

    def step():
        s = torch.cuda.current_stream().cuda_stream
        for c in calls:
            st = fn(*c, s)
            if st != 0:
                raise RuntimeError(f"tl_e0m4_matmul failed: {binding.tl_status_string(st)}")

    return step


def make_batch_step(binding, torch, problems, M, ws):
    """One tl_e0m4_matmul_batch call for the whole stack (a persistent kernel per 192 problems)."""
    import ctypes

    arr = binding.make_problem_array([(p["x"], p["packed"], p["scales"], p["y"]) for p in problems])
    fn = binding.lib().tl_e0m4_matmul_batch
    ptr = ctypes.cast(arr, ctypes.c_void_p)

    def step():
        st = fn(ptr, len(arr), M, 128, ws.data_ptr(), ws.numel(), torch.cuda.current_stream().cuda_stream)
        if st != 0:
            raise RuntimeError(f"tl_e0m4_matmul_batch failed: {binding.tl_status_string(st)}")

    return step, arr


def capture(binding, torch, step):
    """Captures `step` into a CUDA graph; returns (graph, kernel launches per replay)."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    before = binding.tl_e0m4_launch_count()
    with torch.cuda.graph(graph, stream=side):
        step()
    return graph, binding.tl_e0m4_launch_count() - before


def time_events(torch, fn, iters):
    start = torch.cuda.Event(enable_timing=True)
    end = torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record()
    for _ in range(iters):
        fn()
    end.record()
    torch.cuda.synchronize()
    return start.elapsed_time(end) / iters  # ms per call


def time_events_clocked(torch, fn, iters, index):
    """time_events plus the SM clock read while the timed work is still in flight."""
    sampler = ClockSampler(index)
    start = torch.cuda.Event(enable_timing=True)
    end = torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    sampler.start()
    start.record()
    for _ in range(iters):
        fn()
    end.record()
    clocks = sampler.stop()
    torch.cuda.synchronize()
    return start.elapsed_time(end) / iters, clocks["sm_mhz"]


def bench_prefill(binding, workloads, torch, dev, peaks, Ms=(128, 512, 2048)):
    """Matrix-matrix path on one ChatGLM2-6B-shaped layer (activations with 1% outlier
    channels).  Returns TFLOP/s per M over the four matrices of the layer."""
    spec = workloads.STACKS["chatglm2_6b"]
    mats = []
    for name, K, N in spec["matrices"]:
        w = workloads.weights_torch(K, N, workloads.seed_for("prefill", name), dev)
        packed, scales = binding.tl_e0m4_quantize(w)
        del w
        mats.append((name, K, N, packed, scales))
    out = {}
    for M in Ms:
        xs = {K: workloads.activations_torch(M, K, workloads.seed_for("prefill", "x", K, M), dev, 0.01)
              for _, K, _, _, _ in mats}
        ys = {N: torch.empty((M, N), dtype=torch.float16, device=dev) for _, _, N, _, _ in mats}
        ws_bytes = max(binding.tl_e0m4_matmul_workspace(M, K, N) for _, K, N, _, _ in mats)
        ws = binding.tl_e0m4_workspace(ws_bytes, dev)

        def layer():
            for _, K, N, packed, scales in mats:
                binding.tl_e0m4_matmul(xs[K], packed, scales, N, y=ys[N], workspace=ws)

        for _ in range(3):
            layer()
        ms = time_events(torch, layer, 5 if M >= 1024 else 10)
        flops = sum(2.0 * M * K * N for _, K, N, _, _ in mats)
        tf = flops / (ms * 1e-3) / 1e12
        out[f"M{M}"] = {"tflops": tf, "ms_per_layer": ms,
                        "frac_of_measured_bf16_burst": tf / peaks["bf16_tflops"],
                        "frac_of_nominal_2250": tf / 2250.0}
        if M == max(Ms):
            # context: the library GEMM on the same shapes with weights already dequantized to fp16
            dense = [(xs[K], binding.tl_e0m4_dequant(packed, scales, K, N)) for _, K, N, packed, scales in mats]

            def dense_layer():
                for a, b in dense:
                    torch.matmul(a, b)

            for _ in range(3):
                dense_layer()
            out[f"M{M}"]["torch_matmul_fp16_dense_tflops"] = flops / (time_events(torch, dense_layer, 5) * 1e-3) / 1e12
            del dense
    best = max(out.values(), key=lambda r: r["tflops"])
    roofline = {"bound": "tensor", "achieved": best["tflops"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": best["tflops"] / peaks["bf16_tflops"], "traffic": None, "peak_source": peaks["source"],
                "peak_kind": "bf16 GEMM burst (fp16 shares the tensor peak)", "kernel": "gemm_tc_kernel",
                "frac_of_sustained": best["tflops"] / peaks["bf16_tflops_sustained"]}
    return {"workload": "one ChatGLM2-6B-shaped layer (qkv, o, gate_up, down), fp16 x with 1% "
                        "outlier channels x20", "dtype": "f16", "unit": "TFLOP/s", **out,
            "roofline": roofline}


def bench_int4_twin(binding, workloads, torch, dev, peaks):
    """Section 3.4 restated on this GPU with synthetic weights.  Table 1: latency of the M = 1
    matmul on its three weight shapes with E0M4 and with INT4 weights (the same kernel serves
    both containers; every timed launch reads a different copy of the weights so that nothing
    comes from L2).  Table 2: mean absolute error of both formats on the seven matrices of a
    Qwen1.5-4B-shaped first layer (hidden 2560, intermediate 6912)."""
    table1 = []
    for _, K, N in workloads.STACKS["table1"]["matrices"]:
        w = workloads.weights_torch(K, N, workloads.seed_for("table1", K, N), dev)
        x = workloads.activations_torch(1, K, workloads.seed_for("table1", "x", K), dev)
        y = torch.empty((1, N), dtype=torch.float16, device=dev)
        ws = binding.tl_e0m4_workspace(binding.tl_e0m4_matmul_workspace(1, K, N), dev)
        row = {"K": K, "N": N}
        for fmt, quantize in (("fp4", binding.tl_e0m4_quantize), ("int4", binding.tl_int4_quantize)):
            p0, s0 = quantize(w)
            copies = int(400e6 // p0.numel()) + 1
            packed = [p0] + [p0.clone() for _ in range(copies - 1)]
            scales = [s0] + [s0.clone() for _ in range(copies - 1)]

            def sweep():
                for i in range(copies):
                    binding.tl_e0m4_matmul(x, packed[i], scales[i], N, y=y, workspace=ws)

            graph, _ = capture(binding, torch, sweep)
            graph.replay()
            ms = time_events(torch, graph.replay, 10) / copies
            row[f"{fmt}_us"] = ms * 1e3
            row[f"{fmt}_gbps"] = (K * N * BYTES_PER_WEIGHT + 2 * (K + N)) / (ms * 1e-3) / 1e9
            del packed, scales, graph
        row["acceleration"] = row["int4_us"] / row["fp4_us"]
        table1.append(row)
        del w
    table2 = []
    H, F = 2560, 6912
    for name, K, N in (("q_proj", H, H), ("k_proj", H, H), ("v_proj", H, H), ("o_proj", H, H),
                       ("up_proj", H, F), ("gate_proj", H, F), ("down_proj", F, H)):
        w = workloads.weights_torch(K, N, workloads.seed_for("table2", name), dev)
        mae = {}
        for fmt, quantize in (("fp4", binding.tl_e0m4_quantize), ("int4", binding.tl_int4_quantize)):
            w_hat = binding.tl_e0m4_dequant(*quantize(w), K, N)
            mae[fmt] = float((w_hat.double() - w.double()).abs().mean())
        table2.append({"matrix": name, "mae_fp4": mae["fp4"], "mae_int4": mae["int4"],
                       "ratio": mae["fp4"] / mae["int4"]})
    return {"what": "Section 3.4 with synthetic N(0, 0.02) weights: both formats live in one packed container, "
                    "so one kernel serves both and the dequantization costs the same",
            "table1_m1_latency": table1, "table2_mae": table2,
            "paper": {"table1_acceleration": "1.00 (Adreno), 1.33-1.56 (Mali)", "table2_ratio": "0.955-0.957"}}


def bench_group_sizes(binding, workloads, torch, dev, peaks):
    """Group sizes 128, 64 and 32 (Section 2.3 quantizes "each subgroup"; Section 3.1 uses 128):
    mean absolute quantization error, decode bandwidth (M = 1, three copies of a ChatGLM2-6B-shaped
    layer in one batch launch, 325 MB of codes: nothing comes from L2) and the prefill rate of the
    gate_up matrix at M = 2048.  Algorithmic bytes per weight are 0.5 + 4 / group."""
    import ctypes

    out = []
    shapes = [(K, N) for _ in range(3) for _, K, N in workloads.STACKS["chatglm2_6b"]["matrices"]]
    ws = binding.tl_e0m4_workspace(binding.tl_e0m4_matmul_batch_workspace(), dev)
    for group in (128, 64, 32):
        row = {"group": group, "bytes_per_weight": 0.5 + 4.0 / group}
        probs, nbytes, err, cnt = [], 0.0, 0.0, 0
        for i, (K, N) in enumerate(shapes):
            w = workloads.weights_torch(K, N, workloads.seed_for("groups", i), dev)
            packed, scales = binding.tl_e0m4_quantize(w, group=group)
            if i < 4:
                w_hat = binding.tl_e0m4_dequant(packed, scales, K, N, group=group)
                err += float((w_hat.float() - w).abs().sum())
                cnt += K * N
                del w_hat
            del w
            x = workloads.activations_torch(1, K, workloads.seed_for("groups", "x", i), dev)
            y = torch.empty((1, N), dtype=torch.float16, device=dev)
            probs.append((x, packed, scales, y))
            nbytes += K * N * row["bytes_per_weight"] + 2 * (K + N)
        row["mae"] = err / cnt
        arr = binding.make_problem_array(probs)
        fn, ptr = binding.lib().tl_e0m4_matmul_batch, ctypes.cast(arr, ctypes.c_void_p)

        def step():
            st = fn(ptr, len(arr), 1, group, ws.data_ptr(), ws.numel(), torch.cuda.current_stream().cuda_stream)
            if st != 0:
                raise RuntimeError(binding.tl_status_string(st))

        graph, _ = capture(binding, torch, step)
        graph.replay()
        ms = time_events(torch, graph.replay, 50)
        row["decode_m1_gbps"] = nbytes / (ms * 1e-3) / 1e9
        row["decode_frac_of_measured_hbm"] = row["decode_m1_gbps"] / peaks["hbm_gbs"]
        del graph
        # prefill: the gate_up matrix of the layer (index 2) at M = 2048
        K, N = shapes[2]
        M = 2048
        x = workloads.activations_torch(M, K, 5, dev)
        y = torch.empty((M, N), dtype=torch.float16, device=dev)
        pws = binding.tl_e0m4_workspace(binding.tl_e0m4_matmul_workspace(M, K, N), dev)
        run = lambda: binding.tl_e0m4_matmul(x, probs[2][1], probs[2][2], N, y=y, workspace=pws, group=group)
        for _ in range(3):
            run()
        ms = time_events(torch, run, 20)
        row["prefill_m2048_tflops"] = 2.0 * M * K * N / (ms * 1e-3) / 1e12
        out.append(row)
        del probs, arr, x, y
    return out


def bench_e0m8(binding, workloads, torch, dev, peaks, tokens=(1, 4, 16, 64, 128, 512, 2048)):
    """E0M8 (the construction of Section 2.3 with eight fraction bits kept; one byte per code plus
    4 bytes per group of 128, 1.03125 bytes per weight): mean absolute error beside E0M4's, the
    quantizer and dequantizer, and the matmul on three copies of a ChatGLM2-6B-shaped layer (631 MB
    of codes) from 1 to 2048 tokens: as one tl_e0m8_matmul call per matrix and, up to 128 tokens, as
    one tl_e0m8_matmul_batch call for all twelve, each captured in a CUDA graph.
    t_roof = max(bytes / measured HBM peak, flops / measured tensor peak)."""
    bpw = 1.0 + 4.0 / 128.0
    out = {"bytes_per_weight": bpw}
    K, N = 4096, 27392
    w = workloads.weights_torch(K, N, workloads.seed_for("e0m8", "offline"), dev)
    packed, scales = binding.tl_e0m8_quantize(w)
    ms = time_events(torch, lambda: binding.tl_e0m8_quantize(w, packed=packed, scales=scales), 20)
    out["quantize_gbps"] = K * N * (4 + bpw) / (ms * 1e-3) / 1e9
    w_hat = binding.tl_e0m8_dequant(packed, scales, K, N)
    ms = time_events(torch, lambda: binding.tl_e0m8_dequant(packed, scales, K, N, out=w_hat), 20)
    out["dequant_gbps"] = K * N * (2 + bpw) / (ms * 1e-3) / 1e9
    out["mae"] = float((w_hat.float() - w).abs().mean())
    p4, s4 = binding.tl_e0m4_quantize(w)
    out["mae_e0m4"] = float((binding.tl_e0m4_dequant(p4, s4, K, N).float() - w).abs().mean())
    del w, w_hat, packed, scales, p4, s4
    shapes = [(K, N) for _ in range(3) for _, K, N in workloads.STACKS["chatglm2_6b"]["matrices"]]
    mats = []
    for i, (K, N) in enumerate(shapes):
        w = workloads.weights_torch(K, N, workloads.seed_for("e0m8", i), dev)
        mats.append((K, N) + tuple(binding.tl_e0m8_quantize(w)))
        del w
    rows = []
    for M in tokens:
        xs = [workloads.activations_torch(M, K, workloads.seed_for("e0m8", "x", i), dev) for i, (K, _, _, _) in enumerate(mats)]
        ys = [torch.empty((M, N), dtype=torch.float16, device=dev) for _, N, _, _ in mats]
        ws = binding.tl_e0m4_workspace(max([256] + [binding.tl_e0m8_matmul_workspace(M, K, N) for K, N, _, _ in mats]), dev)

        def step():
            for (K, N, pk, sc), x, y in zip(mats, xs, ys):
                binding.tl_e0m8_matmul(x, pk, sc, N, y=y, workspace=ws)

        graph, launches = capture(binding, torch, step)
        graph.replay()
        ms = time_events(torch, graph.replay, 20)
        nbytes = sum(K * N * bpw + 2 * M * (K + N) for K, N, _, _ in mats)
        flops = sum(2.0 * M * K * N for K, N, _, _ in mats)
        t_roof = max(nbytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12))
        row = {"M": M, "us": ms * 1e3, "launches": launches, "gbps": nbytes / (ms * 1e-3) / 1e9,
               "tflops": flops / (ms * 1e-3) / 1e12, "t_roof_over_t": t_roof / (ms * 1e-3)}
        del graph
        if M <= 128:
            lws = binding.tl_e0m4_workspace(binding.tl_e0m4_matmul_batch_workspace(), dev)
            arr = binding.make_problem_array([(x, pk, sc, y) for (_, _, pk, sc), x, y in zip(mats, xs, ys)])
            graph, launches = capture(binding, torch, lambda: binding.tl_e0m8_matmul_batch(arr, M, lws))
            graph.replay()
            ms = time_events(torch, graph.replay, 20)
            row["list"] = {"us": ms * 1e3, "launches": launches, "gbps": nbytes / (ms * 1e-3) / 1e9,
                           "tflops": flops / (ms * 1e-3) / 1e12, "t_roof_over_t": t_roof / (ms * 1e-3),
                           "frac_of_measured_hbm": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
            del graph, arr, lws
        rows.append(row)
        del xs, ys
    out["matmul"] = rows
    return out


def bench_e0mx(binding, workloads, torch, dev, peaks):
    """E0M3 and E0M5 (the construction of Section 2.3 with three or five fraction bits kept; bits / 8 + 4 / 128
    bytes per weight): mean absolute error, quantizer and dequantizer rates on a 4096 x 27392 matrix and the
    tensor-core matmul on it at 16 and 2048 tokens."""
    K, N = 4096, 27392
    w = workloads.weights_torch(K, N, workloads.seed_for("e0mx", "offline"), dev)
    rows = []
    for bits in (3, 5):
        bpw = bits / 8.0 + 4.0 / 128.0
        packed, scales = binding.tl_e0mx_quantize(w, bits)
        ms = time_events(torch, lambda: binding.tl_e0mx_quantize(w, bits, packed=packed, scales=scales), 10)
        row = {"bits": bits, "bytes_per_weight": bpw, "quantize_gbps": K * N * (4 + bpw) / (ms * 1e-3) / 1e9}
        w_hat = binding.tl_e0mx_dequant(packed, scales, K, N, bits)
        ms = time_events(torch, lambda: binding.tl_e0mx_dequant(packed, scales, K, N, bits, out=w_hat), 10)
        row["dequant_gbps"] = K * N * (2 + bpw) / (ms * 1e-3) / 1e9
        row["mae"] = float((w_hat.float() - w).abs().mean())
        del w_hat
        for M in (16, 2048):
            x = workloads.activations_torch(M, K, workloads.seed_for("e0mx", "x", M), dev, 0.01 if M > 16 else 0.0)
            y = torch.empty((M, N), dtype=torch.float16, device=dev)
            ws = binding.tl_e0m4_workspace(max(256, int(binding.lib().tl_e0mx_matmul_workspace(M, K, N, bits))), dev)
            run = lambda: binding.tl_e0mx_matmul(x, packed, scales, N, bits, y=y, workspace=ws)
            for _ in range(3):
                run()
            us = time_events(torch, run, 10) * 1e3
            row[f"matmul_m{M}"] = {"us": us, "gbps": (K * N * bpw + 2 * M * (K + N)) / us / 1e3,
                                   "tflops": 2.0 * M * K * N / us / 1e6}
        rows.append(row)
    return rows


def bench_list_sweep(binding, workloads, torch, dev, peaks, layers=4):
    """Batched decoding: `layers` ChatGLM2-6B-shaped layers (433 MB of weights at 4 layers, every matrix
    with its own activations) as ONE tl_e0m4_matmul_batch call against one tl_e0m4_matmul call per
    matrix, at token counts where the weights still bound the step.  t_roof = max(bytes / measured HBM
    peak, flops / measured tensor peak)."""
    out = []
    for M in (4, 16, 64, 128):
        problems, x_all, y_all = build_stack(binding, workloads, torch, dev, "chatglm2_6b", layers, M, seed=77)
        nbytes = sum(p["K"] * p["N"] * BYTES_PER_WEIGHT + 2 * M * (p["K"] + p["N"]) for p in problems)
        flops = sum(2.0 * M * p["K"] * p["N"] for p in problems)
        ws = binding.tl_e0m4_workspace(max([binding.tl_e0m4_matmul_batch_workspace()] +
                                           [binding.tl_e0m4_matmul_workspace(M, p["K"], p["N"]) for p in problems]), dev)
        row = {"M": M, "layers": layers,
               "t_roof_us": max(nbytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)) * 1e6}
        batch_step, _arr = make_batch_step(binding, torch, problems, M, ws)
        for name, step in (("list", batch_step), ("per_call", make_call_step(binding, torch, problems, M, ws))):
            graph, launches = capture(binding, torch, step)
            graph.replay()
            us = time_events(torch, graph.replay, 20) * 1e3
            row[name] = {"us": us, "launches": launches, "gbps": nbytes / us / 1e3, "tflops": flops / us / 1e6,
                         "t_roof_over_t": row["t_roof_us"] / us}
            del graph
        out.append(row)
        del problems, x_all, y_all, ws
    return out


def bench_decode_layer_chain(binding, workloads, torch, dev, peaks, layers=6, M=1):
    """One decode token through `layers` ChatGLM2-6B-shaped transformer layers as a framework would
    run them, every matmul DEPENDING on the one before (no list call possible), with this library's
    fused entry points:  s = rmsnorm(h) -> qkv = s.Wqkv + bias -> (attention left out; its output
    stands in as the first 4096 features of qkv) -> h = a.Wo + h -> s = rmsnorm(h) ->
    g = swiglu(s.Wgate_up) -> h = g.Wdown + h.  Six launches per layer, all in one CUDA graph with
    programmatic dependent launch between them; weights of every layer distinct (no L2 reuse)."""
    H, QKV, F = 4096, 4608, 13696
    ws = binding.tl_e0m4_workspace(max(binding.tl_e0m4_matmul_workspace(M, H, 2 * F), 256), dev)
    lw = []
    for layer in range(layers):
        mats = {}
        for name, K, N in (("qkv", H, QKV), ("o", H, H), ("gate_up", H, 2 * F), ("down", F, H)):
            w = workloads.weights_torch(K, N, workloads.seed_for("chain", layer, name), dev)
            mats[name] = binding.tl_e0m4_quantize(w)
            del w
        lw.append(mats)
    gamma = torch.ones(H, dtype=torch.float16, device=dev)
    bias = torch.zeros(QKV, dtype=torch.float16, device=dev)
    h = workloads.activations_torch(M, H, 1234, dev)
    s = torch.empty_like(h)
    qkv = torch.empty((M, QKV), dtype=torch.float16, device=dev)
    g = torch.empty((M, F), dtype=torch.float16, device=dev)

    def step():
        for mats in lw:
            binding.tl_rmsnorm(h, gamma, 1e-5, y=s)
            binding.tl_e0m4_matmul_bias(s, mats["qkv"][0], mats["qkv"][1], QKV, bias, y=qkv, workspace=ws)
            binding.tl_e0m4_matmul_add(qkv[:, :H], mats["o"][0], mats["o"][1], H, h, y=h, workspace=ws)
            binding.tl_rmsnorm(h, gamma, 1e-5, y=s)
            binding.tl_e0m4_matmul_swiglu(s, mats["gate_up"][0], mats["gate_up"][1], 2 * F, y=g, workspace=ws)
            binding.tl_e0m4_matmul_add(g, mats["down"][0], mats["down"][1], H, h, y=h, workspace=ws)

    graph, launches = capture(binding, torch, step)
    graph.replay()
    us = time_events(torch, graph.replay, 20) * 1e3 / layers
    nbytes = (H * QKV + H * H + H * 2 * F + F * H) * BYTES_PER_WEIGHT
    out = {"layers": layers, "M": M, "launches_per_layer": launches // layers, "us_per_layer": us,
           "weight_gbps": nbytes / us / 1e3, "t_roof_us": nbytes / (peaks["hbm_gbs"] * 1e3),
           "t_roof_over_t": nbytes / (peaks["hbm_gbs"] * 1e3) / us}
    del graph
    # The same layers as ONE tl_e0m4_matmul_chain call: four steps per layer, each waiting for its
    # predecessor inside the persistent kernel, the two rms-norms folded into the steps that consume
    # them (gamma = 1 here, so the weights are the same).
    cws = binding.tl_e0m4_workspace(binding.tl_e0m4_matmul_chain_workspace(), dev)
    steps = []
    for mats in lw:
        steps.append(dict(x=h, packed=mats["qkv"][0], scales=mats["qkv"][1], y=qkv, epilogue="bias", addend=bias,
                          rms_eps=1e-5, after_previous=True))
        steps.append(dict(x=qkv[:, :H], packed=mats["o"][0], scales=mats["o"][1], y=h, epilogue="add", addend=h,
                          after_previous=True))
        steps.append(dict(x=h, packed=mats["gate_up"][0], scales=mats["gate_up"][1], y=g, epilogue="swiglu",
                          rms_eps=1e-5, after_previous=True))
        steps.append(dict(x=g, packed=mats["down"][0], scales=mats["down"][1], y=h, epilogue="add", addend=h,
                          after_previous=True))
    arr = binding.make_step_array(steps)
    graph, launches = capture(binding, torch, lambda: binding.tl_e0m4_matmul_chain(arr, M, cws))
    for _ in range(3):
        graph.replay()
    cus = time_events(torch, graph.replay, 20) * 1e3 / layers
    out.update({"chain_launches": launches, "chain_us_per_layer": cus, "chain_weight_gbps": nbytes / cus / 1e3,
                "chain_t_roof_over_t": nbytes / (peaks["hbm_gbs"] * 1e3) / cus,
                "chain_launch": "one tl_e0m4_matmul_chain call for all layers (rms-norms folded into qkv and gate_up)"})
    return out


def bench_rmsnorm(binding, workloads, torch, dev, peaks):
    """Fused rms-norm on a prefill-sized activation (larger than L2 over the rotating set), with
    the residual add folded in, and the fused layer-norm on the same activation.  Algorithmic bytes: 2 read + 2 written per element; with
    a residual 4 read + 4 written (the sum goes back to the residual stream)."""
    M, K = 8192, 4096
    xs = [workloads.activations_torch(M, K, 900 + i, dev, 0.01) for i in range(4)]   # 4 x 64 MB
    rs = [workloads.activations_torch(M, K, 910 + i, dev) for i in range(4)]
    gamma = torch.ones(K, dtype=torch.float16, device=dev)
    y = torch.empty((M, K), dtype=torch.float16, device=dev)

    def plain():
        for x in xs:
            binding.tl_rmsnorm(x, gamma, 1e-5, y=y)

    def fused_add():
        for x, r in zip(xs, rs):
            binding.tl_rmsnorm(x, gamma, 1e-5, residual=r, sum_out=r, y=y)

    beta = torch.zeros(K, dtype=torch.float16, device=dev)

    def layer():
        for x in xs:
            binding.tl_layernorm(x, gamma, beta, 1e-5, y=y)

    out = {"shape": [M, K], "dtype": "f16"}
    for name, fn, bytes_per_elem in (("plain", plain, 4), ("with_residual", fused_add, 8), ("layernorm", layer, 4)):
        for _ in range(3):
            fn()
        ms = time_events(torch, fn, 5) / len(xs)
        gbps = M * K * bytes_per_elem / (ms * 1e-3) / 1e9
        out[name] = {"ms": ms, "gbps": gbps, "frac_of_measured_hbm": gbps / peaks["hbm_gbs"]}
    x1 = workloads.activations_torch(1, K, 920, dev)
    y1 = torch.empty_like(x1)
    graph, _ = capture(binding, torch, lambda: [binding.tl_rmsnorm(x1, gamma, 1e-5, y=y1) for _ in range(20)])
    graph.replay()
    out["decode_row_us"] = time_events(torch, graph.replay, 10) / 20 * 1e3
    return out


def bench_matmul_add(binding, workloads, torch, dev):
    """The matmul with the residual add fused in (tl_e0m4_matmul_add) beside the plain matmul and
    the unfused pair (plain matmul, then an element-wise add kernel of the framework)."""
    out = []
    for M, K, N in ((1, 13696, 4096), (2048, 4096, 4096)):
        w = workloads.weights_torch(K, N, workloads.seed_for("fuse", K, N), dev)
        packed, scales = binding.tl_e0m4_quantize(w)
        del w
        x = workloads.activations_torch(M, K, 930, dev)
        r = workloads.activations_torch(M, N, 931, dev)
        y = torch.empty((M, N), dtype=torch.float16, device=dev)
        ws = binding.tl_e0m4_workspace(binding.tl_e0m4_matmul_workspace(M, K, N), dev)

        def plain():
            binding.tl_e0m4_matmul(x, packed, scales, N, y=y, workspace=ws)

        def fused():
            binding.tl_e0m4_matmul_add(x, packed, scales, N, r, y=y, workspace=ws)

        def unfused():
            binding.tl_e0m4_matmul(x, packed, scales, N, y=y, workspace=ws)
            torch.add(y, r, out=y)

        row = {"M": M, "K": K, "N": N}
        for name, fn in (("matmul_us", plain), ("fused_add_us", fused), ("matmul_then_add_us", unfused)):
            for _ in range(3):
                fn()
            row[name] = time_events(torch, fn, 20) * 1e3
        out.append(row)
    return out


def bench_matmul_swiglu(binding, workloads, torch, dev):
    """ChatGLM2-6B-shaped gate_up (4096 x 2*13696, gate and up columns interleaved in blocks of 8)
    with the gated activation fused in (tl_e0m4_matmul_swiglu), beside the plain matmul and the
    unfused sequence (plain matmul, then the framework's silu and multiply kernels)."""
    K, F = 4096, 13696
    w = binding.interleave_gate_up(workloads.weights_torch(K, F, 940, dev), workloads.weights_torch(K, F, 941, dev))
    packed, scales = binding.tl_e0m4_quantize(w)
    del w
    out = []
    for M in (1, 2048):
        x = workloads.activations_torch(M, K, 942, dev)
        y = torch.empty((M, 2 * F), dtype=torch.float16, device=dev)
        o = torch.empty((M, F), dtype=torch.float16, device=dev)
        ws = binding.tl_e0m4_workspace(binding.tl_e0m4_matmul_workspace(M, K, 2 * F), dev)

        def plain():
            binding.tl_e0m4_matmul(x, packed, scales, 2 * F, y=y, workspace=ws)

        def fused():
            binding.tl_e0m4_matmul_swiglu(x, packed, scales, 2 * F, y=o, workspace=ws)

        def unfused():
            binding.tl_e0m4_matmul(x, packed, scales, 2 * F, y=y, workspace=ws)
            yb = y.view(M, F // 8, 2, 8)
            torch.mul(torch.nn.functional.silu(yb[:, :, 0, :]), yb[:, :, 1, :], out=o.view(M, F // 8, 8))

        row = {"M": M, "K": K, "N": 2 * F}
        for name, fn in (("matmul_us", plain), ("fused_swiglu_us", fused), ("matmul_then_silu_mul_us", unfused)):
            for _ in range(3):
                fn()
            row[name] = time_events(torch, fn, 10) * 1e3
        out.append(row)
    return out


def bench_kv_append(binding, workloads, torch, dev, peaks):
    """In-place KV-cache append: a prefill-sized write (8 x 32 heads x 2048 new rows of 128 into
    caches of 4096 rows, two caches in rotation: 134 MB of new rows are read and written per
    call) and one decode step (1 new row per head).  Algorithmic bytes: 2 read + 2 written per new element."""
    B, H, L, D = 8, 32, 4096, 128
    S = 2048
    caches = [torch.zeros((B, H, L, D), dtype=torch.float16, device=dev) for _ in range(2)]
    fresh = [torch.randn((B, H, S, D), dtype=torch.float16, device=dev) for _ in range(2)]
    pos = torch.full((B,), 1024, dtype=torch.int32, device=dev)

    def prefill():
        for c, f in zip(caches, fresh):
            binding.tl_kv_append(c, f, pos)

    for _ in range(3):
        prefill()
    ms = time_events(torch, prefill, 5) / len(caches)
    gbps = B * H * S * D * 4 / (ms * 1e-3) / 1e9
    one = torch.randn((B, H, 1, D), dtype=torch.float16, device=dev)
    graph, _ = capture(binding, torch, lambda: [binding.tl_kv_append(caches[0], one, pos) for _ in range(20)])
    graph.replay()
    step_us = time_events(torch, graph.replay, 10) / 20 * 1e3
    return {"cache": [B, H, L, D], "prefill_rows": S, "prefill_ms": ms, "prefill_gbps": gbps,
            "frac_of_measured_hbm": gbps / peaks["hbm_gbs"], "decode_step_us": step_us,
            "copy_avoided_per_decode_step_mb": B * H * L * D * 2 * 2 / 1e6}


def bench_offline(binding, workloads, torch, dev):
    """Throughput of the offline steps on one 4096 x 27392 matrix."""
    K, N = 4096, 27392
    w = workloads.weights_torch(K, N, 123, dev)
    packed, scales = binding.tl_e0m4_quantize(w)
    out = torch.empty((K, N), dtype=torch.float16, device=dev)
    for _ in range(3):
        binding.tl_e0m4_quantize(w, packed, scales)
        binding.tl_e0m4_dequant(packed, scales, K, N, out=out)
    q_ms = time_events(torch, lambda: binding.tl_e0m4_quantize(w, packed, scales), 5)
    d_ms = time_events(torch, lambda: binding.tl_e0m4_dequant(packed, scales, K, N, out=out), 5)
    q_bytes = K * N * (4 + BYTES_PER_WEIGHT)
    d_bytes = K * N * (2 + BYTES_PER_WEIGHT)
    return ({"gbps": q_bytes / (q_ms * 1e-3) / 1e9, "ms": q_ms, "shape": [K, N], "input": "f32"},
            {"gbps": d_bytes / (d_ms * 1e-3) / 1e9, "ms": d_ms, "shape": [K, N]})


def bench_m_sweep(binding, workloads, torch, dev, peaks, stack_name, tokens, layers=8):
    """The M sweep of a configuration on `layers` layers of its stack (every layer has its own
    weights, 0.9-1.3 GB in all, so nothing comes from L2).  Up to 128 tokens a point is measured
    twice: as ONE tl_e0m4_matmul_batch call over all matrices (every matrix with its own
    activations) and as one tl_e0m4_matmul call per matrix; above 128 tokens per call only (the
    activations of a layer are then shared by all layers to bound memory).  Every leg is a CUDA
    graph.  t_roof = max(bytes / measured HBM peak, flops / measured tensor peak); `bound` names the
    larger of the two."""
    spec = workloads.STACKS[stack_name]
    mats = []
    for layer in range(layers):
        for name, K, N in spec["matrices"]:
            w = workloads.weights_torch(K, N, workloads.seed_for("sweep", stack_name, layer, name), dev)
            mats.append((K, N) + tuple(binding.tl_e0m4_quantize(w)))
            del w
    rows = []
    for M in tokens:
        own = M <= 128  # own activations per matrix (what a list call needs); shared per shape above
        outl = 0.01 if M > 16 else 0.0
        if own:
            xs = [workloads.activations_torch(M, K, workloads.seed_for("sweep", "x", i), dev, outl)
                  for i, (K, _, _, _) in enumerate(mats)]
            ys = [torch.empty((M, N), dtype=torch.float16, device=dev) for _, N, _, _ in mats]
        else:
            xk = {K: workloads.activations_torch(M, K, workloads.seed_for("sweep", "x", K), dev, outl)
                  for K, _, _, _ in mats}
            yn = {N: torch.empty((M, N), dtype=torch.float16, device=dev) for _, N, _, _ in mats}
            xs = [xk[K] for K, _, _, _ in mats]
            ys = [yn[N] for _, N, _, _ in mats]
        nbytes = sum(K * N * BYTES_PER_WEIGHT + 2 * M * (K + N) for K, N, _, _ in mats)
        flops = sum(2.0 * M * K * N for K, N, _, _ in mats)
        t_hbm, t_tc = nbytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)
        t_roof = max(t_hbm, t_tc)
        row = {"M": M, "bound": "hbm" if t_hbm >= t_tc else "tensor", "t_roof_us": t_roof * 1e6}
        ws = binding.tl_e0m4_workspace(max([binding.tl_e0m4_matmul_batch_workspace()] +
                                           [binding.tl_e0m4_matmul_workspace(M, K, N) for K, N, _, _ in mats]), dev)
        legs = []
        if own:
            arr = binding.make_problem_array([(x, pk, sc, y) for (_, _, pk, sc), x, y in zip(mats, xs, ys)])
            legs.append(("list", lambda: binding.tl_e0m4_matmul_batch(arr, M, ws)))

        def per_call():
            for (K, N, pk, sc), x, y in zip(mats, xs, ys):
                binding.tl_e0m4_matmul(x, pk, sc, N, y=y, workspace=ws)

        legs.append(("per_call", per_call))
        for name, fn in legs:
            graph, launches = capture(binding, torch, fn)
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            time.sleep(0.1)  # let the power-cap controller forget the previous point
            us, mhz = time_events_clocked(torch, graph.replay, 20 if M <= 256 else 5, dev.index or 0)
            us *= 1e3
            row[name] = {"us": us, "launches": launches, "gbps": nbytes / us / 1e3, "tflops": flops / us / 1e6,
                         "t_roof_over_t": t_roof * 1e6 / us, "sm_mhz": mhz}
            del graph
        row["best"] = max(row[k]["t_roof_over_t"] for k, _ in legs)
        rows.append(row)
        del xs, ys, ws
    return {"stack": stack_name, "layers": layers, "weight_bytes": sum(K * N * BYTES_PER_WEIGHT for K, N, _, _ in mats),
            "points": rows}


def run_sustained(torch, graph, nbytes, index, seconds=1.5, chunk_steps=None, ms_per_step=1.0):
    """The headline step launched back to back for `seconds`, the SM clock sampled every 10 ms inside
    the region.  The steps are timed in chunks (a CUDA event after each), every chunk gets the median of
    the clock samples that fall into it (the host clock and the device time line are aligned at the first
    record), and the rate is reported overall and per 50-MHz clock bin."""
    chunk_steps = chunk_steps or max(1, int(round(50.0 / ms_per_step)))   # chunks of about 50 ms
    chunks = max(4, int(seconds * 1e3 / (chunk_steps * ms_per_step)))
    events = [torch.cuda.Event(enable_timing=True) for _ in range(chunks + 1)]
    samples = []
    stop = threading.Event()
    sampler = ClockSampler(index)

    def poll(t0):
        while not stop.is_set() and sampler.nv is not None:
            try:
                samples.append((time.perf_counter() - t0, sampler.nv.nvmlDeviceGetClockInfo(sampler.h, sampler.nv.NVML_CLOCK_SM)))
                sampler._once()
            except Exception:
                break
            stop.wait(0.01)

    torch.cuda.synchronize()
    t0 = time.perf_counter()
    events[0].record()
    thread = threading.Thread(target=poll, args=(t0,), daemon=True)
    thread.start()
    for c in range(chunks):
        for _ in range(chunk_steps):
            graph.replay()
        events[c + 1].record()
    torch.cuda.synchronize()
    stop.set()
    thread.join()
    edges = [0.0] + [events[0].elapsed_time(e) * 1e-3 for e in events[1:]]
    total_s = edges[-1]
    bins = {}
    for c in range(chunks):
        inside = sorted(mhz for t, mhz in samples if edges[c] <= t < edges[c + 1])
        if not inside:
            continue
        key = int(round(inside[len(inside) // 2] / 50.0) * 50)
        b = bins.setdefault(key, [0.0, 0])
        b[0] += edges[c + 1] - edges[c]
        b[1] += chunk_steps
    all_mhz = sorted(m for _, m in samples)
    first = nbytes * chunk_steps / (edges[1] - edges[0]) / 1e9
    last = nbytes * chunk_steps / (edges[-1] - edges[-2]) / 1e9
    return {"value": nbytes * chunks * chunk_steps / total_s / 1e9, "unit": UNIT, "seconds": total_s,
            "steps": chunks * chunk_steps, "first_chunk_gbps": first, "last_chunk_gbps": last,
            "sm_mhz_median": all_mhz[len(all_mhz) // 2] if all_mhz else None, "sm_max_mhz": sampler.max_mhz,
            "reasons": sorted(sampler.reasons), "clock_samples": len(all_mhz),
            "gbps_by_sm_mhz": {str(k): nbytes * v[1] / v[0] / 1e9 for k, v in sorted(bins.items())}}


def bench_launch_floor(binding, torch, dev):
    """What a launch costs on this machine whatever the kernel does: the smallest problem the matmul
    accepts (one tile: 128 x 16) launched back to back in one CUDA graph, each launch depending on
    its predecessor through programmatic dependent launch as every launch of the library does."""
    w = torch.zeros((128, 16), dtype=torch.float32, device=dev)
    pk, sc = binding.tl_e0m4_quantize(w)
    x = torch.zeros((1, 128), dtype=torch.float16, device=dev)
    y = torch.empty((1, 16), dtype=torch.float16, device=dev)
    ws = binding.tl_e0m4_workspace(binding.tl_e0m4_matmul_workspace(1, 128, 16), dev)
    graph, _ = capture(binding, torch, lambda: [binding.tl_e0m4_matmul(x, pk, sc, 16, y=y, workspace=ws) for _ in range(100)])
    graph.replay()
    return {"one_tile_matmul_back_to_back_us": time_events(torch, graph.replay, 10) * 1e3 / 100}


def _r(v, digits=4):
    return None if v is None else round(float(v), digits)


def make_summary(line, peaks):
    """The figures that matter, in one short object printed as the LAST key of the line."""
    out = {"workload": line["config"]["workload"], "value_gbps": _r(line["value"], 1),
           "roofline_frac": _r(line["roofline"]["frac"]), "hbm_peak_gbs": peaks["hbm_gbs"],
           "tensor_peak_tflops": peaks["bf16_tflops"],
           "per_call_gbps": _r(line["per_call"]["value"], 1),
           "per_call_frac": _r(line["per_call"]["value"] / line["n_gpus"] / peaks["hbm_gbs"]),
           "e2e_one_stream_gbps": _r(line["e2e"]["value"], 1),
           "e2e_two_streams_gbps": _r(line["e2e"]["two_streams"]["value"], 1),
           "two_lanes_gbps": _r(line["two_lanes"]["value"], 1)}
    if line.get("sustained"):
        out["sustained_gbps"] = _r(line["sustained"]["value"], 1)
        out["sustained_frac"] = _r(line["sustained"]["frac_of_measured_hbm"])
        out["sustained_sm_mhz"] = line["sustained"]["sm_mhz_median"]
    if "prefill" in line:
        out["prefill_tflops"] = {k: _r(v["tflops"], 1) for k, v in line["prefill"].items() if k.startswith("M")}
        out["prefill_frac_of_burst"] = {k: _r(v["frac_of_measured_bf16_burst"]) for k, v in line["prefill"].items()
                                        if k.startswith("M")}
    for name, sweep in line.get("sweeps", {}).items():
        out["sweep_" + name] = {f"M{r['M']}": [r["bound"], _r(r["best"], 3)] for r in sweep["points"]}
    if "decode_layer_chain" in line:
        out["decode_layer_chain"] = {k: _r(v, 3) for k, v in line["decode_layer_chain"].items()
                                     if k in ("us_per_layer", "t_roof_over_t", "chain_us_per_layer", "chain_t_roof_over_t")}
    if "int4_twin" in line:
        row = line["int4_twin"]["table1_m1_latency"][0]
        floor = line.get("launch_floor", {}).get("one_tile_matmul_back_to_back_us")
        t_roof = (row["K"] * row["N"] * BYTES_PER_WEIGHT + 2 * (row["K"] + row["N"])) / (peaks["hbm_gbs"] * 1e3)
        out["config1_gemv_4096x4096_m1"] = {"us": _r(row["fp4_us"], 2), "frac_of_hbm_roofline": _r(t_roof / row["fp4_us"]),
                                            "launch_floor_us": _r(floor, 2),
                                            "frac_of_roofline_plus_launch_floor":
                                                _r((t_roof + floor) / row["fp4_us"]) if floor else None}
    if "cpu_baseline" in line:
        out["cpu_oracle_gbps"] = _r(line["cpu_baseline"]["value"], 4)
    return out


def run_native(args):
    import torch

    from paper_2403_20041_b200 import binding, build, replicas, workloads

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build()
    if dist is not None:
        dist.barrier()
    binding.lib()
    peaks = load_peaks()
    if args.object:
        # only one of the extra objects (a profiling aid: one JSON line); --M picks the token count where one applies
        if rank == 0:
            one = {"e0m8": lambda: bench_e0m8(binding, workloads, torch, dev, peaks, (args.M,)),
                   "sweep": lambda: bench_m_sweep(binding, workloads, torch, dev, peaks, args.stack, (args.M,),
                                                  layers=args.layers or 8),
                   "list_sweep": lambda: bench_list_sweep(binding, workloads, torch, dev, peaks),
                   "e0mx": lambda: bench_e0mx(binding, workloads, torch, dev, peaks),
                   "chain": lambda: bench_decode_layer_chain(binding, workloads, torch, dev, peaks,
                                                             layers=args.layers or 6),
                   "prefill": lambda: bench_prefill(binding, workloads, torch, dev, peaks),
                   "int4_twin": lambda: bench_int4_twin(binding, workloads, torch, dev, peaks),
                   "launch_floor": lambda: bench_launch_floor(binding, torch, dev)}[args.object]()
            print(json.dumps({"object": args.object, args.object: one}), flush=True)
        return

    spec = workloads.STACKS[args.stack]
    layers = args.layers or spec["layers"]
    M = args.M
    # every rank streams its own replica of the stack for its own token (weak scaling):
    problems, x_all, y_all = build_stack(binding, workloads, torch, dev, args.stack, layers, M,
                                         seed=replicas.rank_seed(0, rank))
    ws = binding.tl_e0m4_workspace(binding.tl_e0m4_matmul_batch_workspace(), dev)
    nbytes = step_bytes(spec["matrices"], layers, M)
    warm = max(args.warmup, 3)

    # headline: the whole stack as one batch (one persistent kernel per 192 problems), replayed
    # as a CUDA graph
    batch_step, _arr = make_batch_step(binding, torch, problems, M, ws)
    graph, launches_per_step = capture(binding, torch, batch_step)
    for _ in range(warm):
        graph.replay()
    torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    start = torch.cuda.Event(enable_timing=True)
    end = torch.cuda.Event(enable_timing=True)
    replicas.barrier(dist)
    torch.cuda.synchronize()
    sampler.start()
    start.record()
    for _ in range(args.steps):
        graph.replay()
    end.record()
    clocks = sampler.stop()  # graph replays are asynchronous: the GPU is still inside the timed region
    torch.cuda.synchronize()
    replicas.barrier(dist)
    total_ms = replicas.max_over_ranks(start.elapsed_time(end), dist, dev)
    ms_per_step = total_ms / args.steps
    value = replicas.whole_job_throughput(nbytes, ms_per_step * 1e-3, world) / 1e9
    # the same stack as one tl_e0m4_matmul call per matrix (one kernel launch each), also a graph
    call_graph, call_launches = capture(binding, torch, make_call_step(binding, torch, problems, M, ws))
    for _ in range(warm):
        call_graph.replay()
    call_ms = time_events(torch, call_graph.replay, max(3, min(args.steps, 100)))
    per_call = {"value": nbytes / (call_ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": call_ms,
                "launches_per_step": call_launches,
                "launch": "one tl_e0m4_matmul call per matrix, all captured in one CUDA graph"}

    # end to end through the host-buffer entry point: all x of the step in one pinned buffer,
    # copied in, the batch, all y copied back to pinned host memory
    e2e_steps = max(3, min(args.steps, 100))
    hx = torch.empty(x_all.shape, dtype=torch.float16).pin_memory()
    hx.copy_(x_all.cpu())
    hy = torch.empty(y_all.shape, dtype=torch.float16).pin_memory()

    def host_step():
        binding.tl_e0m4_matmul_batch_host(_arr, M, hx, x_all, hy, y_all, ws)

    for _ in range(3):
        host_step()
    serial_ms = time_events(torch, host_step, e2e_steps)
    serial_ms = replicas.max_over_ranks(serial_ms, dist, dev)
    h2d = x_all.numel() * 2
    d2h = y_all.numel() * 2

    # The same call issued on two streams in turn, each with its own staging buffers, pinned host
    # buffers and scratch (the weights are shared): step i + 1's copy-in and step i - 1's copy-out
    # run under step i's kernel.  Every step still copies its x in and its y out.
    x_b, y_b = torch.empty_like(x_all), torch.empty_like(y_all)
    probs_b, xo, yo = [], 0, 0
    for pr in problems:
        K, N = pr["K"], pr["N"]
        probs_b.append((x_b[xo:xo + M * K].view(M, K), pr["packed"], pr["scales"], y_b[yo:yo + M * N].view(M, N)))
        xo += M * K
        yo += M * N
    arr_b = binding.make_problem_array(probs_b)
    ws_b = binding.tl_e0m4_workspace(binding.tl_e0m4_matmul_batch_workspace(), dev)
    hx_b = torch.empty(x_all.shape, dtype=torch.float16).pin_memory()
    hx_b.copy_(hx)
    hy_b = torch.empty(y_all.shape, dtype=torch.float16).pin_memory()
    lanes = [(_arr, hx, x_all, hy, y_all, ws, torch.cuda.Stream()),
             (arr_b, hx_b, x_b, hy_b, y_b, ws_b, torch.cuda.Stream())]
    main = torch.cuda.current_stream()

    def pipelined(steps, host=True):
        begin, done = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        begin.record(main)
        for lane in lanes:
            lane[6].wait_event(begin)
        for k in range(steps):
            arr_k, hx_k, xs_k, hy_k, ys_k, ws_k, st_k = lanes[k & 1]
            if host:
                binding.tl_e0m4_matmul_batch_host(arr_k, M, hx_k, xs_k, hy_k, ys_k, ws_k, stream=st_k)
            else:
                binding.tl_e0m4_matmul_batch(arr_k, M, ws_k, stream=st_k)
        for lane in lanes:
            ev = torch.cuda.Event()
            ev.record(lane[6])
            main.wait_event(ev)
        done.record(main)
        torch.cuda.synchronize()
        return begin.elapsed_time(done) / steps

    pipelined(4)
    e2e_ms = replicas.max_over_ranks(pipelined(e2e_steps), dist, dev)
    e2e_value = replicas.whole_job_throughput(nbytes, e2e_ms * 1e-3, world) / 1e9
    # (split panels meet in fp32 atomics, so the lanes may differ in the last fp16 bit)
    if not (hy.float() - hy_b.float()).norm() <= 1e-3 * hy.float().norm():
        raise RuntimeError("the two lanes of the end-to-end leg disagree")
    # the same two lanes with the inputs resident (no copies): what two independent steps in flight
    # gain over one step at a time, whose launch, fill and tail nothing hides
    pipelined(4, host=False)
    lanes_ms = replicas.max_over_ranks(pipelined(max(3, min(args.steps, 200)), host=False), dist, dev)
    two_lanes = {"value": replicas.whole_job_throughput(nbytes, lanes_ms * 1e-3, world) / 1e9, "unit": UNIT,
                 "ms_per_step": lanes_ms,
                 "launch": "tl_e0m4_matmul_batch issued on two streams in turn (two independent steps in flight)"}

    extra = {}
    if rank == 0 and world == 1:
        del call_graph
        torch.cuda.empty_cache()
        if not args.no_prefill:
            def settled(fn, *a, **kw):
                # every object starts from an idle GPU: the power-cap controller forgets the object before
                torch.cuda.synchronize()
                time.sleep(0.5)
                return fn(*a, **kw)

            extra["prefill"] = settled(bench_prefill, binding, workloads, torch, dev, peaks)
            extra["quantize"], extra["dequant"] = settled(bench_offline, binding, workloads, torch, dev)
            extra["int4_twin"] = settled(bench_int4_twin, binding, workloads, torch, dev, peaks)
            extra["group_sizes"] = settled(bench_group_sizes, binding, workloads, torch, dev, peaks)
            extra["e0m8"] = settled(bench_e0m8, binding, workloads, torch, dev, peaks)
            extra["e0mx"] = settled(bench_e0mx, binding, workloads, torch, dev, peaks)
            extra["sweeps"] = {
                "chatglm2_6b": settled(bench_m_sweep, binding, workloads, torch, dev, peaks, "chatglm2_6b",
                                       (1, 4, 16, 128, 512, 2048)),
                "llm14b": settled(bench_m_sweep, binding, workloads, torch, dev, peaks, "llm14b",
                                  (1, 2, 4, 8, 16, 64, 256, 1024, 4096)),
            }
            extra["launch_floor"] = settled(bench_launch_floor, binding, torch, dev)
            extra["decode_layer_chain"] = settled(bench_decode_layer_chain, binding, workloads, torch, dev, peaks)
            extra["rmsnorm"] = settled(bench_rmsnorm, binding, workloads, torch, dev, peaks)
            extra["matmul_add"] = settled(bench_matmul_add, binding, workloads, torch, dev)
            extra["matmul_swiglu"] = settled(bench_matmul_swiglu, binding, workloads, torch, dev)
            extra["kv_append"] = settled(bench_kv_append, binding, workloads, torch, dev, peaks)
        if not args.no_cpu_baseline:
            cb_bytes, times, desc = time_oracle(args.stack, M, 3)
            extra["cpu_baseline"] = {"value": cb_bytes * len(times) / sum(times) / 1e9, "unit": UNIT,
                                     "cores": host_threads(), "kind": "oracle", "sample": desc}

    # Last, so that its heat does not colour the other objects: the headline step back to back for more
    # than a second, i.e. what the power cap leaves of the burst figure.
    sustained = None
    if not args.no_sustained:
        sustained = run_sustained(torch, graph, nbytes, local_rank, seconds=args.sustained_seconds,
                                  ms_per_step=ms_per_step)
        step_s = replicas.max_over_ranks(sustained["seconds"] / sustained["steps"], dist, dev)
        sustained["value"] = replicas.whole_job_throughput(nbytes, step_s, world) / 1e9
        sustained["frac_of_measured_hbm"] = sustained["value"] / world / peaks["hbm_gbs"]

    if rank == 0:
        achieved = value / world
        # which roofline bounds a step at this M: the weight bytes or the tensor-core rate
        flops = 2.0 * M * sum(K * N for _, K, N in spec["matrices"]) * layers
        kernel = "gemv_decode_kernel" if M <= 8 else "gemm_tc_batch_kernel"
        if nbytes / peaks["hbm_gbs"] >= flops / (peaks["bf16_tflops"] * 1e3):
            roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": achieved / peaks["hbm_gbs"],
                        "traffic": (DECODE_TRAFFIC_BYTES_PER_LAYER_M1[args.stack] * layers / launches_per_step
                                    if M == 1 and DECODE_TRAFFIC_BYTES_PER_LAYER_M1.get(args.stack) else None),
                        "algorithmic_bytes_per_launch": nbytes / launches_per_step}
        else:
            tflops = flops / (ms_per_step * 1e-3) / 1e12
            roofline = {"bound": "tensor", "achieved": tflops, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                        "frac": tflops / peaks["bf16_tflops"], "traffic": None,
                        "algorithmic_flops_per_launch": flops / launches_per_step}
        roofline.update({"peak_source": peaks["source"], "kernel": kernel, "launches_per_step": launches_per_step})
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": dict(workload_config(args.stack, layers, len(spec["matrices"]), M, nbytes, world),
                           tokens_per_s_equivalent=world * M / (ms_per_step * 1e-3)),
            "roofline": roofline,
            # like `value`, one step at a time: copy x in, the list call, copy y out, on one stream
            "e2e": {"value": replicas.whole_job_throughput(nbytes, serial_ms * 1e-3, world) / 1e9, "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": serial_ms,
                    "issue": "tl_e0m4_matmul_batch_host, one stream, one step at a time",
                    "two_streams": {"value": e2e_value, "ms_per_step": e2e_ms,
                                    "issue": "the same call on two streams in turn, own staging and scratch each: "
                                             "a step's copies run under its neighbour's kernel"}},
            "two_lanes": two_lanes,
            "sustained": sustained,
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks,
            "per_call": per_call,
        }
        line.update(extra)
        line["summary"] = make_summary(line, peaks)
        print(json.dumps(line, separators=(",", ":")), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["native", "reference"], default="native")
    ap.add_argument("--stack", default="llm14b")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (0 = the stack's own)")
    ap.add_argument("--M", type=int, default=1)
    ap.add_argument("--object", default=None,
                    choices=["e0m8", "e0mx", "sweep", "list_sweep", "chain", "prefill", "int4_twin", "launch_floor"],
                    help="run only this extra object (at --M tokens where one applies) and print it")
    ap.add_argument("--no-prefill", action="store_true")
    ap.add_argument("--no-sustained", action="store_true")
    ap.add_argument("--sustained-seconds", type=float, default=1.5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus))
    else:
        if int(os.environ.get("WORLD_SIZE", "1")) != args.gpus:
            raise SystemExit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={os.environ.get('WORLD_SIZE', '1')}: "
                             "launch one rank per GPU (or run without a torchrun environment and let bench.py start them)")
        run_native(args)


def spawn_ranks(n):
    """`--gpus N` given to a plain `python bench.py`: start N ranks of this same command under
    torch.distributed.run (one replica per GPU) and pass their exit code on.  Refuses loudly when
    the box has fewer than N GPUs: a run must never report fewer GPUs than it was asked for."""
    import socket
    import subprocess

    import torch

    have = torch.cuda.device_count()
    if have < n:
        raise SystemExit(f"bench.py: --gpus {n} asked for, but this machine has {have} CUDA device(s)")
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


if __name__ == "__main__":
    main()
