#!/usr/bin/env python
"""Benchmark of the 4-bit training hot path on B200.

A step is one pass of the whole path over one batch of the ResNet-50-shaped
im2col workload (M=50176, K=2304, N=256, fp32 inputs):
    amax(A) amax(W) quant_int4(A) quant_int4(W) gemm_fwd
    amax(G) quant_grad(G) gemm_bwd gemm_wgrad
`value` is whole-step throughput in TFLOP/s counting the useful 3 x 2MNK flops,
quantization included, inputs resident in HBM.  The line also carries the LUQ
quantizer's HBM GB/s, the roofline of the dominant kernel, an end-to-end number
with host buffers, and the CPU oracle timed on a bounded sample.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 (torchrun) every rank runs an independent replica of the workload
(the path has no exchange step); time is the maximum over ranks.
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

import numpy as np  # noqa: E402

METRIC = "4bit_train_step_tflops_incl_quantize"
UNIT = "TFLOP/s"
WORKLOAD = "cfg2"
KERNELS = ("amax_A", "amax_W", "quant_int4_A", "quant_int4_W", "gemm_fwd",
           "amax_G", "quant_grad_G", "gemm_bwd", "gemm_wgrad")

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the cfg2 kernels, from the ncu
# capture summarised in profiles/kernels_cfg2_full_size.md (other workloads: None).
NCU_TRAFFIC_BYTES = {"amax_A": 469.0e6, "quant_int4_A": 511.6e6, "gemm_fwd": 64.1e6, "amax_G": 51.4e6,
                     "quant_grad_G": 52.3e6, "gemm_bwd": 416.4e6, "gemm_wgrad": 74.3e6, "amax_W": 2.4e6,
                     "quant_int4_W": 2.4e6}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def algorithmic(cfg, ns):
    """Per kernel: (bytes, flops) one launch must move / compute."""
    M, K, N = cfg.M, cfg.K, cfg.N
    eb = 2 if cfg.dtype == "bf16" else 4
    return {
        "amax_A": (eb * M * K, 0), "amax_W": (eb * N * K, 0), "amax_G": (eb * M * N, 0),
        "quant_int4_A": ((eb + 0.5) * M * K, 0), "quant_int4_W": ((eb + 0.5) * N * K, 0),
        "quant_grad_G": ((eb + 0.5 * ns) * M * N, 0),
        "gemm_fwd": (0.5 * M * K + 0.5 * N * K + 4 * M * N, 2 * M * N * K),
        "gemm_bwd": (0.5 * ns * M * N + 0.5 * N * K + 4 * M * K, 2 * M * N * K),
        "gemm_wgrad": (0.5 * ns * M * N + 0.5 * M * K + 4 * N * K, 2 * M * N * K),
    }


class ClockSampler(threading.Thread):
    """Samples SM clock, power and throttle reasons (NVML) while the timed region runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index = index
        self.samples = []
        self.stop_flag = threading.Event()
        self.ready = threading.Event()       # set after the first sample (NVML start-up can take a second)
        self.error = None

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_sm = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            while not self.stop_flag.is_set():
                sm = nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)
                pw = nv.nvmlDeviceGetPowerUsage(h) / 1000.0
                try:
                    rs = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                except Exception:
                    rs = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                self.samples.append((sm, pw, rs))
                self.ready.set()
                self.stop_flag.wait(0.01)
        except Exception as e:  # pragma: no cover
            self.error = repr(e)
            self.ready.set()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable: %s" % self.error]}
        import pynvml as nv
        names = {"hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap}
        sm = sorted(s[0] for s in self.samples)
        reasons = sorted(n for n, bit in names.items() if any(s[2] & bit for s in self.samples))
        return {"sm_mhz": float(sm[len(sm) // 2]), "sm_min_mhz": float(sm[0]), "sm_max_mhz": float(self.max_sm),
                "power_w_max": round(max(s[1] for s in self.samples), 1), "samples": len(self.samples),
                "reasons": reasons}


def gpu_physical_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# ---------------------------------------------------------------- CPU oracle --

def oracle_sample(cfg, rows: int, ns: int, tensors=None):
    """The oracle, as it stands, on the first `rows` rows of the workload's batch
    dimension.  Returns (seconds, useful flops, threads)."""
    import oracle
    from paper_2112_10769_b200 import inputs
    A, W, G = tensors if tensors is not None else inputs.layer_inputs(cfg, rows=rows)
    M, K, N = A.shape[0], cfg.K, cfg.N
    oracle.build()
    t0 = time.perf_counter()
    ca, sa, _ = oracle.quant_int4(A, oracle.amax(A)[0])
    cw, sw, _ = oracle.quant_int4(W, oracle.amax(W)[0])
    cg, al, _ = oracle.quant_luq(G, oracle.amax(G)[0], cfg.luq_seed, ns)
    oracle.gemm_fwd(ca, sa, cw, sw, M, N, K)
    oracle.gemm_bwd(cg, al, ns, cw, sw, M, N, K)
    oracle.gemm_wgrad(cg, al, ns, ca, sa, M, N, K)
    dt = time.perf_counter() - t0
    return dt, 3 * 2.0 * M * N * K, oracle.host_threads()


def run_reference(args):
    """Reference arm: the CPU oracle on the host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2112_10769_b200 import inputs
    cfg = inputs.CONFIGS[args.workload]
    rows = min(512, cfg.M)  # about a quarter of a second per step on eight cores
    tensors = inputs.layer_inputs(cfg, rows=rows)
    for _ in range(args.warmup):
        oracle_sample(cfg, rows, cfg.n_samples, tensors)
    times, flops, threads = [], 0.0, 1
    for _ in range(args.steps):
        dt, flops, threads = oracle_sample(cfg, rows, cfg.n_samples, tensors)
        times.append(dt)
    mean = sum(times) / len(times)
    value = flops / mean / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": mean * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.workload}: M={cfg.M} K={cfg.K} N={cfg.N} {cfg.dtype}, first {rows} rows of the batch per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"first {rows} of {cfg.M} batch rows, all nine stages"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ------------------------------------------------------------------ GPU arm --

def run_sweep(args, binding, inputs, torch, local):
    """Quantizer bandwidth sweep (config 4): amax + LUQ quantize-and-pack on 1-D fp32
    gradient tensors of 2^20..2^30 elements, 1 and 2 samples.  GB/s = algorithmic bytes
    (4 + 4 + 0.5 n_s per element: the tensor is read twice, codes written once) / time.
    "cold": a 512 MB buffer is overwritten before every repetition (L2 flushed);
    "warm": back-to-back repetitions."""
    ctx = binding.Context(local)
    peaks = load_peaks()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    rows = []
    for e in inputs.SWEEP_EXPONENTS:
        n = 1 << e
        x = torch.from_numpy(inputs.sweep_tensor(e)).cuda()
        mx, al = torch.empty(1, device="cuda"), torch.empty(1, device="cuda")
        for ns in (1, 2):
            codes = torch.empty((ns, n // 2), dtype=torch.uint8, device="cuda")
            reps = 20 if e <= 26 else 5
            res = {}
            for mode in ("cold", "warm"):
                times = {"amax": [], "quant": []}
                for it in range(reps + 3):
                    if mode == "cold":
                        flush.fill_(it & 0xFF)
                    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
                    ev[0].record(); ctx.amax(x, mx); ev[1].record(); ctx.quant_grad(x, mx, 0, ns, codes, al); ev[2].record()
                    torch.cuda.synchronize()
                    if it >= 3:
                        times["amax"].append(ev[0].elapsed_time(ev[1])); times["quant"].append(ev[1].elapsed_time(ev[2]))
                med = {k: sorted(v)[len(v) // 2] for k, v in times.items()}
                total = med["amax"] + med["quant"]
                res[mode] = {"amax_us": round(med["amax"] * 1e3, 2), "quant_us": round(med["quant"] * 1e3, 2),
                             "quant_gbs": round((4 + 0.5 * ns) * n / (med["quant"] * 1e-3) / 1e9, 1),
                             "amax_plus_quant_gbs": round((8 + 0.5 * ns) * n / (total * 1e-3) / 1e9, 1),
                             "frac_of_hbm_peak": round((8 + 0.5 * ns) * n / (total * 1e-3) / 1e9 / peaks["hbm_gbs"], 3)}
            # the two variants the paper proposes against the max pass and the division:
            # in-hindsight maximum (one pass over the tensor) and power-of-two scale
            mh = mx.clone()
            extra = {}
            for name, fn, nbytes in (
                    ("hindsight", lambda: ctx.quant_grad_hindsight(x, mh, 0.1, 0, ns, False, codes, al, mx), (4 + 0.5 * ns) * n),
                    ("hindsight_pw2", lambda: ctx.quant_grad_hindsight(x, mh, 0.1, 0, ns, True, codes, al, mx), (4 + 0.5 * ns) * n),
                    ("amax_plus_pw2", lambda: (ctx.amax(x, mx), ctx.quant_grad_pw2(x, mx, 0, ns, codes, al)), (8 + 0.5 * ns) * n),
                    # deterministic round-to-nearest-power (the biased FP4 baseline): no generator, one plane
                    ("amax_plus_nearest", lambda: (ctx.amax(x, mx), ctx.quant_grad_nearest(x, mx, codes, al)), 8.5 * n),
                    # the ablation's other arms (quantizer alone, max given): one region of the LUQ grid
                    # deterministic, and the uniform grid with stochastic rounding
                    ("ablation_fp4_sr", lambda: ctx.quant_grad_ablation(x, mx, 0, binding.SCHEME_FP4_SR, ns, codes, al),
                     (4 + 0.5 * ns) * n),
                    ("ablation_int4_sr", lambda: ctx.quant_grad_ablation(x, mx, 0, binding.SCHEME_INT4_SR, ns, codes, al),
                     (4 + 0.5 * ns) * n)):
                ts = []
                for it in range(reps + 3):
                    flush.fill_(it & 0xFF)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(); fn(); e1.record()
                    torch.cuda.synchronize()
                    if it >= 3:
                        ts.append(e0.elapsed_time(e1))
                t = sorted(ts)[len(ts) // 2]
                extra[name] = {"us": round(t * 1e3, 2), "gbs": round(nbytes / (t * 1e-3) / 1e9, 1),
                               "frac_of_hbm_peak": round(nbytes / (t * 1e-3) / 1e9 / peaks["hbm_gbs"], 3)}
            rows.append({"elements": n, "n_samples": ns, **res, **extra})
            del codes
        del x
        torch.cuda.empty_cache()
    assert ctx.status() == 0
    print(json.dumps({"metric": "luq_quantizer_hbm_gbs", "unit": "GB/s", "workload": "cfg4 sweep", "dtype": "f32",
                      "hbm_peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"], "rows": rows}))
    ctx.close()


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2112_10769_b200 import binding, inputs, replicas

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    if args.workload == "cfg4":
        run_sweep(args, binding, inputs, torch, local)
        return

    cfg = inputs.CONFIGS[args.workload]
    if args.rows:
        import dataclasses
        cfg = dataclasses.replace(cfg, M=min(cfg.M, args.rows))
    M, K, N, ns, seed = cfg.M, cfg.K, cfg.N, cfg.n_samples, cfg.luq_seed
    A_h, W_h, G_h = inputs.layer_inputs(cfg)
    if cfg.dtype == "bf16":
        A_h, W_h, G_h = (t.view(np.int16) for t in (A_h, W_h, G_h))
    pin = lambda a: torch.from_numpy(a).pin_memory()  # noqa: E731
    A_p, W_p, G_p = pin(A_h), pin(W_h), pin(G_h)
    A, W, G = A_p.cuda(), W_p.cuda(), G_p.cuda()
    if cfg.dtype == "bf16":
        A, W, G = (t.view(torch.bfloat16) for t in (A, W, G))
        A_p, W_p, G_p = (t.view(torch.bfloat16) for t in (A_p, W_p, G_p))
    ctx = binding.Context(local)
    if args.mma_kind is not None:
        ctx.set_option(binding.OPT_MMA_KIND, args.mma_kind)
    dev = A.device
    f32 = lambda *s: torch.empty(s, dtype=torch.float32, device=dev)  # noqa: E731
    u8 = lambda *s: torch.empty(s, dtype=torch.uint8, device=dev)  # noqa: E731
    mA, mW, mG, sA, sW, aG = (f32(1) for _ in range(6))
    cA, cW, cG = u8(M * K // 2), u8(N * K // 2), u8(ns, M * N // 2)
    # Operand bytes (the 8-bit form of the codes, written by the quantizer in the same pass) for
    # the tensors that many GEMM tiles re-read: always W and G; A when the layer is wide enough
    # that the forward product reads each row block of A four times or more.
    i8 = lambda n: torch.empty(n, dtype=torch.int8, device=dev)  # noqa: E731
    oW, oG = i8(N * K), i8(ns * M * N)
    oA = i8(M * K) if N >= 1024 else None
    Z, dA, dW = f32(M, N), f32(M, K), f32(N, K)
    Z_p, dA_p, dW_p = (torch.empty(t.shape, dtype=torch.float32).pin_memory() for t in (Z, dA, dW))

    calls = {
        "amax_A": lambda: ctx.amax(A, mA), "amax_W": lambda: ctx.amax(W, mW),
        "quant_int4_A": lambda: ctx.quant_int4(A, mA, cA, sA, oA),
        "quant_int4_W": lambda: ctx.quant_int4(W, mW, cW, sW, oW),
        "gemm_fwd": lambda: ctx.gemm_fwd(cA, sA, cW, sW, M, N, K, Z, oA, oW),
        "amax_G": lambda: ctx.amax(G, mG), "quant_grad_G": lambda: ctx.quant_grad(G, mG, seed, ns, cG, aG, oG),
        "gemm_bwd": lambda: ctx.gemm_bwd(cG, aG, ns, cW, sW, M, N, K, dA, oG, oW),
        "gemm_wgrad": lambda: ctx.gemm_wgrad(cG, aG, ns, cA, sA, M, N, K, dW, oG, oA),
    }

    def step(events=None):
        for name in KERNELS:
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True); e0.record()
            calls[name]()
            if events is not None:
                e1 = torch.cuda.Event(enable_timing=True); e1.record()
                events[name].append((e0, e1))

    for _ in range(max(args.warmup, 3)):
        step()
    assert ctx.status() == 0

    sampler = ClockSampler(gpu_physical_index(local))
    sampler.start()
    sampler.ready.wait(10.0)
    # The gradient's max and LUQ pass depend on nothing the forward half of the step produces.  With
    # --streams 2 (the default) they run on a second stream, through a second context (a context's
    # scratch and workspace serve one stream at a time), beside the activation/weight quantizers and the
    # forward GEMM; the backward and update GEMMs wait for both.
    ctx_g = binding.Context(local) if args.streams == 2 else ctx
    if args.mma_kind is not None and ctx_g is not ctx:
        ctx_g.set_option(binding.OPT_MMA_KIND, args.mma_kind)
    stream_g = torch.cuda.Stream() if args.streams == 2 else None

    def timed_step():
        if stream_g is None:
            return step()
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event(); fork.record(main)
        stream_g.wait_event(fork)
        with torch.cuda.stream(stream_g):
            ctx_g.amax(G, mG); ctx_g.quant_grad(G, mG, seed, ns, cG, aG, oG)
            join = torch.cuda.Event(); join.record(stream_g)
        for name in ("amax_A", "amax_W", "quant_int4_A", "quant_int4_W", "gemm_fwd"):
            calls[name]()
        main.wait_event(join)
        calls["gemm_bwd"](); calls["gemm_wgrad"]()

    # No call of the path allocates or synchronises with the host, so one step is captured in a CUDA
    # graph and replayed: the small configurations are bound by launch rate otherwise.
    launches0 = ctx.launches + (ctx_g.launches if ctx_g is not ctx else 0)
    timed_step()
    launches_per_step = ctx.launches + (ctx_g.launches if ctx_g is not ctx else 0) - launches0
    run_step, launch_mode = timed_step, "direct calls"
    if not args.no_graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                timed_step()
                torch.cuda.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    timed_step()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph.replay()
            torch.cuda.synchronize()
            run_step, launch_mode = graph.replay, "CUDA graph of the step's calls, replayed"
        except Exception as e:  # pragma: no cover
            launch_mode = f"direct calls (graph capture failed: {e!r})"
    # The timed region: K steps, two events around the whole of it.
    barrier()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        run_step()
    t1.record()
    barrier()
    total_ms = t0.elapsed_time(t1)
    launches = launches_per_step * args.steps
    total_ms = replicas.max_over_ranks(total_ms, dev)
    assert ctx.status() == 0 and ctx_g.status() == 0
    ms_per_step = total_ms / args.steps
    # The same K steps once more with an event pair around every call, for the per-kernel
    # durations (the 18 extra event records per step lengthen a step, so this pass is not
    # the one the throughput comes from).
    events = {k: [] for k in KERNELS}
    # 27 host calls per step here: on the short configurations the host would fall behind the GPU and
    # the idle time would be booked on the kernels.  Hold the GPU back while the host queues the pass.
    try:
        torch.cuda._sleep(int(args.steps * 0.35e-3 * 2.0e9))
    except Exception:  # pragma: no cover
        pass
    t0.record()
    for _ in range(args.steps):
        step(events)
    t1.record()
    barrier()
    sampler.stop_flag.set()
    instrumented_ms = t0.elapsed_time(t1) / args.steps
    flops_step = 3 * 2.0 * M * N * K
    value = world * flops_step / (ms_per_step * 1e-3) / 1e12

    per_kernel_ms = {k: sum(a.elapsed_time(b) for a, b in v) / len(v) for k, v in events.items()}
    alg = algorithmic(cfg, ns)
    peaks = load_peaks()
    # 8-bit tensor peak: the nominal fp8 : bf16 ratio (2) on the measured bf16 BURST figure.  The GEMMs of
    # this step run for tens of microseconds at the full SM clock, far from the power cap under which
    # the sustained figure (1.3 GHz) was taken.
    fp8_peak = 2.0 * peaks["bf16_tflops"]
    props = torch.cuda.get_device_properties(local)
    clocks_summary = sampler.summary()

    def sampler_max_mhz():
        return float(clocks_summary.get("sm_max_mhz") or 1965.0)
    kernels = {}
    for k, ms in per_kernel_ms.items():
        b, f = alg[k]
        t_hbm = b / (peaks["hbm_gbs"] * 1e9)
        t_tc = f / (fp8_peak * 1e12)
        bound = "tensor" if t_tc > t_hbm else "hbm"
        if bound == "hbm":
            ach, peak, unit = b / (ms * 1e-3) / 1e9, peaks["hbm_gbs"], "GB/s"
        else:
            ach, peak, unit = f / (ms * 1e-3) / 1e12, fp8_peak, "TFLOP/s"
        if k == "quant_grad_G":
            # The LUQ quantizer is bound by instruction issue, not by HBM: per 32 elements about 21 issue
            # cycles of decision and packing plus, per sample, 20 for the five wide multiplies of
            # Philox4x32-10 (4 issue cycles each, measured) and 3 for the operand bytes.  Peak = what
            # 4 sub-partitions per SM issue at the SM clock.
            cycles = 21 + ns * (20 + 3)
            alu_peak = props.multi_processor_count * 4 * sampler_max_mhz() * 1e6 * 32 / cycles / 1e9   # Gelt/s
            if alu_peak * 1e9 < (peaks["hbm_gbs"] * 1e9) / (b / (M * N)):
                bound, ach, peak, unit = "alu", M * N / (ms * 1e-3) / 1e9, round(alu_peak, 1), "Gelt/s"
        kernels[k] = {"ms": round(ms, 5), "bound": bound, "achieved": round(ach, 2), "peak": peak, "unit": unit,
                      "frac": round(ach / peak, 4), "tflops": round(f / (ms * 1e-3) / 1e12, 2) if f else None,
                      "gbs": round(b / (ms * 1e-3) / 1e9, 1)}
    dominant = max(per_kernel_ms, key=per_kernel_ms.get)
    d = kernels[dominant]
    roofline = {"kernel": dominant, "bound": d["bound"], "achieved": d["achieved"], "peak": d["peak"], "unit": d["unit"],
                "frac": d["frac"],
                "traffic": NCU_TRAFFIC_BYTES.get(dominant) if (args.workload == "cfg2" and not args.rows) else None,
                "algorithmic_bytes": alg[dominant][0], "algorithmic_flops": alg[dominant][1],
                "peak_source": {"hbm": f"{peaks['source']} hbm copy",
                                "tensor": f"{peaks['source']} bf16 burst x2 (8-bit operands)",
                                "alu": "derived: issue cycles per element x SM sub-partitions x SM clock"}[d["bound"]]}

    # ---- the variant the paper proposes against the max passes (Sec. 7): every tensor is quantized with
    # the estimate of earlier steps while its own maximum is measured in the same kernel - six launches
    # instead of nine, one read of each tensor instead of two.  Reported beside the headline, not as it:
    # the codes differ (a lagging estimate saturates / clips), the named path is max-then-quantize.
    hindsight = None
    if not args.no_graph:
        try:
            eA, eW, eG = mA.clone(), mW.clone(), mG.clone()      # estimates, initialised with the true maxima
            meas = torch.empty(3, device=dev)

            def hindsight_step():
                main = torch.cuda.current_stream()
                fork = torch.cuda.Event(); fork.record(main)
                side_stream = stream_g if stream_g is not None else main
                if stream_g is not None:
                    stream_g.wait_event(fork)
                with torch.cuda.stream(side_stream):
                    ctx_g.quant_grad_hindsight(G, eG, 0.1, seed, ns, False, cG, aG, meas[2:3], oG)
                    join = torch.cuda.Event(); join.record(side_stream)
                ctx.quant_int4_hindsight(A, eA, 0.1, cA, sA, meas[0:1], oA)
                ctx.quant_int4_hindsight(W, eW, 0.1, cW, sW, meas[1:2], oW)
                calls["gemm_fwd"]()
                main.wait_event(join)
                calls["gemm_bwd"](); calls["gemm_wgrad"]()

            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                hindsight_step()
                torch.cuda.synchronize()
                hgraph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(hgraph, stream=side):
                    hindsight_step()
            torch.cuda.current_stream().wait_stream(side)
            for _ in range(3):
                hgraph.replay()
            barrier()
            t0.record()
            for _ in range(args.steps):
                hgraph.replay()
            t1.record()
            barrier()
            h_ms = replicas.max_over_ranks(t0.elapsed_time(t1) / args.steps, dev)
            assert ctx.status() == 0 and ctx_g.status() == 0
            hindsight = {"ms_per_step": h_ms, "value": world * flops_step / (h_ms * 1e-3) / 1e12, "unit": UNIT,
                         "launches_per_step": 6 + (launches_per_step - 9),
                         "what": "in-hindsight maxima for A, W and G (eta 0.1): no max pass, one kernel per tensor"}
        except Exception as e:  # pragma: no cover
            hindsight = {"unavailable": repr(e)}

    # ---- end to end: host buffers in, host buffers out, through the same calls
    e2e = None
    cpu_baseline = None

    # Every step copies its inputs from pinned host memory and its three results back.  The copies
    # of neighbouring steps overlap with the kernels and with each other (both copy engines): two
    # sets of device buffers, a copy-in stream, the compute stream, a copy-out stream.
    if not args.kernel_only:
        e2e_steps = max(6, min(args.steps, 10))
        s_cmp = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        ins = [(A, W, G), tuple(torch.empty_like(t) for t in (A, W, G))]
        outs = [(Z, dA, dW), tuple(torch.empty_like(t) for t in (Z, dA, dW))]
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_done = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]

        def e2e_calls(a, w, g, z, da, dw):
            ctx.amax(a, mA); ctx.amax(w, mW)
            ctx.quant_int4(a, mA, cA, sA, oA); ctx.quant_int4(w, mW, cW, sW, oW)
            ctx.gemm_fwd(cA, sA, cW, sW, M, N, K, z, oA, oW)
            ctx.amax(g, mG); ctx.quant_grad(g, mG, seed, ns, cG, aG, oG)
            ctx.gemm_bwd(cG, aG, ns, cW, sW, M, N, K, da, oG, oW)
            ctx.gemm_wgrad(cG, aG, ns, cA, sA, M, N, K, dw, oG, oA)

        def e2e_run(n_steps):
            for i in range(n_steps):
                b = i & 1
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(ev_done[b])          # the step that last read this input set has finished
                    for dst, src in zip(ins[b], (A_p, W_p, G_p)):
                        dst.copy_(src, non_blocking=True)
                    ev_in[b].record(s_in)
                s_cmp.wait_event(ev_in[b])
                if i >= 2:
                    s_cmp.wait_event(ev_out[b])              # this output set has been copied out
                e2e_calls(*ins[b], *outs[b])
                ev_done[b].record(s_cmp)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_done[b])
                    for dst, src in zip((Z_p, dA_p, dW_p), outs[b]):
                        dst.copy_(src, non_blocking=True)
                    ev_out[b].record(s_out)
            s_cmp.wait_stream(s_out)
            s_cmp.wait_stream(s_in)

        e2e_run(2)
        barrier()
        t0.record()
        e2e_run(e2e_steps)
        t1.record()
        barrier()
        assert ctx.status() == 0
        e2e_ms = t0.elapsed_time(t1) / e2e_steps
        e2e_ms = replicas.max_over_ranks(e2e_ms, dev)
        h2d = sum(t.numel() * t.element_size() for t in (A_p, W_p, G_p))
        d2h = sum(t.numel() * t.element_size() for t in (Z_p, dA_p, dW_p))
        e2e = {"value": world * flops_step / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
               "steps": e2e_steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "overlap": "copies of neighbouring steps overlap with the kernels (3 streams, 2 buffer sets)"}
        del ins, outs
        torch.cuda.empty_cache()

    if rank == 0 and world == 1 and not args.kernel_only:
        rows = min(32768, M)   # about 15 s of host time on config 2
        dt, fl, threads = oracle_sample(cfg, rows, ns)
        cpu_baseline = {"value": fl / dt / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle",
                        "sample": f"first {rows} of {M} batch rows, all nine stages, {dt:.2f} s"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": {None: "int8 operands, int32 accumulate", 0: "e4m3 operands, f32 accumulate",
                                        1: "int8 operands, int32 accumulate", 2: "int8 operands, int32 accumulate"}[args.mma_kind], "data": "synthetic",
            "config": {"workload": f"{args.workload}: M={M} K={K} N={N}, {cfg.dtype} inputs, "
                                   f"LUQ seed {seed}, {ns} sample(s)",
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                       "launch": launch_mode,
                       "streams": "2: gradient max + LUQ beside the activation/weight quantizers and the forward GEMM"
                                  if args.streams == 2 else "1",
                       "l2": "inputs (%d MB of activations per step) against a 126 MB L2; no explicit flush" % (A.numel() * A.element_size() >> 20)},
            "luq_quantizer_gbs": kernels["quant_grad_G"]["gbs"],
            "amax_plus_luq_gbs": round((alg["amax_G"][0] + alg["quant_grad_G"][0]) /
                                       ((per_kernel_ms["amax_G"] + per_kernel_ms["quant_grad_G"]) * 1e-3) / 1e9, 1),
            "ms_per_step_with_per_kernel_events": round(instrumented_ms, 5),
            "hindsight_variant": hindsight,
            "roofline": roofline, "kernels": kernels, "e2e": e2e, "cpu_baseline": cpu_baseline,
            "gpu_launches": int(launches), "clocks": clocks_summary,
        }
        print(json.dumps(line))
    if ctx_g is not ctx:
        ctx_g.close()
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=WORKLOAD, choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"],
                    help="layer shape (the headline number is cfg2), or cfg4 = the quantizer bandwidth sweep")
    ap.add_argument("--rows", type=int, default=None, help="truncate the batch dimension M (small profiling runs)")
    ap.add_argument("--streams", type=int, choices=(1, 2), default=2,
                    help="2: the gradient's max and LUQ pass run on a second stream beside the forward half")
    ap.add_argument("--no-graph", action="store_true", help="time direct calls instead of a replayed CUDA graph")
    ap.add_argument("--kernel-only", action="store_true", help="skip the end-to-end and CPU-baseline legs")
    ap.add_argument("--mma-kind", type=int, default=None, choices=[0, 1, 2],
                    help="tensor-core operand type: 0 e4m3 (kind::f8f6f4), 1 int8 (kind::i8), 2 per product; default: the library's")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
