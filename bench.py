#!/usr/bin/env python
"""Benchmark of the 4-bit training hot path on B200.

A step is one pass of the whole path over one batch of the ResNet-50-shaped
im2col workload (M=50176, K=2304, N=256, fp32 inputs):
    amax(A) amax(W) quant_int4(A) quant_int4(W) gemm_fwd
    amax(G) quant_grad(G) gemm_bwd gemm_wgrad
(for a layer with one column of output tiles, N <= 256, quant_int4(A) and gemm_fwd
are one kernel: luq_quant_int4_gemm_fwd; `--no-fused` keeps them apart).
`value` is whole-step throughput in TFLOP/s counting the useful 3 x 2MNK flops,
quantization included, inputs resident in HBM: the timed region is R blocks of
K replays each (R chosen so that the region lasts at least a second), the
reported step time is the median block.  The line also carries the LUQ
quantizer's HBM GB/s, the roofline of the dominant kernel, the 8-bit tensor peak
measured on this GPU with a library GEMM, the other configurations in compact
form (`configs`), an end-to-end number with host buffers, and the CPU oracle
timed on a bounded sample.

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

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the cfg2 kernels.  NOT measured by this run:
# copied from the committed single-pass ncu capture of the same step (other workloads: None).
TRAFFIC_SOURCE = "profiles/launch_list_and_dram_traffic_cfg2_step.md (committed ncu capture of this step, not this run)"
TRAFFIC_SOURCE_UNFUSED = "profiles/kernels_cfg2_full_size.md (committed ncu capture, not this run)"
NCU_TRAFFIC_BYTES = {"amax_A": 463.4e6, "amax_W": 2.4e6, "quant_int4_W": 2.4e6, "quant_int4_A+gemm_fwd": 546.3e6,
                     "amax_G": 51.4e6, "quant_grad_G": 51.4e6, "gemm_bwd": 413.0e6, "gemm_wgrad": 89.8e6}
NCU_TRAFFIC_BYTES_UNFUSED = {"quant_int4_A": 511.6e6, "gemm_fwd": 64.1e6}


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

def measure_tensor_peak(torch, seconds: float = 1.0):
    """Dense 8-bit tensor throughput of THIS GPU with library GEMMs (cuBLASLt through torch), outside
    the timed region and outside the product path: int8 x int8 -> int32 and e4m3 x e4m3 -> bf16 at
    8192^3, best of 10 launches (burst) and back to back for `seconds` (sustained).  The denominators
    of the tensor-bound fractions."""
    n = 8192
    out = {"shape": f"{n}^3", "how": "torch._int_mm / torch._scaled_mm, CUDA events; burst = best of 10, "
                                     f"sustained = back to back for >= {seconds} s"}
    flops = 2.0 * n ** 3

    def run(name, fn):
        try:
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            best = float("inf")
            for _ in range(10):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); fn(); e1.record(); torch.cuda.synchronize()
                best = min(best, e0.elapsed_time(e1))
            reps = max(10, int(seconds * 1e3 / best) + 1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                fn()
            e1.record(); torch.cuda.synchronize()
            out[name + "_burst_tflops"] = round(flops / (best * 1e-3) / 1e12, 1)
            out[name + "_sustained_tflops"] = round(flops * reps / (e0.elapsed_time(e1) * 1e-3) / 1e12, 1)
        except Exception as e:  # pragma: no cover
            out[name + "_error"] = repr(e)[:200]

    a8 = torch.randint(-7, 8, (n, n), dtype=torch.int8, device="cuda")
    b8 = torch.randint(-7, 8, (n, n), dtype=torch.int8, device="cuda").t()     # column-major B, as the library wants
    run("int8", lambda: torch._int_mm(a8, b8))
    try:
        af = a8.to(torch.float32).to(torch.float8_e4m3fn)
        bf = b8.t().contiguous().to(torch.float32).to(torch.float8_e4m3fn).t()
        one = torch.ones((), device="cuda")
        run("fp8_e4m3", lambda: torch._scaled_mm(af, bf, scale_a=one, scale_b=one, out_dtype=torch.bfloat16))
    except Exception as e:  # pragma: no cover
        out["fp8_e4m3_error"] = repr(e)[:200]
    bursts = [out[k] for k in ("int8_burst_tflops", "fp8_e4m3_burst_tflops") if k in out]
    sust = [out[k] for k in ("int8_sustained_tflops", "fp8_e4m3_sustained_tflops") if k in out]
    out["burst_tflops"] = max(bursts) if bursts else None
    out["sustained_tflops"] = max(sust) if sust else None
    del a8, b8
    torch.cuda.empty_cache()
    return out


class LayerBench:
    """One layer configuration resident on the GPU: inputs, code buffers, outputs, the contexts and
    streams of the step's schedule, and the ways to run and time a step."""

    def __init__(self, torch, binding, cfg, host_tensors, local, args, ns=None):
        self.torch, self.binding, self.cfg, self.args = torch, binding, cfg, args
        M, K, N = cfg.M, cfg.K, cfg.N
        self.M, self.K, self.N = M, K, N
        self.ns = cfg.n_samples if ns is None else ns
        self.seed = cfg.luq_seed
        A_h, W_h, G_h = host_tensors
        if cfg.dtype == "bf16":
            A_h, W_h, G_h = (t.view(np.int16) if t.dtype == np.uint16 else t for t in (A_h, W_h, G_h))
        pin = lambda a: torch.from_numpy(a).pin_memory() if isinstance(a, np.ndarray) else a  # noqa: E731
        self.host = [pin(t) for t in (A_h, W_h, G_h)]
        self.A, self.W, self.G = (t.cuda() for t in self.host)
        if cfg.dtype == "bf16":
            self.A, self.W, self.G = (t.view(torch.bfloat16) for t in (self.A, self.W, self.G))
            self.host = [t.view(torch.bfloat16) for t in self.host]
        self.ctx = binding.Context(local)
        self.ctx_g = binding.Context(local) if args.streams == 2 else self.ctx
        for c in {id(self.ctx): self.ctx, id(self.ctx_g): self.ctx_g}.values():
            if args.mma_kind is not None:
                c.set_option(binding.OPT_MMA_KIND, args.mma_kind)
            if args.pairs is not None:
                c.set_option(binding.OPT_PAIRS, args.pairs)
            if args.sum_samples and cfg.n_samples > 1:
                c.set_option(binding.OPT_SUM_SAMPLES, 1)
        self.sum_samples = bool(args.sum_samples and cfg.n_samples > 1)
        self.stream_g = torch.cuda.Stream() if args.streams == 2 else None
        dev = self.A.device
        f32 = lambda *s: torch.empty(s, dtype=torch.float32, device=dev)  # noqa: E731
        u8 = lambda *s: torch.empty(s, dtype=torch.uint8, device=dev)  # noqa: E731
        i8 = lambda n: torch.empty(n, dtype=torch.int8, device=dev)  # noqa: E731
        ns = self.ns
        self.mA, self.mW, self.mG, self.sA, self.sW, self.aG = (f32(1) for _ in range(6))
        self.cA, self.cW, self.cG = u8(M * K // 2), u8(N * K // 2), u8(ns, M * N // 2)
        # Operand bytes (the 8-bit form of the codes, written by the quantizer in the same pass) for the
        # tensors that many GEMM tiles re-read: always W and G; A when the layer is wide enough that the
        # forward product reads each row block of A four times or more.
        self.oW, self.oG = i8(N * K), i8((1 if self.sum_samples else ns) * M * N)
        self.oA = i8(M * K) if N >= 1024 else None
        self.Z, self.dA, self.dW = f32(M, N), f32(M, K), f32(N, K)
        # the forward half as one kernel where the layer has a single column of output tiles
        self.fused = (not args.no_fused) and N <= 256 and args.mma_kind != 0
        c, s = self.ctx, self
        self.calls = {
            "amax_A": lambda: c.amax(s.A, s.mA), "amax_W": lambda: c.amax(s.W, s.mW),
            "quant_int4_A": lambda: c.quant_int4(s.A, s.mA, s.cA, s.sA, s.oA),
            "quant_int4_W": lambda: c.quant_int4(s.W, s.mW, s.cW, s.sW, s.oW),
            "gemm_fwd": lambda: c.gemm_fwd(s.cA, s.sA, s.cW, s.sW, M, N, K, s.Z, s.oA, s.oW),
            "quant_int4_A+gemm_fwd": lambda: c.quant_int4_gemm_fwd(s.A, s.mA, s.cW, s.sW, M, N, K, s.cA, s.sA, s.Z, s.oW),
            "amax_G": lambda: c.amax(s.G, s.mG),
            "quant_grad_G": lambda: c.quant_grad(s.G, s.mG, s.seed, ns, s.cG, s.aG, s.oG),
            "gemm_bwd": lambda: c.gemm_bwd(s.cG, s.aG, ns, s.cW, s.sW, M, N, K, s.dA, s.oG, s.oW),
            "gemm_wgrad": lambda: c.gemm_wgrad(s.cG, s.aG, ns, s.cA, s.sA, M, N, K, s.dW, s.oG, s.oA),
        }
        if self.fused:
            self.kernels = ("amax_A", "amax_W", "quant_int4_W", "quant_int4_A+gemm_fwd",
                            "amax_G", "quant_grad_G", "gemm_bwd", "gemm_wgrad")
        else:
            self.kernels = KERNELS

    # ---- one step ------------------------------------------------------------------------------
    def step_one_stream(self, events=None):
        torch = self.torch
        for name in self.kernels:
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True); e0.record()
            self.calls[name]()
            if events is not None:
                e1 = torch.cuda.Event(enable_timing=True); e1.record()
                events[name].append((e0, e1))

    def step(self):
        """The gradient's max and LUQ pass depend on nothing the forward half of the step produces.  With
        two streams they run on a second stream, through a second context (a context's scratch and
        workspace serve one stream at a time), beside the activations' and weights' passes; the backward
        and update products wait for both.  The maxima of A and W come from one launch (luq_amax_multi):
        the small tensor's launch and reduction latency hides behind the large one's stream."""
        torch = self.torch
        if self.stream_g is None:
            return self.step_one_stream()
        s, c = self, self.ctx
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event(); fork.record(main)
        self.stream_g.wait_event(fork)
        with torch.cuda.stream(self.stream_g):
            self.ctx_g.amax(s.G, s.mG)
            self.ctx_g.quant_grad(s.G, s.mG, s.seed, s.ns, s.cG, s.aG, s.oG)
            join = torch.cuda.Event(); join.record(self.stream_g)
        if self.args.multi_amax:
            c.amax_multi([s.A, s.W], [s.mA, s.mW])
        else:
            self.calls["amax_A"](); self.calls["amax_W"]()
        if self.fused:
            self.calls["quant_int4_W"]()
            self.calls["quant_int4_A+gemm_fwd"]()
        else:
            if self.args.multi_amax:     # A and W through one quantizer launch as well
                c.quant_int4_multi([s.A, s.W], [s.mA, s.mW], [s.cA, s.cW], [s.sA, s.sW], [s.oA, s.oW])
            else:
                self.calls["quant_int4_W"](); self.calls["quant_int4_A"]()
            self.calls["gemm_fwd"]()
        main.wait_event(join)
        if self.args.wgrad_first:
            self.calls["gemm_wgrad"](); self.calls["gemm_bwd"]()
        else:
            self.calls["gemm_bwd"](); self.calls["gemm_wgrad"]()

    def launches(self):
        return self.ctx.launches + (self.ctx_g.launches if self.ctx_g is not self.ctx else 0)

    def status(self):
        return self.ctx.status() | (self.ctx_g.status() if self.ctx_g is not self.ctx else 0)

    def capture(self, fn=None, steps=1):
        """No call of the path allocates or synchronises with the host, so the steps are captured in a
        CUDA graph and replayed: the small configurations are bound by launch rate otherwise.  A graph
        holds as many consecutive steps (each complete, in stream order) as divide `steps` evenly, up to
        `--steps-per-graph`: between two graph launches the GPU idles for about 4 us, inside a graph
        the next step's first kernel is launched like any other.  The returned callable runs
        `.steps` steps per call."""
        torch = self.torch
        fn = self.step if fn is None else fn
        if self.args.no_graph:
            fn_direct = lambda: fn()  # noqa: E731
            fn_direct.steps = 1
            return fn_direct, "direct calls"
        per_graph = max(d for d in range(1, max(1, self.args.steps_per_graph) + 1) if steps % d == 0)
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                fn()
                torch.cuda.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for _ in range(per_graph):
                        fn()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph.replay()
            torch.cuda.synchronize()
            self._graphs = getattr(self, "_graphs", []) + [graph]
            replay = lambda: graph.replay()  # noqa: E731
            replay.steps = per_graph
            what = "CUDA graph of the step's calls, replayed" if per_graph == 1 else \
                f"CUDA graph of {per_graph} consecutive steps, replayed"
            return replay, what
        except Exception as e:  # pragma: no cover
            fn_direct = lambda: fn()  # noqa: E731
            fn_direct.steps = 1
            return fn_direct, f"direct calls (graph capture failed: {e!r})"

    def time_blocks(self, run_step, steps, min_seconds, barrier, max_blocks=400):
        """R blocks of `steps` replays, one event pair per block, no host synchronisation inside the
        region; R is chosen from a trial block so that the region lasts at least `min_seconds`.
        Returns the per-step milliseconds of every block."""
        torch = self.torch
        per_call = getattr(run_step, "steps", 1)
        assert steps % per_call == 0, "a block is a whole number of graph replays"
        calls = steps // per_call
        ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731
        e0, e1 = ev(), ev()
        e0.record()
        for _ in range(calls):
            run_step()
        e1.record(); torch.cuda.synchronize()
        trial_ms = max(e0.elapsed_time(e1), 1e-3)
        blocks = int(min(max_blocks, max(1, -(-min_seconds * 1e3 // trial_ms))))
        barrier()
        marks = [ev() for _ in range(blocks + 1)]
        marks[0].record()
        for b in range(blocks):
            for _ in range(calls):
                run_step()
            marks[b + 1].record()
        barrier()
        return [marks[b].elapsed_time(marks[b + 1]) / steps for b in range(blocks)]

    def close(self):
        if self.ctx_g is not self.ctx:
            self.ctx_g.close()
        self.ctx.close()


def block_stats(per_block_ms):
    v = sorted(per_block_ms)
    med = v[len(v) // 2] if len(v) % 2 else 0.5 * (v[len(v) // 2 - 1] + v[len(v) // 2])
    return {"blocks": len(v), "ms_median": med, "ms_min": v[0], "ms_max": v[-1],
            "ms_spread": (v[-1] - v[0]) / med if med else None}

def variance_study(torch, binding, inputs, local, rows=4096, block=64, pairs=256):
    """Config 5's variance study (Sec. 5.1: averaging N independent samples divides the variance of the
    weight gradient by N and leaves its mean alone; Table 1: Var[SR(x)] = (x - l)(u - x)).
    A block x block corner of dW over the first `rows` batch rows of the config-2/5 tensors:
    for each of `pairs` seed pairs (2p, 2p + 1) the GPU path quantizes G with two samples and forms
    dW from the first sample alone (n_s = 1) and from both (n_s = 2).  Reported: the empirical
    variance summed over the block for both, their ratio, and each against the closed form
        Var[dW[n,k]] = (s_A^2 / n_s) sum_m qA[m,k]^2 (|G[m,n]| - lo)(hi - |G[m,n]|)
    whose lo / hi are the CPU oracle's bin ends (the check against the oracle; outside any timed region)."""
    import oracle
    cfg = inputs.CONFIGS["cfg5"]
    A, _, G = inputs.layer_inputs(cfg, rows=rows)
    A, G = np.ascontiguousarray(A[:, :block]), np.ascontiguousarray(G[:, :block])
    M, K, N = rows, block, block
    ctx = binding.Context(local)
    Ad, Gd = torch.from_numpy(A).cuda(), torch.from_numpy(G).cuda()
    ca, sa = ctx.quant_int4(Ad, ctx.amax(Ad))
    mG = ctx.amax(Gd)
    cg = torch.empty((2, M * N // 2), dtype=torch.uint8, device="cuda")
    al = torch.empty(1, device="cuda")
    d1 = torch.empty((pairs, N, K), device="cuda")
    d2 = torch.empty((pairs, N, K), device="cuda")
    for p in range(pairs):
        ctx.quant_grad(Gd, mG, 2 * p, 2, cg, al)
        ctx.gemm_wgrad(cg[0:1], al, 1, ca, sa, M, N, K, d1[p])
        ctx.gemm_wgrad(cg, al, 2, ca, sa, M, N, K, d2[p])
    assert ctx.status() == 0
    d1, d2 = d1.double(), d2.double()
    var1 = d1.var(dim=0, unbiased=True).cpu().numpy()
    var2 = d2.var(dim=0, unbiased=True).cpu().numpy()
    mean2 = d2.mean(dim=0).cpu().numpy()
    # closed form from the oracle's bins and codes
    oa, osa, _ = oracle.quant_int4(A, oracle.amax(A)[0])
    assert np.array_equal(ca.cpu().numpy(), oa) and sa.item() == osa
    omx = oracle.amax(G)[0]
    lo, hi, _ = oracle.luq_bins(G, omx)
    alpha = float(oracle.luq_alpha(omx))
    g = np.abs(G.astype(np.float64)).reshape(-1)
    v = np.maximum((g - lo * alpha) * (hi * alpha - g), 0.0).reshape(M, N)
    Aq = oracle.dequant(oa, M * K, osa, "int4").reshape(M, K)
    closed1 = v.T @ (Aq ** 2)
    target = G.astype(np.float64).T @ Aq                      # E[dW]: LUQ is unbiased
    # the block's sum: T = sum_{m,n} Q(G)[m,n] * (sum_k Aq[m,k]), a sum of independent terms
    var_T = float((v * (Aq.sum(axis=1) ** 2)[:, None]).sum()) / 2
    z_T = abs(float(mean2.sum()) - float(target.sum())) / max(np.sqrt(var_T / pairs), 1e-300)
    ctx.close()
    return {"what": f"dW[{block}x{block}] over the first {rows} batch rows, {pairs} seed pairs (2p, 2p+1)",
            "var_ns1": float(var1.sum()), "var_ns2": float(var2.sum()),
            "ratio_ns2_over_ns1": float(var2.sum() / var1.sum()),
            "closed_form_ns1": float(closed1.sum()),
            "ns1_over_closed_form": float(var1.sum() / closed1.sum()),
            "ns2_over_closed_form": float(var2.sum() / (closed1.sum() / 2)),
            "bias_of_block_sum_in_sd": float(z_T)}


def bench_layer_compact(torch, binding, inputs, local, args, name, barrier, host_tensors=None, min_seconds=0.3):
    """Step time of one more configuration, same schedule and launch mode as the headline."""
    cfg = inputs.CONFIGS[name]
    lb = LayerBench(torch, binding, cfg, host_tensors if host_tensors is not None else inputs.layer_inputs(cfg),
                    local, args)
    for _ in range(3):
        lb.step()
    assert lb.status() == 0
    n0 = lb.launches(); lb.step(); per_step = lb.launches() - n0
    run_step, mode = lb.capture(steps=20)
    st = block_stats(lb.time_blocks(run_step, 20, min_seconds, barrier))
    assert lb.status() == 0
    M, K, N = cfg.M, cfg.K, cfg.N
    out = {"workload": f"M={M} K={K} N={N} {cfg.dtype}, {lb.ns} sample(s)", "ms_per_step": round(st["ms_median"], 5),
           "ms_min": round(st["ms_min"], 5), "blocks": st["blocks"],
           "tflops": round(3 * 2.0 * M * N * K / (st["ms_median"] * 1e-3) / 1e12, 2),
           "launches_per_step": per_step, "launch": mode, "fused_forward": lb.fused}
    if lb.ns > 1:
        out["sample_planes"] = "summed into one (LUQ_OPT_SUM_SAMPLES)" if lb.sum_samples else "one per sample"
    lb.close()
    del lb
    torch.cuda.empty_cache()
    return out

def run_sweep(args, binding, inputs, torch, local, exponents=None, extras=True, emit=True):
    """Quantizer bandwidth sweep (config 4): amax + LUQ quantize-and-pack on 1-D fp32
    gradient tensors of 2^20..2^30 elements, 1 and 2 samples.  GB/s = algorithmic bytes
    (4 + 4 + 0.5 n_s per element: the tensor is read twice, codes written once) / time.
    "cold": a 512 MB buffer is overwritten before every repetition (L2 flushed);
    "warm": back-to-back repetitions."""
    ctx = binding.Context(local)
    peaks = load_peaks()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    rows = []
    for e in (exponents or inputs.SWEEP_EXPONENTS):
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
            for name, fn, nbytes in () if not extras else (
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
    ctx.close()
    del flush
    torch.cuda.empty_cache()
    if emit:
        print(json.dumps({"metric": "luq_quantizer_hbm_gbs", "unit": "GB/s", "workload": "cfg4 sweep", "dtype": "f32",
                          "hbm_peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"], "rows": rows}))
    return rows


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
        exps = tuple(int(e) for e in args.sweep_exponents.split(",")) if args.sweep_exponents else None
        run_sweep(args, binding, inputs, torch, local, exponents=exps, extras=not args.sweep_quick)
        return

    cfg = inputs.CONFIGS[args.workload]
    if args.rows:
        import dataclasses
        cfg = dataclasses.replace(cfg, M=min(cfg.M, args.rows))
    host_tensors = inputs.layer_inputs(cfg)
    lb = LayerBench(torch, binding, cfg, host_tensors, local, args)
    M, K, N, ns, seed = lb.M, lb.K, lb.N, lb.ns, lb.seed
    dev = lb.A.device
    ctx, ctx_g = lb.ctx, lb.ctx_g

    for _ in range(max(args.warmup, 3)):
        lb.step_one_stream()
    assert lb.status() == 0

    sampler = ClockSampler(gpu_physical_index(local))
    sampler.start()
    sampler.ready.wait(10.0)
    launches0 = lb.launches()
    lb.step()
    launches_per_step = lb.launches() - launches0
    run_step, launch_mode = lb.capture(steps=args.steps)
    # The timed region: blocks of K replays, an event pair around each, at least a second in total.
    t_region = time.perf_counter()
    per_block = lb.time_blocks(run_step, args.steps, args.min_seconds, barrier)
    t_region = time.perf_counter() - t_region
    assert lb.status() == 0
    stats = block_stats(per_block)
    ms_per_step = replicas.max_over_ranks(stats["ms_median"], dev)
    launches = launches_per_step * args.steps * stats["blocks"]
    # The same K steps once more, on one stream, with an event pair around every call, for the
    # per-kernel durations (the extra event records lengthen a step, so this pass is not the one the
    # throughput comes from).
    events = {k: [] for k in lb.kernels}
    try:   # hold the GPU back while the host queues the pass, or idle time would be booked on the kernels
        torch.cuda._sleep(int(args.steps * 0.35e-3 * 2.0e9))
    except Exception:  # pragma: no cover
        pass
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        lb.step_one_stream(events)
    t1.record()
    barrier()
    sampler.stop_flag.set()
    instrumented_ms = t0.elapsed_time(t1) / args.steps
    flops_step = 3 * 2.0 * M * N * K
    value = world * flops_step / (ms_per_step * 1e-3) / 1e12

    per_kernel_ms = {k: sum(a.elapsed_time(b) for a, b in v) / len(v) for k, v in events.items()}
    alg = algorithmic(cfg, ns)
    alg["quant_int4_A+gemm_fwd"] = (alg["quant_int4_A"][0] + 0.5 * N * K + 4 * M * N, alg["gemm_fwd"][1])
    peaks = load_peaks()
    # 8-bit tensor peak: measured here with a library GEMM (burst: these kernels run for tens of
    # microseconds at the full SM clock); the nominal 2 x bf16 figure is kept beside it.
    tensor_peak = None if args.no_peak else measure_tensor_peak(torch)
    nominal_peak = 2.0 * peaks["bf16_tflops"]
    fp8_peak = (tensor_peak or {}).get("burst_tflops") or nominal_peak
    tensor_peak_source = ("measured in this run: library 8-bit GEMM, burst" if (tensor_peak or {}).get("burst_tflops")
                          else f"{peaks['source']} bf16 burst x2 (nominal ratio; no 8-bit library GEMM ran)")
    props = torch.cuda.get_device_properties(local)
    clocks_summary = sampler.summary()
    sm_max_mhz = float(clocks_summary.get("sm_max_mhz") or 1965.0)
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
        kernels[k] = {"ms": round(ms, 5), "bound": bound, "achieved": round(ach, 2), "peak": peak, "unit": unit,
                      "frac": round(ach / peak, 4), "tflops": round(f / (ms * 1e-3) / 1e12, 2) if f else None,
                      "gbs": round(b / (ms * 1e-3) / 1e9, 1), "frac_hbm": round(b / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)}
        if f:
            kernels[k]["frac_tensor_nominal_2x_bf16"] = round(f / (ms * 1e-3) / 1e12 / nominal_peak, 4)
        if k == "quant_grad_G":
            # Secondary figure, a MODEL, not a roofline: issue cycles per warp and element of the LUQ kernel
            # (about 21 for decision and packing plus, per sample, 20 for the five wide multiplies of
            # Philox4x32-10 and 3 for the operand bytes) against what 4 sub-partitions per SM issue.
            cycles = 21 + ns * (20 + 3)
            issue_peak = props.multi_processor_count * 4 * sm_max_mhz * 1e6 * 32 / cycles / 1e9   # Gelt/s
            kernels[k]["issue_model_frac"] = round(M * N / (ms * 1e-3) / 1e9 / issue_peak, 4)
            kernels[k]["issue_model_peak_gelts"] = round(issue_peak, 1)
    dominant = max(per_kernel_ms, key=per_kernel_ms.get)
    d = kernels[dominant]
    full_cfg2 = args.workload == "cfg2" and not args.rows
    roofline = {"kernel": dominant, "bound": d["bound"], "achieved": d["achieved"], "peak": d["peak"], "unit": d["unit"],
                "frac": d["frac"],
                "traffic": (NCU_TRAFFIC_BYTES.get(dominant) or NCU_TRAFFIC_BYTES_UNFUSED.get(dominant)) if full_cfg2 else None,
                "traffic_source": (TRAFFIC_SOURCE if dominant in NCU_TRAFFIC_BYTES else
                                   TRAFFIC_SOURCE_UNFUSED if dominant in NCU_TRAFFIC_BYTES_UNFUSED else None) if full_cfg2 else None,
                "algorithmic_bytes": alg[dominant][0], "algorithmic_flops": alg[dominant][1],
                "peak_source": {"hbm": f"{peaks['source']} hbm copy", "tensor": tensor_peak_source}[d["bound"]]}
    # whole step against its own HBM ceiling: every tensor read twice (max, quantize), codes written and
    # read by the GEMMs, fp32 outputs written
    eb = 2 if cfg.dtype == "bf16" else 4
    step_bytes = (2 * eb * (M * K + N * K + M * N) + 0.5 * (M * K + N * K + ns * M * N)
                  + (0.5 * M * K + 0.5 * N * K + 4 * M * N) + (0.5 * ns * M * N + 0.5 * N * K + 4 * M * K)
                  + (0.5 * ns * M * N + 0.5 * M * K + 4 * N * K))
    step_roofline = {"algorithmic_bytes": step_bytes, "hbm_floor_ms": step_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3,
                     "frac_of_hbm_ceiling": round(step_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3 / ms_per_step, 4),
                     "frac_of_tensor_peak": round(value / world / fp8_peak, 4)}

    # ---- the variant the paper proposes against the max passes (Sec. 7): every tensor is quantized with
    # the estimate of earlier steps while its own maximum is measured in the same kernel - one read of each
    # tensor instead of two.  Reported beside the headline, not as it: the codes differ (a lagging
    # estimate saturates / clips), the named path is max-then-quantize.
    hindsight = None
    if not args.no_graph and not args.rows and not args.no_variants:
        try:
            eA, eW, eG = lb.mA.clone(), lb.mW.clone(), lb.mG.clone()      # estimates, initialised with the true maxima
            meas = torch.empty(3, device=dev)

            def hindsight_step():
                main = torch.cuda.current_stream()
                fork = torch.cuda.Event(); fork.record(main)
                side_stream = lb.stream_g if lb.stream_g is not None else main
                if lb.stream_g is not None:
                    lb.stream_g.wait_event(fork)
                with torch.cuda.stream(side_stream):
                    ctx_g.quant_grad_hindsight(lb.G, eG, 0.1, seed, ns, False, lb.cG, lb.aG, meas[2:3], lb.oG)
                    join = torch.cuda.Event(); join.record(side_stream)
                ctx.quant_int4_hindsight(lb.W, eW, 0.1, lb.cW, lb.sW, meas[1:2], lb.oW)
                if lb.fused:     # A: quantized, measured and multiplied by one kernel
                    ctx.quant_int4_hindsight_gemm_fwd(lb.A, eA, 0.1, lb.cW, lb.sW, M, N, K, lb.cA, lb.sA, meas[0:1],
                                                      lb.Z, lb.oW)
                else:
                    ctx.quant_int4_hindsight(lb.A, eA, 0.1, lb.cA, lb.sA, meas[0:1], lb.oA)
                    lb.calls["gemm_fwd"]()
                main.wait_event(join)
                lb.calls["gemm_bwd"](); lb.calls["gemm_wgrad"]()

            n0 = lb.launches(); hindsight_step(); h_launches = lb.launches() - n0
            h_run, _ = lb.capture(hindsight_step, steps=args.steps)
            hs = block_stats(lb.time_blocks(h_run, args.steps, 0.3, barrier))
            h_ms = replicas.max_over_ranks(hs["ms_median"], dev)
            assert lb.status() == 0
            hindsight = {"ms_per_step": h_ms, "value": world * flops_step / (h_ms * 1e-3) / 1e12, "unit": UNIT,
                         "launches_per_step": h_launches,
                         "what": "in-hindsight maxima for A, W and G (eta 0.1): no max pass, one kernel per tensor" +
                                 (", A's inside the forward product (luq_quant_int4_hindsight_gemm_fwd)" if lb.fused else "")}
        except Exception as e:  # pragma: no cover
            hindsight = {"unavailable": repr(e)}

    # ---- the nine separate calls, for comparison, when the headline used the fused forward kernel
    named = None
    if lb.fused and not args.rows and not args.no_variants:
        saved = lb.kernels, lb.fused
        lb.kernels, lb.fused = KERNELS, False
        try:
            n_run, _ = lb.capture(steps=args.steps)
            nst = block_stats(lb.time_blocks(n_run, args.steps, 0.3, barrier))
            named = {"ms_per_step": nst["ms_median"], "value": world * flops_step / (nst["ms_median"] * 1e-3) / 1e12,
                     "what": "quant_int4(A) and gemm_fwd as two kernels (nine calls per step)"}
        except Exception as e:  # pragma: no cover
            named = {"unavailable": repr(e)}
        lb.kernels, lb.fused = saved
        assert lb.status() == 0

    # ---- end to end: host buffers in, host buffers out, through the same calls.  Every step copies its
    # inputs from pinned host memory and its three results back; the copies of neighbouring steps overlap
    # with the kernels and with each other (both copy engines): two sets of device buffers, a copy-in
    # stream, the compute stream, a copy-out stream.
    e2e = None
    cpu_baseline = None
    if not args.kernel_only:
        A_p, W_p, G_p = lb.host
        Z_p, dA_p, dW_p = (torch.empty(t.shape, dtype=torch.float32).pin_memory() for t in (lb.Z, lb.dA, lb.dW))
        e2e_steps = max(6, min(args.steps, 10))
        s_cmp = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        ins = [(lb.A, lb.W, lb.G), tuple(torch.empty_like(t) for t in (lb.A, lb.W, lb.G))]
        outs = [(lb.Z, lb.dA, lb.dW), tuple(torch.empty_like(t) for t in (lb.Z, lb.dA, lb.dW))]
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_done = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]

        def e2e_calls(a, w, g, z, da, dw):
            ctx.amax(a, lb.mA); ctx.amax(w, lb.mW)
            ctx.quant_int4(w, lb.mW, lb.cW, lb.sW, lb.oW)
            if lb.fused:
                ctx.quant_int4_gemm_fwd(a, lb.mA, lb.cW, lb.sW, M, N, K, lb.cA, lb.sA, z, lb.oW)
            else:
                ctx.quant_int4(a, lb.mA, lb.cA, lb.sA, lb.oA)
                ctx.gemm_fwd(lb.cA, lb.sA, lb.cW, lb.sW, M, N, K, z, lb.oA, lb.oW)
            ctx.amax(g, lb.mG); ctx.quant_grad(g, lb.mG, seed, ns, lb.cG, lb.aG, lb.oG)
            ctx.gemm_bwd(lb.cG, lb.aG, ns, lb.cW, lb.sW, M, N, K, da, lb.oG, lb.oW)
            ctx.gemm_wgrad(lb.cG, lb.aG, ns, lb.cA, lb.sA, M, N, K, dw, lb.oG, lb.oA)

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
        e2e_ms = replicas.max_over_ranks(t0.elapsed_time(t1) / e2e_steps, dev)
        h2d = sum(t.numel() * t.element_size() for t in (A_p, W_p, G_p))
        d2h = sum(t.numel() * t.element_size() for t in (Z_p, dA_p, dW_p))
        e2e = {"value": world * flops_step / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
               "steps": e2e_steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "overlap": "copies of neighbouring steps overlap with the kernels (3 streams, 2 buffer sets)"}
        del ins, outs
        torch.cuda.empty_cache()

    # ---- the other configurations in compact form (rank 0, one GPU): cfg1, cfg3, cfg5 step times and the
    # quantizer sweep's two largest practical sizes; config 5 with its variance study
    configs = None
    variance = None
    if rank == 0 and world == 1 and not args.kernel_only and not args.rows and not args.no_configs:
        configs = {}
        try:
            if args.workload in ("cfg2", "cfg5"):
                other = "cfg5" if args.workload == "cfg2" else "cfg2"
                configs[other] = bench_layer_compact(torch, binding, inputs, local, args, other, barrier,
                                                     host_tensors=lb.host)
            for name in ("cfg1", "cfg3"):
                if name != args.workload:
                    configs[name] = bench_layer_compact(torch, binding, inputs, local, args, name, barrier)
            configs["cfg4"] = [{k: r[k] for k in ("elements", "n_samples", "cold")}
                               for r in run_sweep(args, binding, inputs, torch, local, exponents=(26, 28),
                                                  extras=False, emit=False)]
        except Exception as e:  # pragma: no cover
            configs["error"] = repr(e)[:300]
    if rank == 0 and world == 1 and not args.kernel_only and not args.rows and (args.workload == "cfg5" or configs is not None):
        try:
            variance = variance_study(torch, binding, inputs, local)
            if configs is not None and "cfg5" in configs:
                configs["cfg5"]["variance"] = variance
        except Exception as e:  # pragma: no cover
            variance = {"unavailable": repr(e)[:300]}

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
                       "fused_forward": "quant_int4(A) + gemm_fwd in one kernel (luq_quant_int4_gemm_fwd)" if lb.fused else "no",
                       "operand_bytes": "W,G" + (",A" if lb.oA is not None else "") +
                                        ": the quantizers also write the codes' 8-bit form, the GEMMs are handed it",
                       "sample_planes": ("one operand plane = the sum of the samples' bytes (LUQ_OPT_SUM_SAMPLES); "
                                         "the gradient products read it once and divide by the sample count")
                                        if lb.sum_samples else "one per sample",
                       "streams": "2: gradient max + LUQ beside the activation/weight passes and the forward product"
                                  if args.streams == 2 else "1",
                       "amax_A_and_W": ("one launch (luq_amax_multi; without the fused forward kernel also luq_quant_int4_multi)"
                                        if (args.multi_amax and args.streams == 2) else "two launches"),
                       "l2": "inputs (%d MB of activations per step) against a 126 MB L2; no explicit flush" % (lb.A.numel() * lb.A.element_size() >> 20)},
            "timing": {"blocks": stats["blocks"], "steps_per_block": args.steps, "ms_per_step": "median block",
                       "ms_min": stats["ms_min"], "ms_max": stats["ms_max"], "ms_spread": stats["ms_spread"],
                       "timed_region_s": round(t_region, 3)},
            "step_roofline": step_roofline,
            "tensor_peak_measured": tensor_peak, "tensor_peak_nominal_2x_bf16": nominal_peak,
            "luq_quantizer_gbs": kernels["quant_grad_G"]["gbs"],
            "luq_quantizer_frac_hbm": kernels["quant_grad_G"]["frac_hbm"],
            "amax_plus_luq_gbs": round((alg["amax_G"][0] + alg["quant_grad_G"][0]) /
                                       ((per_kernel_ms["amax_G"] + per_kernel_ms["quant_grad_G"]) * 1e-3) / 1e9, 1),
            "ms_per_step_with_per_kernel_events": round(instrumented_ms, 5),
            "hindsight_variant": hindsight, "separate_forward_kernels_variant": named,
            "roofline": roofline, "kernels": kernels, "configs": configs, "variance": variance,
            "e2e": e2e, "cpu_baseline": cpu_baseline,
            "gpu_launches": int(launches), "clocks": clocks_summary,
        }
        print(json.dumps(line))
    lb.close()
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
    ap.add_argument("--min-seconds", type=float, default=1.0, help="least duration of the timed region")
    ap.add_argument("--no-graph", action="store_true", help="time direct calls instead of a replayed CUDA graph")
    ap.add_argument("--sweep-exponents", default=None,
                    help="cfg4: comma-separated log2 sizes instead of the whole sweep (e.g. 26 for a profiling run)")
    ap.add_argument("--sweep-quick", action="store_true", help="cfg4: max + LUQ only, without the variant quantizers")
    ap.add_argument("--sum-samples", type=int, default=1, choices=(0, 1),
                    help="1 (default) = with several samples the quantizer writes one operand plane, the sum of the "
                         "samples' bytes, and the backward / update products read it (LUQ_OPT_SUM_SAMPLES): same "
                         "results bit for bit at one sample's product cost; 0 = one plane per sample")
    ap.add_argument("--steps-per-graph", type=int, default=10,
                    help="a replayed CUDA graph holds up to this many consecutive steps (the largest divisor of --steps "
                         "not above it); 1 = one step per graph launch")
    ap.add_argument("--wgrad-first", type=int, default=0, choices=(0, 1),
                    help="1 = update product before the backward product")
    ap.add_argument("--multi-amax", type=int, default=1, choices=(0, 1),
                    help="1: max|A| and max|W| from one launch (luq_amax_multi) in the timed step")
    ap.add_argument("--no-fused", action="store_true", help="quant_int4(A) and gemm_fwd as two kernels")
    ap.add_argument("--no-peak", action="store_true", help="do not measure the 8-bit tensor peak with a library GEMM")
    ap.add_argument("--no-variants", action="store_true",
                    help="skip the in-hindsight and separate-forward-kernels variants (launch lists of the timed step alone)")
    ap.add_argument("--no-configs", action="store_true", help="skip the compact runs of the other configurations")
    ap.add_argument("--kernel-only", action="store_true", help="skip the end-to-end, other-configuration and CPU-baseline legs")
    ap.add_argument("--pairs", type=int, default=None, choices=[0, 1, 2],
                    help="CTA pairs (cta_group::2) for products whose operands both arrive as bytes; default: the library's choice")
    ap.add_argument("--mma-kind", type=int, default=None, choices=[0, 1, 2],
                    help="tensor-core operand type: 0 e4m3 (kind::f8f6f4), 1 int8 (kind::i8), 2 per product; default: the library's")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
