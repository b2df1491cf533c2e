#!/usr/bin/env python
"""Benchmark of the online W4A4 WUSH linear layer (Eq. 7) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference]

A step is one pass of the whole hot path - fused transform + quantise of X, then the
block-scaled FP4 GEMM against the pre-quantised weights - over one batch of synthetic tokens
(`wush_linear`).  Rank 0 prints ONE JSON line.  `value` is 2*M*N*K / step time summed over
ranks (each rank runs its own replica of the layer on its own tokens: weak scaling, no
data-path collective).  The line also carries the roofline of the dominant kernel, the
quantiser's HBM figure, the cuBLAS bf16 GEMM of the same shape, an end-to-end number with
host buffers, sampled clocks, and the CPU oracle timed on the host cores.

`--impl reference` times the CPU oracle (the only "reference" this method has here).
"""
import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "W4A4 WUSH linear TFLOP/s (2MNK / step time; transform+quant + FP4 GEMM)"


def load_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    except Exception:
        return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index):
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

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def pick_config(args):
    from paper_2512_00956_b200 import synth
    cfg = synth.CONFIGS[args.config]
    fmt = args.fmt or cfg.formats[0]
    M = args.m or cfg.M
    return cfg, fmt, M


def oracle_sample_seconds(cfg, fmt, M, rows, dynamic=False, budget_s=12.0):
    """Times the CPU oracle's online path (transform, quantise, dequantised product) on `rows` tokens:
    one untimed pass, then whole passes until about `budget_s` seconds of CPU work are spent.
    Returns (seconds per pass, passes)."""
    from oracle import pipeline as P
    from paper_2512_00956_b200 import synth
    d = synth.layer_inputs(cfg, M=rows)
    L = P.PreparedLayer(d["W"], d["Xc"], fmt)            # offline part, not timed
    L.forward(d["X"], dynamic=dynamic)
    n, t0 = 0, time.perf_counter()
    while True:
        L.forward(d["X"], dynamic=dynamic)
        n += 1
        dt = time.perf_counter() - t0
        if dt >= budget_s or n >= 200:
            return dt / n, n


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    """The oracle, as it stands, on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, fmt, M = pick_config(args)
    from oracle import pipeline as P
    from paper_2512_00956_b200 import synth
    rows = min(M, args.ref_rows)
    d = synth.layer_inputs(cfg, M=rows)
    L = P.PreparedLayer(d["W"], d["Xc"], fmt)
    dyn = bool(args.dynamic_ts and fmt == "nvfp4")
    for _ in range(args.warmup):
        L.forward(d["X"], dynamic=dyn)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        L.forward(d["X"], dynamic=dyn)
    dt = (time.perf_counter() - t0) / args.steps
    tf = 2.0 * rows * cfg.N * cfg.K / dt / 1e12
    sample = f"{rows} of {M} token rows x all N={cfg.N}, K={cfg.K} per step (fp64 numpy)"
    line = {"impl": "reference", "metric": METRIC, "value": tf, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "M": M, "K": cfg.K, "N": cfg.N, "format": fmt, "sample_rows": rows},
            "cpu_baseline": {"value": tf, "unit": "TFLOP/s", "cores": host_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": tf, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def run_ours(args):
    import numpy as np
    import torch
    from paper_2512_00956_b200 import dist as D
    from paper_2512_00956_b200 import prepare, synth, wush

    rank, local_rank, world = D.init()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    wush.lib()                                           # fail loudly if the library is missing
    peaks = load_peaks()
    cfg, fmt, M = pick_config(args)
    g = synth.GROUP[fmt]
    K, N = cfg.K, cfg.N
    out_dtype = torch.bfloat16 if args.out == "bf16" else torch.float32

    def up(bits):
        return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(dev)

    Xh_bits = synth.activations(cfg, M=M)
    W, Xc = up(synth.weights(cfg)), up(synth.calibration(cfg))
    layer = prepare.QuantizedLinear(W, Xc, fmt, transform=args.transform)
    X0 = up(Xh_bits)
    ws_bytes = wush.linear_workspace_bytes(M, K, g)
    stream = torch.cuda.current_stream()

    # ---- buffer rotation: every step works on its own copy of X, workspace, Y and of the quantised
    # weights, and the copies together exceed twice the L2 capacity, so each step's data is cold
    # while the (tiny) kernel code stays warm.
    set_bytes = X0.numel() * 2 + ws_bytes + M * N * (2 if args.out == "bf16" else 4) + layer.w_codes.numel() + layer.w_scales.numel()
    nsets = max(2, int((2 * 126e6) // set_bytes) + 2)
    sets = []
    for i in range(nsets):
        sets.append(dict(X=X0.clone(), Y=torch.empty((M, N), dtype=out_dtype, device=dev),
                         ws=torch.empty(ws_bytes, dtype=torch.uint8, device=dev),
                         wq=layer.w_codes.clone(), wsc=layer.w_scales.clone(),
                         status=torch.zeros(4, dtype=torch.int32, device=dev)))
    for d_ in sets:
        d_["xq"] = d_["ws"][: M * K // 2].view(M, K // 2)
        d_["xs"] = d_["ws"][(M * K // 2 + 15) // 16 * 16:][: wush.scale_bytes(M, K, g, wush.SF_TILED)]

    dynamic = bool(args.dynamic_ts and fmt == "nvfp4")
    ts_step = None if dynamic else layer.x_tensor_scale      # None: wush_linear finds the scale of each batch itself
    ts_buf = torch.zeros(4, dtype=torch.float32, device=dev)

    def step(d_):
        wush.linear(d_["X"], layer.T, d_["wq"], d_["wsc"], fmt, ts_step, layer.w_tensor_scale,
                    out=d_["Y"], workspace=d_["ws"])

    def quant_only(d_):
        if dynamic:
            wush.quantize_act_dynamic(d_["X"], layer.T, wush.SF_TILED, out=(d_["xq"], d_["xs"]), x_tensor_scale=ts_buf)
        else:
            wush.quantize_act(d_["X"], layer.T, fmt, layer.x_tensor_scale, wush.SF_TILED, out=(d_["xq"], d_["xs"]))

    def gemm_only(d_):
        wush.gemm_fp4(d_["xq"], d_["xs"], d_["wq"], d_["wsc"], K, fmt, layer.x_tensor_scale, layer.w_tensor_scale,
                      out=d_["Y"], status=d_["status"])

    def timed(fn, steps, what):
        """K launches of fn over the rotating sets inside ONE CUDA graph, bracketed by events on the launching
        stream: pure device time, no per-launch host latency.  Falls back to an eager loop if capture fails."""
        side = torch.cuda.Stream(device=dev)
        graph = None
        try:
            with torch.cuda.stream(side):
                for i in range(min(2, steps)):
                    fn(sets[i % nsets])
                side.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for i in range(steps):
                        fn(sets[i % nsets])
        except Exception as exc:           # pragma: no cover
            sys.stderr.write(f"[bench] CUDA-graph capture of {what} failed ({exc}); timing an eager loop\n")
            graph = None
            torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(side):
            if graph is not None:
                graph.replay()                                           # untimed warm-up replay
            side.synchronize()
            D.barrier()
            a.record(side)
            if graph is not None:
                graph.replay()
            else:
                for i in range(steps):
                    fn(sets[i % nsets])
            b.record(side)
            side.synchronize()
        D.barrier()
        return a.elapsed_time(b) / steps, graph is not None

    for i in range(max(3, args.warmup)):
        step(sets[i % nsets])
    torch.cuda.synchronize()

    # ---- timed region: exactly K steps
    sampler = ClockSampler(local_rank)
    sampler.start()
    wall0 = time.perf_counter()
    ms_rank, used_graph = timed(step, args.steps, "step")
    wall = time.perf_counter() - wall0
    clocks = sampler.stop()
    gemm_status = max(wush.linear_status(d_["ws"], M, K, g) for d_ in sets)

    # ---- per-kernel durations: the same launches, one kind per graph
    q_ms, _ = timed(quant_only, args.steps, "quantiser")
    g_ms, _ = timed(gemm_only, args.steps, "gemm")

    # ---- cuBLAS bf16 GEMM of the same shape (the paper's normaliser), same protocol
    Wb = [W] + [W.clone() for _ in range(max(1, min(3, int(252e6 // (W.numel() * 2)))))]
    Yb = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
    nb = len(Wb)

    def bf16_step(d_, _c=[0]):
        _c[0] += 1
        torch.matmul(d_["X"], Wb[_c[0] % nb].t(), out=Yb)

    bf16_ms, _ = timed(bf16_step, args.steps, "bf16 gemm")

    # ---- the two offline kernels of the path (Algorithm 2), timed once each for the record
    def once(fn, reps=5):
        fn(); torch.cuda.synchronize()
        a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a_.record(stream)
        for _ in range(reps):
            fn()
        b_.record(stream)
        torch.cuda.synchronize()
        return a_.elapsed_time(b_) / reps
    # moments of the weight matrix itself (the larger of the two inputs of Algorithm 2), caller-owned buffers
    mom_buf = torch.zeros((K // g, g, g), dtype=torch.float32, device=dev)
    cnt_buf = torch.zeros(2, dtype=torch.int64, device=dev)
    mom_ws = torch.empty(max(16, wush.lib().wush_calib_moments_workspace_bytes(N, K, g)), dtype=torch.uint8, device=dev)
    mom_ms = once(lambda: wush.calib_moments(W, g, mom_buf, cnt_buf, mom_ws), reps=10)
    wq_out = (torch.empty_like(layer.w_codes), torch.empty_like(layer.w_scales),
              torch.zeros(4, dtype=torch.float32, device=dev), torch.empty(256, dtype=torch.uint8, device=dev))
    wq_ms = once(lambda: wush.quantize_weight(W, layer.Tinv, fmt, sf=wush.SF_TILED, out=wq_out), reps=10)
    offline = {"calib_moments": {"ms": mom_ms, "GB/s": (2.0 * N * K + 4.0 * K * g) / (mom_ms * 1e-3) / 1e9, "rows": N,
                                 "note": "second-moment sums of W[N,K]; warm L2 (same buffers every repetition)"},
               "quantize_weight": {"ms": wq_ms, "GB/s": (2.0 * N * K * (2 if fmt == "nvfp4" else 1) + N * K / 2.0 + N * K / g) / (wq_ms * 1e-3) / 1e9,
                                   "note": "NVFP4 reads W twice (AbsMax pass + quantise pass); warm L2"}}

    # ---- end to end through the public call with HOST buffers: pinned X in, Y back out, every step
    Xh = torch.from_numpy(Xh_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    n_e2e = max(6, min(args.steps, 60))
    # Three streams: the pinned-host -> device copy of step i+1, the kernels of step i and the device -> host
    # copy of step i-1 overlap (the copy engines are full duplex); every step still moves its own input in
    # and its own result out inside the timed region.
    s_in, s_c, s_out = (torch.cuda.Stream(device=dev) for _ in range(3))
    nb3 = min(3, nsets)
    ev_in = [torch.cuda.Event() for _ in range(nb3)]
    ev_c = [torch.cuda.Event() for _ in range(nb3)]
    ev_out = [torch.cuda.Event() for _ in range(nb3)]
    Yh3 = [torch.empty((M, N), dtype=out_dtype).pin_memory() for _ in range(nb3)]

    def e2e_loop(n):
        for i in range(n):
            b = i % nb3
            d_ = sets[b]
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_c[b])                 # the kernels that last read this X buffer are done
                d_["X"].copy_(Xh, non_blocking=True)
                ev_in[b].record(s_in)
            with torch.cuda.stream(s_c):
                s_c.wait_event(ev_in[b])
                s_c.wait_event(ev_out[b])                # the previous result in this Y buffer has left
                step(d_)
                ev_c[b].record(s_c)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_c[b])
                Yh3[b].copy_(d_["Y"], non_blocking=True)
                ev_out[b].record(s_out)

    e2e_loop(3)
    torch.cuda.synchronize()
    D.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for st_ in (s_in, s_c, s_out):
        st_.wait_stream(stream)
    e2e_loop(n_e2e)
    for st_ in (s_in, s_c, s_out):
        stream.wait_stream(st_)
    e1.record(stream)
    torch.cuda.synchronize()
    e2e_ms_rank = e0.elapsed_time(e1) / n_e2e
    X, Y = sets[0]["X"], sets[0]["Y"]

    flops = 2.0 * M * N * K
    rate, t_max = D.whole_job_rate(flops, ms_rank * 1e-3, dev)
    e2e_rate, _ = D.whole_job_rate(flops, e2e_ms_rank * 1e-3, dev)
    D.barrier()
    if rank != 0:
        D.shutdown()
        return

    # ---- rooflines.  Dominant kernel: the FP4 GEMM (dense contraction -> tensor peak for FP4 =
    # measured bf16 burst peak x nominal FP4:bf16 ratio 4).  Quantiser: HBM.
    traffic = {}
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            for ln in f:
                if ln.strip() and not ln.startswith("#"):
                    k_, v_ = ln.split()
                    traffic[k_] = float(v_)
    except Exception:
        traffic = {}
    fp4_peak = peaks["bf16_tflops"] * 4.0
    gemm_tf = flops / (g_ms * 1e-3) / 1e12
    q_bytes = 2.0 * M * K + M * K / 2.0 + M * K / g + 2.0 * K * g
    q_gbs = q_bytes / (q_ms * 1e-3) / 1e9
    # DRAM bytes per launch from the ncu capture of the same kernel and workload (none for other token counts,
    # except M <= 128 on config 5, where the weights are the traffic whatever M is)
    gemm_kernel = "gemm_fp4_2cta_kernel" if M > 128 else "gemm_fp4_kernel"
    same_workload = (M == cfg.M) or (M <= 128 and cfg.index == 5)
    gemm_traffic = traffic.get(f"{gemm_kernel}/config{cfg.index}") if same_workload else None
    roof = {"bound": "tensor", "kernel": "gemm_fp4_2cta_kernel" if M > 128 else "gemm_fp4_kernel", "achieved": gemm_tf, "peak": fp4_peak, "unit": "TFLOP/s",
            "frac": gemm_tf / fp4_peak, "traffic": gemm_traffic, "ms": g_ms,
            "peak_source": f"{peaks['source']} bf16 burst {peaks['bf16_tflops']} TF/s x 4 (nominal FP4:bf16)",
            "frac_of_spec_9pf": gemm_tf / 9000.0,
            # the timed graph replays the kernel back to back for milliseconds, i.e. under the power cap: the
            # sustained bf16 figure x 4 is the like-for-like ceiling; "frac" keeps the stricter burst figure
            "peak_sustained": peaks["bf16_tflops_sustained"] * 4.0,
            "frac_of_sustained": gemm_tf / (peaks["bf16_tflops_sustained"] * 4.0)}
    if M <= 128:
        # decode regime: the GEMM reads every weight byte once and does almost no arithmetic per byte, so its
        # roofline is HBM: algorithmic bytes (codes + scales of X~ and W~, plus Y) over the measured copy rate
        g_bytes = M * K / 2.0 + M * K / g + N * K / 2.0 + N * K / g + M * N * (2 if args.out == "bf16" else 4)
        g_gbs = g_bytes / (g_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "kernel": gemm_kernel, "achieved": g_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": g_gbs / peaks["hbm_gbs"], "traffic": gemm_traffic, "ms": g_ms, "algorithmic_bytes": g_bytes,
                "peak_source": peaks["source"], "frac_of_spec_8tbs": g_gbs / 8000.0, "tflops": gemm_tf}
    roof_q = {"bound": "hbm", "kernel": "tq_stream_kernel", "achieved": q_gbs, "peak": peaks["hbm_gbs"],
              "unit": "GB/s", "frac": q_gbs / peaks["hbm_gbs"], "traffic": traffic.get(f"tq_stream_kernel/config{cfg.index}") if M == cfg.M else None, "ms": q_ms,
              "algorithmic_bytes": q_bytes, "peak_source": peaks["source"], "frac_of_spec_8tbs": q_gbs / 8000.0}

    cpu = None
    if not args.no_cpu_baseline:
        rows = min(M, args.ref_rows)
        sec, passes = oracle_sample_seconds(cfg, fmt, M, rows, dynamic)
        cpu = {"value": 2.0 * rows * N * K / sec / 1e12, "unit": "TFLOP/s", "cores": host_threads(), "kind": "oracle",
               "sample": f"{rows} of {M} token rows x all N per pass of the online path (fp64 numpy); "
                         f"{passes} passes, {sec:.2f} s each, {sec * passes:.0f} s of CPU work"}

    line = {"metric": METRIC, "value": rate / 1e12, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": t_max * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "fp4_e2m1 (fp32 accumulate)", "data": "synthetic",
            "config": {"workload": cfg.name, "M": M, "K": K, "N": N, "format": fmt, "g": g, "y_dtype": args.out, "transform": args.transform,
                       "x_tensor_scale": ("per batch" if dynamic else "static") if fmt == "nvfp4" else None,
                       "l2": f"cold data: {nsets} rotating buffer sets of {set_bytes / 1e6:.0f} MB (> 2x L2)",
                       "launch": "one CUDA graph of K steps" if used_graph else "eager loop", "tokens_per_rank": M},
            "roofline": roof, "roofline_quant": roof_q,
            "bf16_gemm": {"ms": bf16_ms, "tflops": flops / (bf16_ms * 1e-3) / 1e12, "speedup_linear": bf16_ms / ms_rank,
                          "speedup_gemm_only": bf16_ms / g_ms, "impl": "torch.matmul (cuBLAS)"},
            "e2e": {"value": e2e_rate / 1e12, "unit": "TFLOP/s", "h2d_bytes_per_step": int(X.numel() * 2),
                    "d2h_bytes_per_step": int(Y.numel() * Y.element_size()), "ms_per_step": e2e_ms_rank},
            "gpu_launches": (3 if dynamic else 2) * args.steps, "kernel_ms": {"transform_quant": q_ms, "gemm_fp4": g_ms},
            "gemm_status": gemm_status, "offline_kernels": offline, "clocks": clocks, "wall_s_timed_region": wall, "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)
    D.shutdown()


def run_quantiser_sweep(args):
    """`--quantiser-sweep`: wush_quantize_act alone over seven activation shapes, both formats, on a GPU that
    runs nothing else (0.3 s idle before every timed replay), one line of JSON per shape.  Random bf16 data
    and transforms: the kernel's time does not depend on the values."""
    import torch
    from paper_2512_00956_b200 import wush
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    reps = 20
    for M, K in ((2048, 4096), (1024, 8192), (4096, 4096), (4096, 8192), (4096, 14336), (8192, 8192), (16384, 8192)):
        for fmt, g in (("mxfp4", 32), ("nvfp4", 16)):
            nset = max(2, int(300e6 // (M * K * 2)) + 1)            # cold data: more than twice the L2 between reuses
            Xs = [torch.randn(M, K, device=dev).to(torch.bfloat16) for _ in range(nset)]
            T = (torch.randn(K // g, g, g, device=dev) / g ** 0.5).to(torch.bfloat16)
            outs = [(torch.empty(M, K // 2, dtype=torch.uint8, device=dev),
                     torch.zeros(wush.scale_bytes(M, K, g, wush.SF_TILED), dtype=torch.uint8, device=dev)) for _ in range(nset)]
            ts = torch.tensor([0.01], device=dev) if fmt == "nvfp4" else None
            side = torch.cuda.Stream(device=dev)
            with torch.cuda.stream(side):
                for i in range(3):
                    wush.quantize_act(Xs[i % nset], T, fmt, ts, wush.SF_TILED, out=outs[i % nset])
                side.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for i in range(reps):
                        wush.quantize_act(Xs[i % nset], T, fmt, ts, wush.SF_TILED, out=outs[i % nset])
                graph.replay()
                side.synchronize()
                times = []
                for _ in range(5):
                    time.sleep(0.3)
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(side)
                    graph.replay()
                    b.record(side)
                    side.synchronize()
                    times.append(a.elapsed_time(b) / reps * 1e3)
            us = statistics.median(times)
            nbytes = 2.0 * M * K + M * K / 2.0 + M * K / g + 2.0 * K * g
            print(json.dumps({"kernel": "tq_stream_kernel", "M": M, "K": K, "format": fmt, "us": round(us, 2),
                              "us_min": round(min(times), 2), "GB/s": round(nbytes / us / 1e3),
                              "items_per_sm": round((M / 128) * (K / 128) / 148, 1)}), flush=True)
            del Xs, outs, graph


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload index 1..5 (2 = the headline configuration)")
    ap.add_argument("--fmt", default=None, choices=[None, "mxfp4", "nvfp4", "mxfp4_ceil"])
    ap.add_argument("--dynamic-ts", action="store_true",
                    help="NVFP4: activation tensor scale from each batch (one more kernel per step) instead of calibration")
    ap.add_argument("--m", type=int, default=None, help="override the token count (config 5 sweep)")
    ap.add_argument("--out", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--transform", default="wush", choices=["wush", "wus", "hadamard", "identity"],
                    help="activation-side transform: per-block WUSH (default), WUSH without its Hadamard factor, "
                         "one shared Hadamard, or none")
    ap.add_argument("--ref-rows", type=int, default=1024, help="token rows in the CPU-oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--quantiser-sweep", action="store_true",
                    help="time wush_quantize_act alone over seven shapes (one JSON line each) and exit")
    args = ap.parse_args()
    if args.quantiser_sweep:
        run_quantiser_sweep(args)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
