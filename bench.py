#!/usr/bin/env python
"""Benchmark of the quantized backward pass (arXiv 2407.12637) on B200.

One "step" is one pass of the whole hot path over one layer's gradient: abs-max statistics,
quantize + clip-out count, clipping-factor update, code expansion, dgrad and wgrad on the
integer tensor cores -- all through the C-ABI call `lbt_qconv_backward`.

Workload: the square linear layer M = O = I = 8192 (dY fp32 8192x8192; W, X 4-bit codes),
4-bit gradients, stochastic rounding: the shape the INT8-roofline target is quoted on.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

`--impl reference` times the CPU oracle (oracle/) on a bounded sample of the same workload.
With N > 1 (torchrun) every rank runs the same layer on its own GPU (weak scaling, no
collective on the data path) and rank 0 prints the aggregate.  `--dp` instead shards the batch
rows of the layer over the ranks and all-reduces the statistics and the integer weight gradient.
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

M = O = I = 8192
BITS_G = 4
OPS_PER_STEP = 2 * 2.0 * M * O * I            # dgrad + wgrad, 2 ops per multiply-accumulate
N_GRAD = M * O


def set_shape(m: int, o: int, i: int):
    """Another linear-layer shape (used for small profiler captures; the default is the benchmark)."""
    global M, O, I, OPS_PER_STEP, N_GRAD
    M, O, I = m, o, i
    OPS_PER_STEP = 2 * 2.0 * M * O * I
    N_GRAD = M * O


METRIC = "INT4 backward TOPS per layer shape (% INT8 peak); grad quantizer HBM GB/s"
TAP_EVERY = 4          # per-kernel CUDA-event taps are armed on every 4th step of the timed region
KERNELS_PER_STEP = 6   # absmax, quantize (also writes the int8 dY operand), update, expand (W and X in one launch), dgrad GEMM, wgrad GEMM
GEMM_DRAM_TRAFFIC = 329e6   # bytes per GEMM launch at M=O=I=8192, from the ncu capture of the 8192x4096x4096 case
SUSTAINED_SECONDS = 2.5     # length of the back-to-back leg that follows the timed region
BURST_REGION_S = 0.5        # a timed region shorter than this is compared with the burst peaks


def shared_config(world: int = 1) -> dict:
    """The part of `config` that names the workload: identical in the GPU arm and in the reference arm."""
    return {"workload": workload_name(),
            "l2": f"inputs larger than L2 (dY {N_GRAD * 4 >> 20} MiB fp32 + codes + int8 operands per step)",
            "parallelism": f"{world} independent replicas" if world > 1 else "single GPU"}


def workload_name() -> str:
    tag = " (config 4)" if M == O == I == 8192 else " (profiling case)"
    return f"linear M={M} O={O} I={I}, 4-bit gradients (stochastic rounding), INT4 W/X" + tag


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=p["hbm_gbs"], bf16_burst=p["bf16_tflops"],
                    bf16_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) from a thread while the timed
    region runs."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int, period_s: float = 0.0005):
        self.samples, self.mask, self.max_mhz, self.power = [], 0, None, []
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            if visible:
                index = int(visible.split(",")[index])
            self._nv, self._h = pynvml, pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None
            return
        self._period = period_s
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def _run(self):
        nv, k = self._nv, 0
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                self.mask |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                if k % 8 == 0:      # (one NVML call more: not on every sample)
                    self.power.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
            except Exception:
                pass
            k += 1
            time.sleep(self._period)

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        reasons = [name for bit, name in self.REASONS.items() if self.mask & bit]
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(self.samples),
                "power_w_max": max(self.power) if self.power else None}


# ------------------------------------------------------------------------------------ CPU oracle leg
class OraclePrep:
    """Operand codes for the oracle's contractions, decoded / quantized once by the oracle itself."""

    def __init__(self, dY_host, rawW, rawX):
        from oracle import ref
        self.dY = dY_host
        t0 = time.perf_counter()
        self.cW = ref.unpack4(rawW, O * I, True)
        self.cX = ref.unpack4(rawX, M * I, False)
        self.t_unpack = time.perf_counter() - t0
        gm, bad = ref.grad_stats(dY_host)
        self.cY = ref.quantize_grad(dY_host, 1.0, gm, BITS_G, 1, 0, 0, bad).codes.astype(np.int16)


def oracle_quantizer_seconds(prep, n_q: int) -> float:
    """The oracle's statistics + quantize + pack + update (one thread, as it stands) on the first n_q gradients."""
    from oracle import ref
    t0 = time.perf_counter()
    gm, bad = ref.grad_stats(prep.dY[:n_q])
    q = ref.quantize_grad(prep.dY[:n_q], 1.0, gm, BITS_G, 1, 0, 0, bad)
    ref.pack(q.codes, BITS_G)
    ref.update_interval(1.0, 1e-3, 1e-3, 1e-3, 1.0, BITS_G, n_q, q.n_out, bad)
    return time.perf_counter() - t0


def oracle_gemm_seconds(prep, seconds: float, threads: int, rng):
    """dgrad and wgrad of the oracle on randomly chosen outputs, about `seconds` of work on `threads` threads.
    Returns (seconds for both contractions projected to every output, outputs sampled per contraction, time spent)."""
    from oracle import ref
    cal = 64 * threads
    idx = rng.integers(0, M * I, cal)
    t0 = time.perf_counter()
    _sampled(ref, "dgrad", prep.cY, prep.cW, idx, threads)
    per_out = (time.perf_counter() - t0) / cal
    s = max(cal, int(seconds / 2 / max(per_out, 1e-9)))
    idx_d, idx_w = rng.integers(0, M * I, s), rng.integers(0, O * I, s)
    t0 = time.perf_counter()
    _sampled(ref, "dgrad", prep.cY, prep.cW, idx_d, threads)
    _sampled(ref, "wgrad", prep.cY, prep.cX, idx_w, threads)
    t_gemm = time.perf_counter() - t0
    return t_gemm * ((M * I + O * I) / (2.0 * s)), s, t_gemm


def oracle_sample(prep, seconds: float, threads: int, full_quantizer: bool = False, single_thread_seconds: float = 0.0):
    """Time the oracle on a bounded sample: statistics + quantize + pack + update on a prefix of dY (all of it
    with full_quantizer), and dgrad / wgrad on randomly chosen outputs with all cores (and, with
    single_thread_seconds > 0, once more on one thread).  Returns (projected whole-step TOPS, description,
    projected seconds per step, details)."""
    n_q = N_GRAD if full_quantizer else min(N_GRAD, 1 << 22)
    t_quant = oracle_quantizer_seconds(prep, n_q)
    rng = np.random.default_rng(0)
    gemm_all, s, t_gemm = oracle_gemm_seconds(prep, seconds, threads, rng)
    quant_full = t_quant * (N_GRAD / n_q)
    projected = quant_full + prep.t_unpack + gemm_all
    tops = OPS_PER_STEP / projected / 1e12
    desc = (f"quantizer (1 thread) on {'all' if n_q == N_GRAD else 'the first ' + str(n_q) + ' of'} {N_GRAD} gradients "
            f"({t_quant:.2f} s); dgrad and wgrad ({threads} threads) on {s} random outputs each of {M * I} ({t_gemm:.2f} s); "
            f"whole-step time projected by those ratios")
    details = {"quantizer_s": quant_full, "quantizer_elems_timed": n_q, "quantizer_threads": 1,
               "gemm_s_all_cores": gemm_all, "step_s_all_cores": projected}
    if single_thread_seconds > 0.0:
        gemm_one, s1, t1 = oracle_gemm_seconds(prep, single_thread_seconds, 1, rng)
        details.update({"gemm_s_single_thread": gemm_one, "step_s_single_thread": quant_full + prep.t_unpack + gemm_one,
                        "value_single_thread": OPS_PER_STEP / (quant_full + prep.t_unpack + gemm_one) / 1e12,
                        "single_thread_sample": f"{s1} random outputs per contraction ({t1:.2f} s)"})
    return tops, desc, projected, details


def _sampled(ref, kind, cY, other, idx, threads):
    from concurrent.futures import ThreadPoolExecutor
    parts = np.array_split(idx, threads)
    with ThreadPoolExecutor(threads) as ex:
        list(ex.map(lambda p: ref.gemm_backward(kind, cY, other, M, O, I, idx=p), parts))


def host_inputs():
    from paper_2407_12637_b200 import synth
    dY = synth.laplace_outliers(N_GRAD, 1e-3, seed=0)
    rawW = synth.code_bytes(O * I // 2, 0, 1)
    rawX = synth.code_bytes(M * I // 2, 0, 2)
    return dY, rawW, rawX


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    threads = os.cpu_count() or 1
    prep = OraclePrep(*host_inputs())
    per_step = max(0.05, min(20.0, 120.0 / (args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_sample(prep, per_step, threads)
    vals, t0, desc = [], time.perf_counter(), ""
    for _ in range(args.steps):
        v, desc, _, _ = oracle_sample(prep, per_step, threads)
        vals.append(v)
    wall = time.perf_counter() - t0
    value = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TOPS", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": OPS_PER_STEP / value / 1e9,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64 accumulate (CPU oracle)",
        "data": "synthetic", "config": shared_config(args.gpus),
        "sampling": {"sampled": True, "wall_s": wall,
                     "what": "each step times the oracle on a bounded sample of the workload and projects the whole step"},
        "cpu_baseline": {"value": value, "unit": "TOPS", "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------ GPU leg
def _median(v):
    return float(np.median(v)) if len(v) else None


def library_int8_peak(torch, sampler_index):
    """A library int8 GEMM (cuBLASLt through torch._int_mm, 8192^3) timed in this process as a DENOMINATOR only --
    it is not on the product path: best of 10 single launches (burst) and a >= 2 s back-to-back loop under the
    clock sampler (sustained).  None where the routine is unavailable."""
    try:
        n = 8192
        a = torch.randint(-8, 8, (n, n), dtype=torch.int8, device="cuda")
        b = torch.randint(-8, 8, (n, n), dtype=torch.int8, device="cuda")
        for _ in range(3):
            torch._int_mm(a, b)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        best = float("inf")
        for _ in range(10):
            e0.record(); torch._int_mm(a, b); e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        iters = max(10, int(2.2e3 / best))
        sampler = ClockSampler(sampler_index)
        e0.record()
        for _ in range(iters):
            torch._int_mm(a, b)
        e1.record()
        torch.cuda.synchronize()
        clocks = sampler.stop()
        ms = e0.elapsed_time(e1) / iters
        ops = 2.0 * n ** 3
        del a, b
        return {"burst_tops": ops / (best * 1e-3) / 1e12, "sustained_tops": ops / (ms * 1e-3) / 1e12,
                "sustained_clocks": clocks, "what": "torch._int_mm (cuBLASLt) 8192^3 int8 -> int32: best of 10 launches; "
                f"{iters} launches back to back"}
    except Exception as exc:       # noqa: BLE001 -- a missing library routine must not fail the benchmark
        return {"unavailable": f"{type(exc).__name__}: {exc}"[:200]}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2407_12637_b200 import dist_util, lbt, shapes, synth

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    lbt.lib()  # fails loudly if the CUDA library is missing
    peaks = load_peaks()

    desc = lbt.ConvDesc(**shapes.linear(M, O, I))
    dY = synth.laplace_outliers_torch(N_GRAD, 1e-3, seed=rank)
    q_W = synth.code_bytes_torch(O * I // 2, rank, 1)
    q_X = synth.code_bytes_torch(M * I // 2, rank, 2)
    st = lbt.new_state(gamma=1.0, alpha=1e-3, beta=1e-3, bits=BITS_G, rounding=lbt.ROUND_STOCHASTIC, seed=rank)
    stats = lbt.new_stats()
    scales = torch.tensor([0.01, 0.05], device="cuda")
    q_dY = torch.empty(N_GRAD // 2, dtype=torch.uint8, device="cuda")
    dX = torch.empty(M, I, device="cuda")
    dW = torch.empty(O, I, device="cuda")
    ws = torch.empty(lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, desc), dtype=torch.uint8, device="cuda")

    def step():
        lbt.qconv_backward(desc, dY, q_W, q_X, scales.data_ptr(), scales.data_ptr() + 4, st, stats, q_dY,
                           dX, dW, None, None, BITS_G, ws)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    classes = {"stats": lbt.TIME_STATS, "quantize": lbt.TIME_QUANTIZE, "expand": lbt.TIME_EXPAND,
               "dgrad": lbt.TIME_DGRAD, "wgrad": lbt.TIME_WGRAD}
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed_region(n_steps, tap_every):
        """n_steps back-to-back steps between two events, under the clock sampler.  Kernel-level taps on every
        tap_every-th step (at most 64): an armed tap puts two event records around each launch, which also keeps
        the library from chaining its launches programmatically, so the other steps run exactly as a caller's would.
        Returns (ms for the region, max over ranks; mean ms per kernel class; clock record; tapped step count)."""
        tapped_steps = [k for k in range(n_steps) if k % tap_every == 0][:64]
        taps = {name: [lbt.TimingTap(c) for _ in tapped_steps] for name, c in classes.items()}
        sampler = ClockSampler(local) if rank == 0 else None
        barrier()
        e0.record()
        armed = False
        for k in range(n_steps):
            if k in tapped_steps:
                for name in classes:
                    taps[name][tapped_steps.index(k)].arm()
                armed = True
            elif armed:
                for name in classes:
                    taps[name][0].disarm()
                armed = False
            step()
        e1.record()
        barrier()
        clocks = sampler.stop() if sampler else None
        for name in classes:
            taps[name][0].disarm()
        ms = dist_util.max_over_ranks(e0.elapsed_time(e1), "cuda")
        per_kernel = {name: float(np.mean([t.ms() for t in taps[name]])) for name in classes}
        for name in classes:
            for t in taps[name]:
                t.close()
        return ms, per_kernel, clocks, len(tapped_steps)

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    # ---- the timed region: exactly --steps steps
    ms_total, per_kernel, clocks, tapped = timed_region(args.steps, TAP_EVERY)
    state = lbt.read_state(st)
    if state.dev_status != 0:
        raise RuntimeError("device status " + lbt.status_string(state.dev_status))

    # ---- the quantizer alone (statistics, quantize + count, update): back to back ("as in training": whatever
    # of dY the L2 still holds stays) and cold (a buffer larger than L2 written before every run), each run
    # between its own pair of events, medians reported; and the back-to-back loop under one event pair, which
    # leaves out the ~3 us an event pair adds
    def quantizer_once():
        lbt.grad_stats(dY, st, stats); lbt.quantize_grad(dY, st, stats, q_dY); lbt.update_interval(st, stats)

    q_iters = 50
    for _ in range(3):
        quantizer_once()
    barrier()
    e0.record()
    for _ in range(q_iters):
        quantizer_once()
    e1.record()
    barrier()
    quant_loop_ms = dist_util.max_over_ranks(e0.elapsed_time(e1), "cuda") / q_iters
    flush = torch.empty(384 << 20, dtype=torch.uint8, device="cuda")     # 3 x the 126 MB L2
    warm_ms, cold_ms = [], []
    for _ in range(20):
        e0.record(); quantizer_once(); e1.record()
        torch.cuda.synchronize()
        warm_ms.append(e0.elapsed_time(e1))
    for _ in range(20):
        flush.fill_(1)
        e0.record(); quantizer_once(); e1.record()
        torch.cuda.synchronize()
        cold_ms.append(e0.elapsed_time(e1))
    del flush

    # ---- the same step back to back for a few seconds: the regime a training run is in (power cap reached)
    sustained = None
    if not args.no_sustained:
        n_sus = max(args.steps, int(SUSTAINED_SECONDS * 1e3 / (ms_total / args.steps)))
        ms_sus, pk_sus, clocks_sus, tapped_sus = timed_region(n_sus, max(TAP_EVERY, n_sus // 64))
        sustained = {"steps": n_sus, "ms_per_step": ms_sus / n_sus, "seconds": ms_sus * 1e-3,
                     "value": world * n_sus * OPS_PER_STEP / (ms_sus * 1e-3) / 1e12, "unit": "TOPS",
                     "clocks": clocks_sus, "kernels_ms": pk_sus, "tapped_steps": tapped_sus}

    # ---- end to end through the C ABI with host buffers (pinned), copies inside the timed region
    e2e_steps = 0 if args.no_e2e else min(args.steps, 5)
    h_dY = torch.empty(N_GRAD, dtype=torch.float32).pin_memory()
    h_dY.copy_(dY)
    h_W, h_X = q_W.cpu().pin_memory(), q_X.cpu().pin_memory()
    h_dX, h_dW = torch.empty(M, I).pin_memory(), torch.empty(O, I).pin_memory()
    h_stats = torch.empty(40, dtype=torch.uint8).pin_memory()

    def e2e_step():
        dY.copy_(h_dY, non_blocking=True)
        q_W.copy_(h_W, non_blocking=True)
        q_X.copy_(h_X, non_blocking=True)
        step()
        h_dX.copy_(dX, non_blocking=True)
        h_dW.copy_(dW, non_blocking=True)
        h_stats.copy_(stats, non_blocking=True)

    ms_e2e = float("nan")
    ms_e2e_pipelined = float("nan")
    if e2e_steps:
        # (a) one step after the other: copy in, compute, copy out on one stream
        e2e_step()
        barrier()
        e0.record()
        for _ in range(e2e_steps):
            e2e_step()
        e1.record()
        barrier()
        ms_e2e = dist_util.max_over_ranks(e0.elapsed_time(e1), "cuda")

        # (b) the same work as a three-stage pipeline over streams (copy in | compute | copy out) with two
        # sets of device buffers, as a training loop that owns its streams would drive the library
        main = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        bufs = [dict(dY=dY, W=q_W, X=q_X, dX=dX, dW=dW, stats=stats),
                dict(dY=torch.empty_like(dY), W=torch.empty_like(q_W), X=torch.empty_like(q_X),
                     dX=torch.empty_like(dX), dW=torch.empty_like(dW), stats=lbt.new_stats())]
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_comp = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]

        def pipelined(n_steps):
            for i in range(n_steps):
                b = bufs[i & 1]
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(ev_comp[i & 1])      # the inputs of step i-2 have been consumed
                    b["dY"].copy_(h_dY, non_blocking=True)
                    b["W"].copy_(h_W, non_blocking=True)
                    b["X"].copy_(h_X, non_blocking=True)
                    ev_in[i & 1].record(s_in)
                main.wait_event(ev_in[i & 1])
                if i >= 2:
                    main.wait_event(ev_out[i & 1])           # the outputs of step i-2 have left the device
                lbt.qconv_backward(desc, b["dY"], b["W"], b["X"], scales.data_ptr(), scales.data_ptr() + 4, st,
                                   b["stats"], q_dY, b["dX"], b["dW"], None, None, BITS_G, ws)
                ev_comp[i & 1].record(main)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_comp[i & 1])
                    h_dX.copy_(b["dX"], non_blocking=True)
                    h_dW.copy_(b["dW"], non_blocking=True)
                    h_stats.copy_(b["stats"], non_blocking=True)
                    ev_out[i & 1].record(s_out)
            main.wait_stream(s_in)
            main.wait_stream(s_out)

        pipe_steps = 2 * e2e_steps
        pipelined(2)
        barrier()
        e0.record()
        pipelined(pipe_steps)
        e1.record()
        barrier()
        ms_e2e_pipelined = dist_util.max_over_ranks(e0.elapsed_time(e1), "cuda") * e2e_steps / pipe_steps
        del bufs
    h2d = h_dY.numel() * 4 + h_W.numel() + h_X.numel()
    d2h = h_dX.numel() * 4 + h_dW.numel() * 4 + h_stats.numel()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- denominators.  The contraction's own dtype, measured here with a library GEMM; and 2 x the measured
    # bf16 figure (nominal dense int8 : bf16 ratio 4.5 : 2.25).  The region's regime picks burst or sustained.
    lib8 = None if args.no_int8_peak else library_int8_peak(torch, local)
    region_s = ms_total * 1e-3
    regime = "burst" if region_s < BURST_REGION_S else "sustained"

    def int8_peak(which):
        cands = {"2 x bf16 " + which + " (" + peaks["source"] + ")": 2.0 * peaks["bf16_" + which]}
        if lib8 and which + "_tops" in lib8:
            cands["library int8 GEMM " + which + " (measured in this run)"] = lib8[which + "_tops"]
        name = max(cands, key=cands.get)
        return cands[name], name, cands

    def gemm_roofline(pk, which, clk):
        gemm_ms = 0.5 * (pk["dgrad"] + pk["wgrad"])
        achieved = 2.0 * M * O * I / (gemm_ms * 1e-3) / 1e12
        peak, name, cands = int8_peak(which)
        mhz = clk.get("sm_mhz") if clk else None
        return {"achieved": achieved, "peak": peak, "frac": achieved / peak, "peak_source": name,
                "peak_candidates": cands, "gemm_ms": gemm_ms, "sm_mhz": mhz,
                "ms_x_mhz": gemm_ms * mhz if mhz else None,
                "frac_of_spec_4500": achieved / 4500.0,
                "frac_of_clock_peak": achieved / (148 * 16384 * mhz * 1e6 / 1e12) if mhz else None}

    value = world * args.steps * OPS_PER_STEP / (ms_total * 1e-3) / 1e12
    roof = gemm_roofline(per_kernel, regime, clocks)
    quant_ms = per_kernel["stats"] + per_kernel["quantize"]
    line = {
        "metric": METRIC, "value": value, "unit": "TOPS", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_total / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8 MMA on INT4 codes (int32 accumulate); fp32 quantizer",
        "data": "synthetic",
        "config": shared_config(world),
        "timing": {"kernel_taps": f"per-kernel CUDA events on {tapped} of the {args.steps} timed steps (every "
                                  f"{TAP_EVERY}th); the other steps run with the launches chained as a caller's would",
                   "regime": f"{regime}: the timed region lasts {region_s * 1e3:.0f} ms (burst below "
                             f"{BURST_REGION_S} s: the power cap has not pulled the SM clock down yet)"},
        "clocks": clocks,
        "e2e": {"value": world * e2e_steps * OPS_PER_STEP / (ms_e2e_pipelined * 1e-3) / 1e12 if e2e_steps else None,
                "unit": "TOPS",
                "how": "host buffers in pinned memory; per step 335.5 MB to the device and 536.9 MB back inside "
                       "the timed region; copy-in, compute and copy-out pipelined over three streams",
                "value_one_stream": world * e2e_steps * OPS_PER_STEP / (ms_e2e * 1e-3) / 1e12 if e2e_steps else None,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": KERNELS_PER_STEP * args.steps,
        "roofline": {"bound": "tensor", "kernel": "i8_gemm_pair_kernel (dgrad and wgrad launches averaged)",
                     "achieved": roof["achieved"], "peak": roof["peak"], "unit": "TOP/s", "frac": roof["frac"],
                     "regime": regime, "peak_source": roof["peak_source"] + "; the larger of the candidates",
                     "peak_candidates": roof["peak_candidates"],
                     "traffic": GEMM_DRAM_TRAFFIC if (M, O, I) == (8192, 8192, 8192) else None,
                     "traffic_note": "dram read+write bytes per launch: ncu capture of the 8192x4096x4096 case "
                                     "(133.1 MB dgrad, 123.0 MB wgrad) scaled by algorithmic operand + output bytes",
                     "gemm_ms": roof["gemm_ms"], "sm_mhz": roof["sm_mhz"], "ms_x_mhz": roof["ms_x_mhz"],
                     "frac_of_spec_4500": roof["frac_of_spec_4500"], "frac_of_clock_peak": roof["frac_of_clock_peak"],
                     "int8_measured": lib8},
        "kernels_ms": per_kernel,
        "quantizer": {"GBps_two_pass_8.5B_per_elem": 8.5 * N_GRAD / (quant_loop_ms * 1e-3) / 1e9,
                      "frac_of_hbm": 8.5 * N_GRAD / (quant_loop_ms * 1e-3) / 1e9 / peaks["hbm"],
                      "ms_per_pass": quant_loop_ms,
                      "what": "50 x (lbt_grad_stats, lbt_quantize_grad, lbt_update_interval) back to back on the "
                              "benchmark's dY, one event pair around the loop; 8.5 B per element = two fp32 reads + "
                              "the nibble-packed write",
                      "GBps_if_second_read_hit_L2_4.5B_per_elem": 4.5 * N_GRAD / (quant_loop_ms * 1e-3) / 1e9,
                      "warm_ms_median": _median(warm_ms), "cold_ms_median": _median(cold_ms),
                      "warm_cold_what": "20 runs each, one event pair per run (adds ~3 us): warm = back to back, as in "
                                        "training; cold = a 384 MiB buffer written before every run (L2 flushed)",
                      "frac_of_hbm_cold": 8.5 * N_GRAD / (_median(cold_ms) * 1e-3) / 1e9 / peaks["hbm"],
                      "in_fused_step": {"stats_ms": per_kernel["stats"], "quantize_ms": per_kernel["quantize"],
                                        "GBps_9.5B_per_elem": 9.5 * N_GRAD / (quant_ms * 1e-3) / 1e9,
                                        "frac_of_hbm": 9.5 * N_GRAD / (quant_ms * 1e-3) / 1e9 / peaks["hbm"],
                                        "what": "CUDA-event taps inside lbt_qconv_backward; there the quantize kernel "
                                                "also writes the int8 operand of the GEMMs (1 B per element more), "
                                                "which replaces the separate expansion pass over dY"},
                      "hbm_peak": peaks["hbm"], "peak_source": peaks["source"]},
        "gamma_after": state.gamma,
    }
    if sustained is not None:
        sroof = gemm_roofline(sustained["kernels_ms"], "sustained", sustained["clocks"])
        sustained["roofline"] = sroof
        sustained["ms_per_step_x_mhz"] = (sustained["ms_per_step"] * sustained["clocks"]["sm_mhz"]
                                          if sustained["clocks"] and sustained["clocks"].get("sm_mhz") else None)
        line["sustained"] = sustained
        line["ms_per_step_x_mhz"] = (ms_total / args.steps * clocks["sm_mhz"]
                                     if clocks and clocks.get("sm_mhz") else None)
    if world == 1 and not args.no_cpu_baseline:
        threads = os.cpu_count() or 1
        prep = OraclePrep(dY.cpu().numpy(), q_W.cpu().numpy(), q_X.cpu().numpy())
        v, d, _, details = oracle_sample(prep, 10.0, threads, full_quantizer=True, single_thread_seconds=4.0)
        line["cpu_baseline"] = {"value": v, "unit": "TOPS", "cores": threads, "kind": "oracle", "sample": d, **details}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_dp(args):
    """`--dp`: the same layer with its batch rows sharded over the ranks (exact data parallelism): every rank
    holds M rows of dY and X and all of W; g_max, the counters and the int32 weight-gradient accumulators are
    all-reduced (NCCL) inside the step, Philox runs on the element's index in the whole tensor.  Weak scaling: the
    global batch is world x M rows.  With one rank no collective runs and the outputs are checked against the
    fused call bit for bit."""
    import torch
    import torch.distributed as dist
    from paper_2407_12637_b200 import dist_util, dp, lbt, shapes, synth

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local)
    comm = None
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "WARN")      # NCCL's own log stays on
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        comm = dp.DistComm()
    lbt.lib()
    peaks = load_peaks()
    desc = lbt.ConvDesc(**shapes.linear(M, O, I))
    dY = synth.laplace_outliers_torch(N_GRAD, 1e-3, seed=rank)
    q_W = synth.code_bytes_torch(O * I // 2, 0, 1)          # the same weights on every rank
    q_X = synth.code_bytes_torch(M * I // 2, rank, 2)
    st = lbt.new_state(gamma=1.0, alpha=1e-3, beta=1e-3, bits=BITS_G, rounding=lbt.ROUND_STOCHASTIC, seed=0)
    stats = lbt.new_stats()
    scales = torch.tensor([0.01, 0.05], device="cuda")
    q_dY = torch.empty(N_GRAD // 2, dtype=torch.uint8, device="cuda")
    dX, dW = torch.empty(M, I, device="cuda"), torch.empty(O, I, device="cuda")
    accW = torch.empty(O, I, dtype=torch.int32, device="cuda")
    ws = torch.empty(lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, desc), dtype=torch.uint8, device="cuda")
    offset = dp.shard_offsets([N_GRAD] * world)[rank]

    def step():
        dp.sharded_backward(desc, dY, q_W, q_X, scales.data_ptr(), scales.data_ptr() + 4, st, stats, q_dY, dX, dW, accW,
                            BITS_G, ws, index_offset=offset, images_total=world * M, comm=comm)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    check = None
    if world == 1:
        # one rank: the sharded sequence must reproduce the fused call exactly
        st2 = st.clone(); stats2 = lbt.new_stats()
        q2, dX2, dW2 = torch.empty_like(q_dY), torch.empty_like(dX), torch.empty_like(dW)
        lbt.qconv_backward(desc, dY, q_W, q_X, scales.data_ptr(), scales.data_ptr() + 4, st2, stats2, q2, dX2, dW2,
                           None, None, BITS_G, ws)
        step()
        torch.cuda.synchronize()
        same = all(torch.equal(a, b) for a, b in ((q2, q_dY), (dX2, dX), (dW2, dW), (st2, st), (stats2, stats)))
        if not same:
            raise RuntimeError("--dp with one rank differs from lbt_qconv_backward")
        check = "one rank: codes, statistics, state, dX and dW bit-identical to lbt_qconv_backward"
        del q2, dX2, dW2
    for _ in range(max(args.warmup, 3)):
        step()
    sampler = ClockSampler(local) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    clocks = sampler.stop() if sampler else None
    ms_total = dist_util.max_over_ranks(e0.elapsed_time(e1), "cuda")
    # kernel-level taps on a few extra steps (outside the timed region)
    classes = {"dgrad": lbt.TIME_DGRAD, "wgrad": lbt.TIME_WGRAD}
    taps = {name: lbt.TimingTap(c) for name, c in classes.items()}
    gemm = {name: [] for name in classes}
    for _ in range(5):
        for t in taps.values():
            t.arm()
        step()
        torch.cuda.synchronize()
        for name, t in taps.items():
            gemm[name].append(t.ms())
    for t in taps.values():
        t.disarm()
    # end to end: the rank's inputs from pinned host memory, its dX, the layer's dW and the statistics back
    h_dY = torch.empty(N_GRAD, dtype=torch.float32).pin_memory(); h_dY.copy_(dY)
    h_W, h_X = q_W.cpu().pin_memory(), q_X.cpu().pin_memory()
    h_dX, h_dW = torch.empty(M, I).pin_memory(), torch.empty(O, I).pin_memory()
    h_stats = torch.empty(40, dtype=torch.uint8).pin_memory()
    e2e_steps = 0 if args.no_e2e else min(args.steps, 5)

    def e2e_step():
        dY.copy_(h_dY, non_blocking=True); q_W.copy_(h_W, non_blocking=True); q_X.copy_(h_X, non_blocking=True)
        step()
        h_dX.copy_(dX, non_blocking=True); h_dW.copy_(dW, non_blocking=True); h_stats.copy_(stats, non_blocking=True)

    ms_e2e = float("nan")
    if e2e_steps:
        e2e_step()
        barrier()
        e0.record()
        for _ in range(e2e_steps):
            e2e_step()
        e1.record()
        barrier()
        ms_e2e = dist_util.max_over_ranks(e0.elapsed_time(e1), "cuda")
    state = lbt.read_state(st)
    if state.dev_status != 0:
        raise RuntimeError("device status " + lbt.status_string(state.dev_status))
    if rank != 0:
        dist.destroy_process_group()
        return
    region_s = ms_total * 1e-3
    which = "burst" if region_s < BURST_REGION_S else "sustained"
    gemm_ms = 0.5 * (float(np.mean(gemm["dgrad"])) + float(np.mean(gemm["wgrad"])))
    achieved = 2.0 * M * O * I / (gemm_ms * 1e-3) / 1e12
    peak = 2.0 * peaks["bf16_" + which]
    line = {
        "metric": METRIC, "value": world * args.steps * OPS_PER_STEP / (ms_total * 1e-3) / 1e12, "unit": "TOPS",
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int8 MMA on INT4 codes (int32 accumulate); fp32 quantizer", "data": "synthetic",
        "config": {"workload": workload_name() + f", batch rows sharded: {M} rows per rank, {world * M} in all",
                   "l2": "inputs larger than L2",
                   "parallelism": f"dp{world}: all-reduce MAX of g_max (4 B), SUM of the counters (24 B + 8 B) and SUM of "
                                  f"the int32 weight-gradient accumulators ({4 * O * I} B) per step over NCCL",
                   "dp_check": check},
        "clocks": clocks,
        "e2e": {"value": world * e2e_steps * OPS_PER_STEP / (ms_e2e * 1e-3) / 1e12 if e2e_steps else None, "unit": "TOPS",
                "h2d_bytes_per_step": h_dY.numel() * 4 + h_W.numel() + h_X.numel(),
                "d2h_bytes_per_step": h_dX.numel() * 4 + h_dW.numel() * 4 + h_stats.numel(), "steps": e2e_steps},
        "gpu_launches": (8 if world > 1 else 7) * args.steps,
        "roofline": {"bound": "tensor", "kernel": "i8_gemm_pair_kernel (dgrad and wgrad launches averaged, 5 tapped steps "
                                                  "after the timed region)",
                     "achieved": achieved, "peak": peak, "unit": "TOP/s", "frac": achieved / peak,
                     "peak_source": f"2 x bf16 {which} ({peaks['source']})", "traffic": None,
                     "frac_of_spec_4500": achieved / 4500.0},
        "gamma_after": state.gamma,
    }
    if world == 1 and not args.no_cpu_baseline:
        threads = os.cpu_count() or 1
        prep = OraclePrep(dY.cpu().numpy(), q_W.cpu().numpy(), q_X.cpu().numpy())
        v, d, _, details = oracle_sample(prep, 10.0, threads)
        line["cpu_baseline"] = {"value": v, "unit": "TOPS", "cores": threads, "kind": "oracle", "sample": d, **details}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiler captures)")
    ap.add_argument("--no-sustained", action="store_true", help="skip the seconds-long back-to-back leg")
    ap.add_argument("--no-int8-peak", action="store_true", help="skip the library int8 GEMM used as a denominator")
    ap.add_argument("--shape", default=None, help="M,O,I of another linear layer (profiler captures)")
    ap.add_argument("--dp", action="store_true",
                    help="shard the batch rows over the ranks (exact data parallelism with NCCL all-reduces) "
                         "instead of running independent replicas")
    args = ap.parse_args()
    if args.shape:
        set_shape(*[int(v) for v in args.shape.split(",")])
    if args.impl == "reference":
        run_reference(args)
    elif args.dp:
        run_dp(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
