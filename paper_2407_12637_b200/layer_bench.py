"""Per-layer-shape timing of the hot path: `python -m paper_2407_12637_b200.layer_bench [--config N]`.

For every layer shape of the benchmark configurations it runs the fused call `lbt_qconv_backward`
(statistics, quantize, interval update, expansion, dgrad, wgrad) and prints one markdown row with the
CUDA-event duration of each kernel class (median over the timed repetitions), the contractions as
TOPS = 2 * MAC / t and the statistics + quantize pair as GB/s at 8.5 (b <= 4) or 9 bytes per element
(one more byte where the quantizer also writes the int8 operand: linear and 1x1 stride-1 layers).
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

from . import lbt, shapes, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return p["hbm_gbs"], 2.0 * p["bf16_tflops"], "measured"
    return 6650.0, 2.0 * 1590.0, "fallback"


def time_layer(shape, bits=4, reps=20, warmup=5, seed=0):
    desc = lbt.ConvDesc(**shape)
    n = shapes.grad_elems(shape)
    dY = synth.laplace_outliers_torch(n, 1e-3, seed)
    q_W = synth.code_bytes_torch((shape["K"] * shape["R"] * shape["S"] * shape["C"] + 1) // 2, seed, 1)
    q_X = synth.code_bytes_torch((shape["N"] * shape["H"] * shape["W"] * shape["C"] + 1) // 2, seed, 2)
    st = lbt.new_state(gamma=0.8, bits=bits, rounding=lbt.ROUND_STOCHASTIC, seed=seed, beta=0.0)
    stats = lbt.new_stats()
    sc = torch.tensor([0.01, 0.05], device="cuda")
    q_dY = torch.empty((n + 1) // 2 if bits <= 4 else n, dtype=torch.uint8, device="cuda")
    dX = torch.empty(shape["N"] * shape["H"] * shape["W"] * shape["C"], device="cuda")
    dW = torch.empty(shape["K"] * shape["R"] * shape["S"] * shape["C"], device="cuda")
    ws = torch.empty(lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, desc), dtype=torch.uint8, device="cuda")
    classes = {"stats": lbt.TIME_STATS, "quantize": lbt.TIME_QUANTIZE, "expand": lbt.TIME_EXPAND,
               "dgrad": lbt.TIME_DGRAD, "wgrad": lbt.TIME_WGRAD}
    taps = {k: lbt.TimingTap(c) for k, c in classes.items()}
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    samples = {k: [] for k in classes}
    total = []
    for it in range(warmup + reps):
        for t in taps.values():
            t.arm()
        lbt.qconv_backward(desc, dY, q_W, q_X, sc.data_ptr(), sc.data_ptr() + 4, st, stats, q_dY, dX, dW,
                           None, None, bits, ws)
        torch.cuda.synchronize()
        if it >= warmup:
            for k, t in taps.items():
                samples[k].append(t.ms())
    for t in taps.values():
        t.disarm()
        t.close()
    # the whole call, timed without the per-class taps (each armed tap adds two event records to the stream)
    for it in range(warmup + reps):
        e0.record()
        lbt.qconv_backward(desc, dY, q_W, q_X, sc.data_ptr(), sc.data_ptr() + 4, st, stats, q_dY, dX, dW,
                           None, None, bits, ws)
        e1.record()
        torch.cuda.synchronize()
        if it >= warmup:
            total.append(e0.elapsed_time(e1))
    if lbt.read_state(st).dev_status != 0:
        raise RuntimeError("device status " + lbt.status_string(lbt.read_state(st).dev_status))
    out = {k: float(np.median(v)) for k, v in samples.items()}
    out["total"] = float(np.median(total))
    return out


def time_chain(shape, bits=4, reps=20, warmup=5, seed=0):
    """`lbt_qconv_backward_ex` on one layer, three ways: as lbt_qconv_backward runs it; with the statistics of
    dY already in place (dy_stats_ready: no abs-max pass); and with the statistics of dX taken in the dgrad
    epilogue (dx_stats).  Median CUDA-event durations per kernel class (ms)."""
    desc = lbt.ConvDesc(**shape)
    n = shapes.grad_elems(shape)
    dY = synth.laplace_outliers_torch(n, 1e-3, seed)
    q_W = synth.code_bytes_torch((shape["K"] * shape["R"] * shape["S"] * shape["C"] + 1) // 2, seed, 1)
    q_X = synth.code_bytes_torch((shape["N"] * shape["H"] * shape["W"] * shape["C"] + 1) // 2, seed, 2)
    st = lbt.new_state(gamma=0.8, bits=bits, rounding=lbt.ROUND_STOCHASTIC, seed=seed, beta=0.0)
    stats, dx_stats = lbt.new_stats(), lbt.new_stats()
    sc = torch.tensor([0.01, 0.05], device="cuda")
    q_dY = torch.empty((n + 1) // 2 if bits <= 4 else n, dtype=torch.uint8, device="cuda")
    dX = torch.empty(shape["N"] * shape["H"] * shape["W"] * shape["C"], device="cuda")
    dW = torch.empty(shape["K"] * shape["R"] * shape["S"] * shape["C"], device="cuda")
    ws = torch.empty(lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, desc), dtype=torch.uint8, device="cuda")
    classes = {"stats": lbt.TIME_STATS, "quantize": lbt.TIME_QUANTIZE, "dgrad": lbt.TIME_DGRAD}
    taps = {k: lbt.TimingTap(c) for k, c in classes.items()}
    out = {}
    for mode, (ready, want_dx) in {"plain": (False, False), "ready": (True, False), "dx_stats": (False, True)}.items():
        samples = {k: [] for k in classes}
        for it in range(warmup + reps):
            for t in taps.values():
                t.arm()
            lbt.qconv_backward_ex(desc, dY, q_W, q_X, sc.data_ptr(), sc.data_ptr() + 4, st, stats, q_dY, dX, dW,
                                  None, None, bits, ws, dy_stats_ready=ready, dx_stats=dx_stats if want_dx else None)
            torch.cuda.synchronize()
            if it >= warmup:
                for k, t in taps.items():
                    samples[k].append(t.ms())
        out[mode] = {k: float(np.median(v)) for k, v in samples.items()}
    for t in taps.values():
        t.disarm()
        t.close()
    if lbt.read_state(st).dev_status != 0:
        raise RuntimeError("device status " + lbt.status_string(lbt.read_state(st).dev_status))
    return out


def time_forward(shape, bits=4, reps=20, warmup=5, seed=0):
    """The forward side of one layer: activation and weight quantizers (one pass each, 4 bytes read
    and 0.5 or 1 byte written per element) and the integer forward product, each as the median
    CUDA-event duration of its kernel class over `reps` repetitions (ms)."""
    desc = lbt.ConvDesc(**shape)
    nx = shape["N"] * shape["H"] * shape["W"] * shape["C"]
    nw = shape["K"] * shape["R"] * shape["S"] * shape["C"]
    ny = shapes.grad_elems(shape)
    x = synth.laplace_outliers_torch(nx, 0.5, seed).abs_()
    w = synth.laplace_outliers_torch(nw, 0.05, seed + 1)
    io = torch.tensor([1.7, 0.16, 0.0, 0.0], device="cuda")          # c_x, c_w, s_x, s_w
    q_X = torch.empty((nx + 1) // 2 if bits <= 4 else nx, dtype=torch.uint8, device="cuda")
    q_W = torch.empty((nw + 1) // 2 if bits <= 4 else nw, dtype=torch.uint8, device="cuda")
    Y = torch.empty(ny, device="cuda")
    ws = torch.empty(lbt.workspace_bytes(lbt.OP_CONV_FORWARD, desc), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    taps = {k: lbt.TimingTap(c) for k, c in (("quant", lbt.TIME_FWD_QUANT), ("expand", lbt.TIME_EXPAND),
                                             ("forward", lbt.TIME_FORWARD))}
    samples = {"quant_x": [], "quant_w": [], "expand": [], "forward": []}
    for it in range(warmup + reps):
        for t in taps.values():
            t.arm()
        lbt.quantize_act(x, io.data_ptr(), bits, q_X, io.data_ptr() + 8)
        torch.cuda.synchronize()
        tx = taps["quant"].ms()
        lbt.quantize_weight(w, io.data_ptr() + 4, bits, q_W, io.data_ptr() + 12)
        lbt.qconv_forward(desc, q_X, q_W, io.data_ptr() + 8, io.data_ptr() + 12, Y, None, bits, bits, ws, status)
        torch.cuda.synchronize()
        if it >= warmup:
            samples["quant_x"].append(tx)
            samples["quant_w"].append(taps["quant"].ms())
            samples["expand"].append(taps["expand"].ms())
            samples["forward"].append(taps["forward"].ms())
    for t in taps.values():
        t.disarm()
        t.close()
    if int(status.item()) != 0:
        raise RuntimeError("device status " + lbt.status_string(int(status.item())))
    return {k: float(np.median(v)) for k, v in samples.items()}


def bound_us(shape, which, hbm_gbs):
    """Lower bound on one contraction's time in us: the slower of its integer ops at the 4.5 POPS spec
    and its unavoidable HBM traffic (fp32 output written once, int8 operands read once) at the measured
    copy bandwidth.  Small-channel and 1x1 layers are bound by the fp32 output, not by the tensor pipe."""
    d = lbt.ConvDesc(**shape)
    ny, nx = shapes.grad_elems(shape), shape["N"] * shape["H"] * shape["W"] * shape["C"]
    nw = shape["K"] * shape["R"] * shape["S"] * shape["C"]
    out, a, b = {"dgrad": (nx, ny, nw), "wgrad": (nw, ny, nx), "forward": (ny, nx, nw)}[which]
    return max(2.0 * shapes.macs(shape) / 4.5e15, (4.0 * out + a + b) / (hbm_gbs * 1e9)) * 1e6


_ONLY_LAYER = None   # --layer: restrict every table to the layer of this name


def rows_for(config: int):
    table = {0: shapes.CONFIG0, 1: shapes.CONFIG1, 2: shapes.CONFIG2,
             3: {k: v[0] for k, v in shapes.CONFIG3.items()}, 4: shapes.CONFIG4}[config]
    return [(k, v) for k, v in table.items() if _ONLY_LAYER in (None, k)]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=None, help="0..4; default: all")
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--forward", action="store_true", help="time the forward side (quantizers + forward product)")
    ap.add_argument("--chain", action="store_true",
                    help="time lbt_qconv_backward_ex: abs-max pass skipped (statistics ready) and dX statistics in the epilogue")
    ap.add_argument("--layer", default=None, help="only the layer of this name (profiler captures)")
    args = ap.parse_args()
    global _ONLY_LAYER
    _ONLY_LAYER = args.layer
    hbm, int8_peak, src = _peaks()
    print(f"peaks ({src}): HBM {hbm:.0f} GB/s, INT8 tensor 2 x bf16 burst = {int8_peak:.0f} TOPS; public spec 8000 GB/s, 4500 TOPS")
    if args.chain:
        print("| config | layer | grad elems | abs-max + quantize us (two looks) | GB/s at 8.5 (9.5) B | quantize us with "
              "statistics ready (one look) | GB/s at 4.5 (5.5) B | saved us | dgrad us | dgrad us with dX statistics |")
        print("|---|---|---|---|---|---|---|---|---|---|")
        for cfg in ([args.config] if args.config is not None else [2, 3, 4]):
            for name, shape in rows_for(cfg):
                t = time_chain(shape, bits=args.bits, reps=args.reps)
                n = shapes.grad_elems(shape)
                extra = 1.0 if (args.bits <= 4 and shape["R"] == shape["S"] == 1 and shape["stride"] == 1
                                and shape["pad"] == 0 and shape["K"] % 16 == 0) else 0.0
                two = t["plain"]["stats"] + t["plain"]["quantize"]
                one = t["ready"]["quantize"]
                print(f"| {cfg} | {name} | {n} | {two * 1e3:.1f} | {(8.5 + extra) * n / (two * 1e-3) / 1e9:.0f} | "
                      f"{one * 1e3:.1f} | {(4.5 + extra) * n / (one * 1e-3) / 1e9:.0f} | {(two - one) * 1e3:.1f} | "
                      f"{t['plain']['dgrad'] * 1e3:.1f} | {t['dx_stats']['dgrad'] * 1e3:.1f} |", flush=True)
        return
    if args.forward:
        print("| config | layer | X elems | W elems | GMAC | act quant us | GB/s (% HBM) | weight quant us | GB/s | "
              "expand us | forward us | forward TOPS (% meas / % spec) | bound us | % of bound |")
        print("|---|---|---|---|---|---|---|---|---|---|---|---|---|---|")
        bpe = 4.5 if args.bits <= 4 else 5.0
        for cfg in ([args.config] if args.config is not None else [0, 1, 2, 3, 4]):
            for name, shape in rows_for(cfg):
                t = time_forward(shape, bits=args.bits, reps=args.reps)
                nx = shape["N"] * shape["H"] * shape["W"] * shape["C"]
                nw = shape["K"] * shape["R"] * shape["S"] * shape["C"]
                mac = shapes.macs(shape)
                gx, gw = bpe * nx / (t["quant_x"] * 1e-3) / 1e9, bpe * nw / (t["quant_w"] * 1e-3) / 1e9
                tf = 2.0 * mac / (t["forward"] * 1e-3) / 1e12
                print(f"| {cfg} | {name} | {nx} | {nw} | {mac / 1e9:.3f} | {t['quant_x'] * 1e3:.1f} | "
                      f"{gx:.0f} ({100 * gx / hbm:.0f} %) | {t['quant_w'] * 1e3:.1f} | {gw:.0f} | "
                      f"{t['expand'] * 1e3:.1f} | {t['forward'] * 1e3:.1f} | "
                      f"{tf:.0f} ({100 * tf / int8_peak:.0f} % / {100 * tf / 4500:.0f} %) | "
                      f"{bound_us(shape, 'forward', hbm):.1f} | "
                      f"{100 * bound_us(shape, 'forward', hbm) / (t['forward'] * 1e3):.0f} % |", flush=True)
        return
    print("| config | layer | grad elems | GMAC | stats us | quant us | quantizer GB/s (% HBM) | expand us | "
          "dgrad us | dgrad TOPS (% meas / % spec) | wgrad us | wgrad TOPS (% meas / % spec) | step us | "
          "bound us dgrad / wgrad | % of bound |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|")
    for cfg in ([args.config] if args.config is not None else [0, 1, 2, 3, 4]):
        for name, shape in rows_for(cfg):
            t = time_layer(shape, bits=args.bits, reps=args.reps)
            n, mac = shapes.grad_elems(shape), shapes.macs(shape)
            bpe = 8.5 if args.bits <= 4 else 9.0
            if args.bits <= 4 and shape["R"] == shape["S"] == 1 and shape["stride"] == 1 and shape["pad"] == 0 \
                    and shape["K"] % 16 == 0:
                bpe += 1.0   # unpadded layouts: the quantizer also writes the int8 operand of the contractions
            qg = bpe * n / ((t["stats"] + t["quantize"]) * 1e-3) / 1e9
            td, tw = 2.0 * mac / (t["dgrad"] * 1e-3) / 1e12, 2.0 * mac / (t["wgrad"] * 1e-3) / 1e12
            print(f"| {cfg} | {name} | {n} | {mac / 1e9:.3f} | {t['stats'] * 1e3:.1f} | {t['quantize'] * 1e3:.1f} | "
                  f"{qg:.0f} ({100 * qg / hbm:.0f} %) | {t['expand'] * 1e3:.1f} | {t['dgrad'] * 1e3:.1f} | "
                  f"{td:.0f} ({100 * td / int8_peak:.0f} % / {100 * td / 4500:.0f} %) | {t['wgrad'] * 1e3:.1f} | "
                  f"{tw:.0f} ({100 * tw / int8_peak:.0f} % / {100 * tw / 4500:.0f} %) | {t['total'] * 1e3:.1f} | "
                  f"{bound_us(shape, 'dgrad', hbm):.1f} / {bound_us(shape, 'wgrad', hbm):.1f} | "
                  f"{100 * bound_us(shape, 'dgrad', hbm) / (t['dgrad'] * 1e3):.0f} % / "
                  f"{100 * bound_us(shape, 'wgrad', hbm) / (t['wgrad'] * 1e3):.0f} % |", flush=True)


if __name__ == "__main__":
    main()
