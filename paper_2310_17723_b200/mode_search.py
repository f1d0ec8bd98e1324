"""Mixed-precision mode search (Sec. 2.3, Table 1: M1, M2, M3 are three points of a per-module INT8 / FP choice) and
percentile clipping of static scales (the truncation threshold the paper leaves un-tuned).

Everything runs on the device through the library's operators: the all-FP layer is the reference, a candidate mode is
one hero_layer_forward of the layer prepared for that mode, and its cost is the relative error of the layer output on
the calibration batch.

    sensitivity(...)  error of the layer with exactly one module in INT8, and with all but one module in INT8
    search(...)       greedy walk from all-INT8 (M3) towards FP: while the error exceeds the budget, give the module
                      whose release helps most back to FP; returns the mode and the trace
    percentile_scale(...)  static scale from the q-th percentile of |x| (histogram observer), not from absmax
"""
import dataclasses

import numpy as np
import torch

from . import hero, prep
from .layer import Layer

MODULES = prep.MODULES


def _run(h, cfg, params, C, x_in):
    """One forward of the layer prepared for cfg.mode on x_in (FP tensor [M, H] on the device); returns FP32 output."""
    # an FP input feeds an INT8 QKV through an entry quantization that belongs to the previous layer: for the search
    # the layer input is the FP tensor itself, quantized here by the calibrated static scale of the input
    fpt = hero.TORCH_FP[cfg.fp_dtype]
    c = dataclasses.replace(cfg, gran_in="fwq", gran_out="fp")
    L = prep.prepare_layer(c, params, C)
    layer = Layer(h, L)
    M, H = x_in.shape
    out = torch.empty(M, H, dtype=fpt, device="cuda")
    if c.arch == "post_ln" and c.mode["qkv"] == "int8":
        s_in = torch.from_numpy(np.asarray(C["S_in_f"], np.float32)).cuda()
        xq = torch.clamp(torch.round(x_in.float() / s_in[None, :]), -127, 127).to(torch.int8)
        layer.forward(hero.tensor(xq, "fwq", s_in), hero.tensor(out))
    else:
        layer.forward(hero.tensor(x_in), hero.tensor(out))
    h.check()
    return out.float()


def _err(a, ref):
    return float((a - ref).abs().max() / ref.abs().max())


def layer_error(h, cfg, params, C, x_in, mode, ref=None):
    """Relative max-norm error of the layer output in `mode` against the all-FP layer on the same input."""
    if ref is None:
        ref = _run(h, dataclasses.replace(cfg, mode=dict(prep.PRESETS["FP"])), params, C, x_in)
    return _err(_run(h, dataclasses.replace(cfg, mode=dict(mode)), params, C, x_in), ref)


def sensitivity(h, cfg, params, C, x_in):
    """Per module: error with only that module in INT8 ('alone') and with every other module in INT8 ('without')."""
    ref = _run(h, dataclasses.replace(cfg, mode=dict(prep.PRESETS["FP"])), params, C, x_in)
    table = {}
    for m in MODULES:
        alone = {k: ("int8" if k == m else "fp") for k in MODULES}
        without = {k: ("fp" if k == m else "int8") for k in MODULES}
        table[m] = {"alone": layer_error(h, cfg, params, C, x_in, alone, ref),
                    "without": layer_error(h, cfg, params, C, x_in, without, ref)}
    table["all_int8"] = layer_error(h, cfg, params, C, x_in, prep.PRESETS["M3"], ref)
    return table


def search(h, cfg, params, C, x_in, budget):
    """Greedy mode search: the most aggressive mode found whose error stays within `budget`.  Returns (mode, trace)."""
    ref = _run(h, dataclasses.replace(cfg, mode=dict(prep.PRESETS["FP"])), params, C, x_in)
    mode = dict(prep.PRESETS["M3"])
    err = layer_error(h, cfg, params, C, x_in, mode, ref)
    trace = [(dict(mode), err)]
    while err > budget and any(v == "int8" for v in mode.values()):
        best = None
        for m in MODULES:
            if mode[m] != "int8":
                continue
            cand = dict(mode)
            cand[m] = "fp"
            e = layer_error(h, cfg, params, C, x_in, cand, ref)
            if best is None or e < best[1]:
                best = (cand, e)
        mode, err = best
        trace.append((dict(mode), err))
    return mode, trace


def percentile_scale(h, x, q, qmax=127.0):
    """Static scale from the q-th percentile (0 < q <= 1) of |x| over the tensor x (FP, on the device): the clipping
    threshold is the upper edge of the first histogram bin at which the cumulative count reaches q of the total.
    q = 1 reproduces absmax / qmax up to one bin width."""
    amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    h.hero_absmax_observe(hero.tensor(x), None, amax)
    bound = float(amax.item())
    if bound <= 0.0:
        return 1.0
    hist = torch.zeros(hero.HIST_BINS, dtype=torch.int64, device="cuda")
    h.hero_abs_histogram(hero.tensor(x), bound, hist)
    h.check()
    cum = np.cumsum(hist.cpu().numpy().astype(np.float64))
    k = int(np.searchsorted(cum, q * cum[-1] - 0.5))
    thr = bound * (min(k, hero.HIST_BINS - 1) + 1) / hero.HIST_BINS
    return float(np.float32(thr / qmax))
