"""Mixed-precision mode search (Sec. 2.3: Table 1's M1, M2, M3 are three points of a per-module INT8 / FP choice,
"other mixed-precision modes" are left to the user) in fp64 (oracle; test infrastructure only).

Plain loops over `layer.prepare_layer` / `layer.layer_forward`:

  layer_error   relative max-norm distance of the layer output in a given mode from the all-FP layer's output on the
                same input
  sensitivity   per module: that error with only this module in INT8 ('alone') and with every other module in INT8
                ('without'); plus the all-INT8 error
  search        greedy walk from all-INT8 (M3) towards FP: while the error exceeds the budget, the module whose release
                lowers the error most goes back to FP

The layer input is the FP tensor itself; where the QKV module is INT8 it is quantized feature-wise with the calibrated
input scale (Eq. 4), the role the previous layer's LN^quant plays in a stack.  The layer output is taken in FP.
"""
import dataclasses

import numpy as np

from . import layer as L
from . import ops as O


def _output(spec, params, C, x_fp, mode):
    s = dataclasses.replace(spec, mode=dict(mode), gran_in="fwq", gran_out="fp")
    Lp = L.prepare_layer(s, params, C)
    x = O.fp_tensor(x_fp, s.fp_dtype)
    if s.arch == "post_ln" and s.mode["qkv"] == "int8":
        x = O.emit(x.real(), O.OutSpec("fwq", scale=C["S_in_f"]))
    return L.layer_forward(Lp, x)["x_out"].real()


def _rel(a, ref):
    return float(np.max(np.abs(a - ref)) / np.max(np.abs(ref)))


def layer_error(spec, params, C, x_fp, mode, ref=None):
    if ref is None:
        ref = _output(spec, params, C, x_fp, L.MODE_PRESETS["FP"])
    return _rel(_output(spec, params, C, x_fp, mode), ref)


def sensitivity(spec, params, C, x_fp):
    ref = _output(spec, params, C, x_fp, L.MODE_PRESETS["FP"])
    table = {}
    for m in L.MODULES:
        alone = {k: ("int8" if k == m else "fp") for k in L.MODULES}
        without = {k: ("fp" if k == m else "int8") for k in L.MODULES}
        table[m] = {"alone": layer_error(spec, params, C, x_fp, alone, ref),
                    "without": layer_error(spec, params, C, x_fp, without, ref)}
    table["all_int8"] = layer_error(spec, params, C, x_fp, L.MODE_PRESETS["M3"], ref)
    return table


def search(spec, params, C, x_fp, budget):
    """Returns (mode, trace): trace = [(mode, error, candidates)], candidates = {released module: error} examined at the
    step that led to the NEXT entry (empty for the last one)."""
    ref = _output(spec, params, C, x_fp, L.MODE_PRESETS["FP"])
    mode = dict(L.MODE_PRESETS["M3"])
    err = layer_error(spec, params, C, x_fp, mode, ref)
    trace = []
    while True:
        cands = {}
        if err > budget and any(v == "int8" for v in mode.values()):
            for m in L.MODULES:
                if mode[m] == "int8":
                    c = dict(mode)
                    c[m] = "fp"
                    cands[m] = layer_error(spec, params, C, x_fp, c, ref)
        trace.append((dict(mode), err, cands))
        if not cands:
            return mode, trace
        best = min(cands, key=lambda k: (cands[k], L.MODULES.index(k)))     # ties: the earlier module of Table 1
        mode[best] = "fp"
        err = cands[best]
