"""Pins for oracle/search.py (the per-module mode search of Sec. 2.3).  The search is a definition built from the layer
forward, so the pins are structural: the all-FP mode has error exactly 0, every figure equals an independent evaluation
of that mode, every greedy step releases the argmin of the candidates recomputed here with a plain loop, and the walk
ends at the first mode within budget (or at all-FP)."""
import dataclasses

import numpy as np

from oracle import layer as L
from oracle import ops as O
from oracle import search as S
from paper_2310_17723_b200 import workloads as W


def _setup(seed=61):
    shape = W.tiny_shape(B=1, S=64, H=128, nh=2, F=256, eps=1e-5, n_outlier=2)
    spec = L.LayerSpec(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, eps=shape.eps)
    p = W.layer_params(shape, seed)
    x = O.layernorm(W.activations(shape, seed).astype(np.float64), p["ln0_g"], p["ln0_b"], shape.eps)
    x = np.asarray(O.fp_tensor(x, "f16").data)
    return spec, p, L.calibrate(spec, p, x, shape.B), x


def _independent_error(spec, p, C, x, mode):
    """The same figure without oracle/search.py: both layers prepared and run here."""
    def out(m):
        s = dataclasses.replace(spec, mode=dict(m), gran_in="fwq", gran_out="fp")
        Lp = L.prepare_layer(s, p, C)
        t = O.fp_tensor(x, "f16")
        if m["qkv"] == "int8":
            t = O.emit(t.real(), O.OutSpec("fwq", scale=C["S_in_f"]))
        return L.layer_forward(Lp, t)["x_out"].real()
    ref = out(L.MODE_PRESETS["FP"])
    return float(np.max(np.abs(out(mode) - ref)) / np.max(np.abs(ref)))


def test_all_fp_mode_has_zero_error_and_presets_are_ordered_sanely():
    spec, p, C, x = _setup()
    assert S.layer_error(spec, p, C, x, L.MODE_PRESETS["FP"]) == 0.0
    e = {k: S.layer_error(spec, p, C, x, L.MODE_PRESETS[k]) for k in ("M1", "M2", "M3")}
    for k, v in e.items():
        assert 0.0 < v < 0.2, (k, v)                                  # a few percent, never orders of magnitude
        assert v == _independent_error(spec, p, C, x, L.MODE_PRESETS[k])


def test_sensitivity_table_entries_are_the_errors_of_the_modes_they_name():
    spec, p, C, x = _setup(62)
    t = S.sensitivity(spec, p, C, x)
    assert set(t) == set(L.MODULES) | {"all_int8"}
    assert t["all_int8"] == _independent_error(spec, p, C, x, L.MODE_PRESETS["M3"])
    for m in ("qkv", "fc2"):
        alone = {k: ("int8" if k == m else "fp") for k in L.MODULES}
        without = {k: ("fp" if k == m else "int8") for k in L.MODULES}
        assert t[m]["alone"] == _independent_error(spec, p, C, x, alone)
        assert t[m]["without"] == _independent_error(spec, p, C, x, without)
        assert t[m]["alone"] > 0.0


def test_greedy_search_releases_the_argmin_and_stops_at_the_budget():
    spec, p, C, x = _setup(63)
    m3 = S.layer_error(spec, p, C, x, L.MODE_PRESETS["M3"])
    mode, trace = S.search(spec, p, C, x, budget=m3 * 1.01)           # already within budget: nothing is released
    assert mode == L.MODE_PRESETS["M3"] and len(trace) == 1 and trace[0][1] == m3 and not trace[0][2]
    mode, trace = S.search(spec, p, C, x, budget=0.0)                 # nothing but all-FP has error 0
    assert all(v == "fp" for v in mode.values()) and trace[-1][1] == 0.0 and len(trace) == 6
    for (m_a, e_a, cands), (m_b, e_b, _) in zip(trace, trace[1:]):
        released = [k for k in L.MODULES if m_a[k] != m_b[k]]
        assert len(released) == 1 and m_a[released[0]] == "int8" and m_b[released[0]] == "fp"
        assert set(cands) == {k for k in L.MODULES if m_a[k] == "int8"}
        assert e_b == min(cands.values()) == cands[released[0]]
    # one step recomputed without the module: the candidates of the first step
    first = trace[0][2]
    for m in ("attn", "fc1"):
        c = dict(L.MODE_PRESETS["M3"])
        c[m] = "fp"
        assert first[m] == _independent_error(spec, p, C, x, c)
    # a budget between two trace errors stops exactly at the first mode that meets it
    errs = [e for _, e, _ in trace]
    k = next(i for i in range(1, len(errs)) if errs[i] < errs[i - 1])
    mid = 0.5 * (errs[k] + errs[k - 1])
    mode_mid, trace_mid = S.search(spec, p, C, x, budget=mid)
    assert trace_mid[-1][1] <= mid and all(e > mid for _, e, _ in trace_mid[:-1])
    assert [m for m, _, _ in trace_mid] == [m for m, _, _ in trace[:len(trace_mid)]]
