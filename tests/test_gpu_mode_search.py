"""Mode search and percentile clipping (Sec. 2.3 / Sec. 3) on the device."""
import numpy as np
import pytest
import torch

from oracle import ops as O
from paper_2310_17723_b200 import hero, prep, mode_search as MS, workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture
def h():
    hd = hero.Handle()
    yield hd
    hd.check()
    hd.close()


def test_abs_histogram_matches_numpy_and_percentile_scale(h):
    g = np.random.default_rng(3)
    x = torch.from_numpy(g.standard_normal((777, 1024)).astype(np.float32)).to(torch.float16).cuda()
    x[5, 7] = 40.0                                                 # one outlier far beyond the bulk
    ref = np.abs(x.float().cpu().numpy().astype(np.float64))
    bound = float(ref.max())
    hist = torch.zeros(hero.HIST_BINS, dtype=torch.int64, device="cuda")
    h.hero_abs_histogram(hero.tensor(x), bound, hist)
    h.check()
    # the plain definition in fp64: bin = floor(|x| / bound * bins), the last bin closed
    idx = np.minimum(hero.HIST_BINS - 1, np.floor(ref / bound * hero.HIST_BINS).astype(np.int64))
    want = np.bincount(idx.ravel(), minlength=hero.HIST_BINS)
    got = hist.cpu().numpy()
    assert got.sum() == ref.size
    # fp32 arithmetic on the device may put a value that sits within rounding of a bin edge into the neighbouring
    # bin: the cumulative counts may differ by the few values that do
    assert np.abs(np.cumsum(got) - np.cumsum(want)).max() <= 2
    # accumulation over a second call
    h.hero_abs_histogram(hero.tensor(x), bound, hist)
    assert hist.sum().item() == 2 * ref.size
    # q = 1 gives absmax / 127 within one bin; q = 0.9999 cuts the outlier off
    s1 = MS.percentile_scale(h, x, 1.0)
    assert abs(s1 - bound / 127) <= bound / hero.HIST_BINS / 127 * 1.01
    s2 = MS.percentile_scale(h, x, 0.9999)
    q = np.quantile(ref, 0.9999)
    assert q / 127 <= s2 <= (q + 2 * bound / hero.HIST_BINS) / 127 and s2 < 0.2 * s1


def test_sensitivity_and_search_match_the_oracle(h):
    """The device's per-module sensitivity table and greedy walk against the oracle's (oracle/search.py: the same
    definitions as plain loops over its own fp64 layer, with its own calibration and folding).  Both sides measure
    distances of a few percent between layer outputs; the FP16 / BF16 storage of the device's reference layer and the
    rounding ties of the INT8 tensors move them by a few 1e-3, so the figures are compared with an absolute allowance
    of 4e-3 plus 15 %, and the order in which the walk releases modules must agree wherever the oracle's own candidates
    at that step are further apart than that allowance."""
    from oracle import layer as OL, search as OS
    from gpu_util import report
    shape = W.tiny_shape(B=2, S=128, H=256, nh=4, F=512, eps=1e-5, n_outlier=2)
    cfg = prep.LayerConfig(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, eps=shape.eps)
    spec = OL.LayerSpec(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, eps=shape.eps)
    p = W.layer_params(shape, 61)
    x = W.activations(shape, 61)
    cal = np.asarray(O.fp_tensor(O.layernorm(x.astype(np.float64), p["ln0_g"], p["ln0_b"], shape.eps), "f16").data)
    C_dev = prep.calibrate(cfg, p, cal, shape.B)
    C_orc = OL.calibrate(spec, p, cal, shape.B)
    x_in = torch.from_numpy(cal).to(torch.float16).cuda()
    close = lambda a, b: abs(a - b) <= 4e-3 + 0.15 * abs(b)
    t_dev = MS.sensitivity(h, cfg, p, C_dev, x_in)
    t_orc = OS.sensitivity(spec, p, C_orc, cal)
    assert close(t_dev["all_int8"], t_orc["all_int8"]), (t_dev["all_int8"], t_orc["all_int8"])
    for m in MS.MODULES:
        for k in ("alone", "without"):
            assert close(t_dev[m][k], t_orc[m][k]), (m, k, t_dev[m][k], t_orc[m][k])
            report("mode search %s %s" % (m, k), "device %.4f, oracle %.4f" % (t_dev[m][k], t_orc[m][k]))
    mode_d, trace_d = MS.search(h, cfg, p, C_dev, x_in, budget=0.0)
    mode_o, trace_o = OS.search(spec, p, C_orc, cal, budget=0.0)
    assert all(v == "fp" for v in mode_d.values()) and mode_d == mode_o and len(trace_d) == len(trace_o) == 6
    for step, ((md, ed), (mo, eo, cands)) in enumerate(zip(trace_d, trace_o)):
        assert close(ed, eo), (step, ed, eo)
        if md != mo:
            # the device released another module than the oracle: legitimate only if the oracle's candidates for the step
            # that led here were within the allowance of each other
            prev_cands = sorted(trace_o[step - 1][2].values())
            assert step > 0 and close(prev_cands[0], prev_cands[1]), (step, md, mo, prev_cands)
            break                                                    # the walks have parted ways: later steps differ by design


def test_sensitivity_and_greedy_search(h):
    shape = W.tiny_shape(B=2, S=128, H=256, nh=4, F=512, eps=1e-5, n_outlier=2)
    cfg = prep.LayerConfig(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, eps=shape.eps)
    p = W.layer_params(shape, 61)
    x = W.activations(shape, 61)
    cal = O.layernorm(x.astype(np.float64), p["ln0_g"], p["ln0_b"], shape.eps)
    C = prep.calibrate(cfg, p, cal, shape.B)
    x_in = torch.from_numpy(cal).to(torch.float16).cuda()
    t = MS.sensitivity(h, cfg, p, C, x_in)
    assert set(t) == set(MS.MODULES) | {"all_int8"}
    for m in MS.MODULES:
        # one INT8 module perturbs the layer a little, never more than a few percent; all INT8 is the largest error
        assert 0.0 < t[m]["alone"] < 0.1 and t[m]["without"] <= t["all_int8"] * 1.5 + 1e-3
    # a budget above the all-INT8 error keeps M3; a budget of zero walks all the way to FP
    mode, trace = MS.search(h, cfg, p, C, x_in, budget=10.0)
    assert mode == prep.PRESETS["M3"] and len(trace) == 1
    mode, trace = MS.search(h, cfg, p, C, x_in, budget=t["all_int8"] * 0.5)
    assert trace[-1][1] <= t["all_int8"] * 0.5 or all(v == "fp" for v in mode.values())
    errs = [e for _, e in trace]
    assert all(b <= a * 1.2 + 1e-4 for a, b in zip(errs, errs[1:]))     # releasing a module does not make it worse
