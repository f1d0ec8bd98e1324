"""Pins for oracle/quant.py: what Sec. 2.1 and arithmetic fix, independent of the oracle's code."""
import os

import numpy as np
import pytest

from oracle import quant as Q

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        return [l.split() for l in f if l.strip() and not l.startswith("#")]


def test_rne_and_clip_golden():
    for v, want in _rows("rne_cases.txt"):
        assert int(Q.quant_sym(np.array([float(v)]), 1.0)[0]) == int(want), v
        # the same ratio with a non-unit scale (power of two: the ratio stays exact)
        assert int(Q.quant_sym(np.array([float(v) * 0.25]), 0.25)[0]) == int(want), v


def test_reconstruction_half_step_bound():
    g = np.random.default_rng(1)
    x = g.standard_normal((64, 96)) * 3.0
    # TWQ (Eq. 3)
    q, s = Q.quant_twq(x)
    assert q.dtype == np.int8 and s.shape == (64,)
    assert np.all(np.abs(x - s[:, None] * q) <= s[:, None] * 0.5 * (1 + 1e-6))
    assert np.all(np.max(np.abs(q.astype(int)), axis=1) == 127)      # the absmax element maps to +-127
    assert q.min() >= -127
    # column-wise weights (Eq. 2)
    wq, sw = Q.quant_weight_columnwise(x)
    assert sw.shape == (96,)
    assert np.all(np.abs(x - wq * sw[None, :]) <= sw[None, :] * 0.5 * (1 + 1e-6))
    assert np.all(np.max(np.abs(wq.astype(int)), axis=0) == 127)
    # FWQ / SQ with a given scale: bound holds inside the range, saturation outside
    sf = np.full(96, 0.01)
    qf = Q.quant_fwq(x, sf)
    inside = np.abs(x) <= 127 * 0.01
    assert np.all(np.abs(x - qf * 0.01)[inside] <= 0.005 * (1 + 1e-9))
    assert np.all(np.abs(qf[~inside].astype(int)) == 127)
    assert np.array_equal(Q.quant_sq(x, 0.01), qf)


def test_scale_axes_follow_eq3_eq4():
    # a matrix whose rows have very different magnitudes: TWQ must scale per row, FWQ per column
    x = np.outer(np.array([1.0, 10.0, 100.0]), np.ones(5)) * np.array([1, -1, 0.5, 0.25, -0.125])
    q, s = Q.quant_twq(x)
    assert np.allclose(s, np.array([1.0, 10.0, 100.0]) / 127, rtol=1e-6)
    assert np.array_equal(q[0], q[1]) and np.array_equal(q[1], q[2])
    wq, sw = Q.quant_weight_columnwise(x)
    assert np.allclose(sw, 100.0 * np.abs([1, -1, 0.5, 0.25, -0.125]) / 127, rtol=1e-6)


def test_zero_rows_and_columns_get_unit_scale():
    x = np.zeros((3, 4))
    q, s = Q.quant_twq(x)
    assert np.all(q == 0) and np.all(s == 1.0)
    wq, sw = Q.quant_weight_columnwise(x)
    assert np.all(wq == 0) and np.all(sw == 1.0)


def test_unsigned_softmax_code_range_and_golden():
    p = np.linspace(0.0, 1.0, 1001)
    u = Q.quant_unsigned(p, 1.0 / 255)
    assert u.dtype == np.uint8 and u.min() == 0 and u.max() == 255
    assert np.all(np.diff(u.astype(int)) >= 0)
    for S, want in _rows("uniform_softmax_u8.txt"):
        assert int(Q.quant_unsigned(np.array([1.0 / int(S)]), 1.0 / 255)[0]) == int(want)
    assert int(Q.quant_unsigned(np.array([2.0]), 1.0 / 255)[0]) == 255      # clip


def test_scales_are_fp32_representable():
    g = np.random.default_rng(2)
    _, s = Q.quant_twq(g.standard_normal((10, 33)))
    assert np.array_equal(s, s.astype(np.float32).astype(np.float64))


def test_storage_rounding_grids():
    g = np.random.default_rng(3)
    x = g.standard_normal(4096) * 7
    torch = pytest.importorskip("torch")
    for name, tdt, mant in (("f16", torch.float16, 11), ("bf16", torch.bfloat16, 8)):
        r = Q.round_to_storage(x, name)
        # on the grid: survives a trip through the library's type unchanged
        assert np.array_equal(r, torch.from_numpy(r).to(tdt).to(torch.float64).numpy())
        # nearest grid point: error at most half a unit in the last place of that binade
        ulp = 2.0 ** (np.floor(np.log2(np.abs(x))) - (mant - 1))
        assert np.all(np.abs(r - x) <= 0.5 * ulp)
        # agrees with the library's conversion except where its detour through fp32 hits a tie
        lib = torch.from_numpy(x).to(tdt).to(torch.float64).numpy()
        assert np.mean(lib != r) < 1e-3
    # exact ties go to even: 1 + 2^-8 is halfway between bf16 neighbours 1 and 1 + 2^-7
    assert Q.round_to_storage(np.array([1.0 + 2.0 ** -8]), "bf16")[0] == 1.0
    assert Q.round_to_storage(np.array([1.0 + 3 * 2.0 ** -8]), "bf16")[0] == 1.0 + 2.0 ** -6
    assert Q.round_to_storage(np.array([1.0 + 2.0 ** -11]), "f16")[0] == 1.0
    assert Q.round_to_storage(np.array([1.0 + 3 * 2.0 ** -11]), "f16")[0] == 1.0 + 2.0 ** -9


# ------------------------------------------------------------------ FP8 (e4m3) quantizer
def test_e4m3_round_matches_the_library_conversion_and_saturates():
    import torch
    g = np.random.default_rng(40)
    x = np.concatenate([g.standard_normal(20000) * s for s in (1e-3, 0.05, 1.0, 30.0, 200.0)])
    x = x[np.abs(x) <= 448.0]
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).to(torch.float64).numpy()
    # the library converts through fp32 first; on values exactly representable in fp32 the two agree bit for bit
    x32 = x.astype(np.float32).astype(np.float64)
    ref = torch.from_numpy(x32).to(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(Q.e4m3_round(x32), ref)
    # every representable e4m3 value is a fixed point
    codes = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    codes = codes[np.isfinite(codes)]
    assert np.array_equal(Q.e4m3_round(codes), codes) and codes.max() == 448.0
    # ties go to the even mantissa; saturation instead of NaN / inf
    assert Q.e4m3_round(17.0) == 16.0 and Q.e4m3_round(19.0) == 20.0 and Q.e4m3_round(2.0 ** -10) == 0.0
    assert Q.e4m3_round(1.5 * 2.0 ** -9) == 2.0 ** -8 and Q.e4m3_round(1e9) == 448.0 and Q.e4m3_round(-460.0) == -448.0
    # scale convention: the largest magnitude lands on 448
    y = g.standard_normal((7, 64)) * 3
    s = Q.f8_scale(np.abs(y).max())
    assert np.abs(Q.quant_f8(y, s)).max() == 448.0
    # relative reconstruction error of a normal value is at most half a mantissa step (2^-4)
    big = np.abs(y) > s * 2.0 ** -6
    assert np.all(np.abs(Q.quant_f8(y, s) * s - y)[big] <= np.abs(y)[big] * 2.0 ** -4 * (1 + 1e-9))
