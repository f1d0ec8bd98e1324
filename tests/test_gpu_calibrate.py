"""Calibration on the device (Sec. 2.1; Eq. 2, Eq. 4-5, Eq. 16, Eq. 20-23, Eq. 32) against the oracle's fp64 calibration:
the observers are exact on the tensor they read; the statistics of the FP16 / BF16 layer differ from the fp64 layer's
only by the storage rounding at every operator border."""
import numpy as np
import pytest
import torch

from oracle import layer as OL
from oracle import ops as O
from paper_2310_17723_b200 import hero, prep, calibrate as CAL, workloads as W
from paper_2310_17723_b200.layer import Layer
from gpu_util import assert_int8_close, rel_err, qt_to_device, TORCH_FP

pytestmark = pytest.mark.gpu


@pytest.fixture
def h():
    hd = hero.Handle()
    yield hd
    hd.check()
    hd.close()


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("rows,cols,pad", [(1, 64, 0), (7, 768, 8), (1000, 1024, 0), (4099, 3072, 1024), (333, 16384, 0)])
def test_absmax_observe_is_exact_and_accumulates(h, dt, rows, cols, pad):
    rng = np.random.default_rng(rows * 131 + cols)
    buf = torch.from_numpy(rng.standard_normal((rows, cols + pad)).astype(np.float32) * 3.0).to(TORCH_FP[dt]).cuda()
    x = buf[:, :cols]                                              # a view with a row pitch larger than its width
    ref = np.abs(x.float().cpu().numpy().astype(np.float64))
    cf = torch.zeros(cols, dtype=torch.float32, device="cuda")
    ct = torch.zeros(1, dtype=torch.float32, device="cuda")
    h.hero_absmax_observe(hero.tensor(x), cf, ct)
    np.testing.assert_array_equal(cf.cpu().numpy().astype(np.float64), ref.max(0))
    assert float(ct.item()) == ref.max()
    # a second batch only raises the running maxima
    y = (x * 0.5).contiguous()
    y[0, 0] = 100.0
    h.hero_absmax_observe(hero.tensor(y), cf, ct)
    want = np.maximum(ref.max(0), np.abs(y.float().cpu().numpy().astype(np.float64)).max(0))
    np.testing.assert_array_equal(cf.cpu().numpy().astype(np.float64), want)
    assert float(ct.item()) == 100.0
    # per-tensor only / per-feature only, and an all-zero tensor leaves zeros (scale_from_absmax maps them to 1)
    z = torch.zeros(5, 64, dtype=TORCH_FP[dt], device="cuda")
    c0 = torch.zeros(64, dtype=torch.float32, device="cuda")
    h.hero_absmax_observe(hero.tensor(z), c0, None)
    assert float(c0.abs().max().item()) == 0.0
    t0 = torch.zeros(1, dtype=torch.float32, device="cuda")
    h.hero_absmax_observe(hero.tensor(x), None, t0)
    assert float(t0.item()) == ref.max()


# every tile kernel the FP product can take: few rows (1-CTA kernels, three tile widths), many rows (CTA pair), ragged M
# and N, with and without the GELU, FP16 and BF16
@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("M,K,N,act", [(40, 256, 64, "none"), (128, 512, 1024, "gelu_erf"), (300, 1024, 4096, "none"),
                                       (1300, 512, 2000, "gelu_erf"), (4099, 1024, 3072, "none")])
def test_linear_epilogue_observer_equals_the_streaming_observer(h, dt, M, K, N, act):
    # the observer fused into the epilogue sees the values as stored: it must agree exactly with hero_absmax_observe on
    # the finished tensor, accumulate over calls, and leave columns it was not given alone
    g = W.rng(9, M + N)
    t = TORCH_FP[dt]
    A = torch.from_numpy(g.standard_normal((M, K)).astype(np.float32)).to(t).cuda()
    Wt = torch.from_numpy((g.standard_normal((N, K)) * 0.05).astype(np.float32)).to(t).cuda()
    bias = torch.from_numpy((g.standard_normal(N) * 0.1).astype(np.float32)).cuda()
    out = torch.empty(M, N, dtype=t, device="cuda")
    fused = torch.zeros(N, dtype=torch.float32, device="cuda")
    h.hero_w8a8_linear(hero.tensor(A), Wt, hero.tensor(out), bias=bias, act=act, out_col_absmax=fused)
    ref = torch.zeros(N, dtype=torch.float32, device="cuda")
    h.hero_absmax_observe(hero.tensor(out), ref, None)
    h.check()
    assert torch.equal(fused, ref)
    assert float(fused.max()) > 0
    # a second batch: running maxima
    A2 = (A * 0.5).contiguous()
    A2[0] = A[0] * 3
    h.hero_w8a8_linear(hero.tensor(A2), Wt, hero.tensor(out), bias=bias, act=act, out_col_absmax=fused)
    h.hero_absmax_observe(hero.tensor(out), ref, None)
    h.check()
    assert torch.equal(fused, ref)


def test_linear_epilogue_observer_refuses_an_int8_output(h):
    A = torch.zeros(256, 256, dtype=torch.int8, device="cuda")
    Wt = torch.zeros(256, 256, dtype=torch.int8, device="cuda")
    out = torch.empty(256, 256, dtype=torch.int8, device="cuda")
    sc = torch.ones(256, dtype=torch.float32, device="cuda")
    with pytest.raises(hero.HeroError) as e:
        h.hero_w8a8_linear(hero.tensor(A), Wt, hero.tensor(out, "fwq", sc), w_scale=sc, out_col_absmax=sc)
    assert e.value.status == hero.ERR_UNSUPPORTED


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("M,H,flavour", [(5, 64, "ln"), (1000, 768, "ln"), (4099, 1024, "add_ln"), (333, 4096, "add_ln"),
                                         (777, 1024, "add_ln_fp"), (1300, 768, "bare_add")])
def test_layernorm_observer_equals_the_streaming_observer(h, dt, M, H, flavour):
    # the observer of the LayerNorm call sees the FP tensor it stores (out; fp_out for the bare residual add) as stored
    g = W.rng(21, M + H)
    t = TORCH_FP[dt]
    mk = lambda s: torch.from_numpy((g.standard_normal((M, H)) * s).astype(np.float32)).to(t).cuda()
    x, br = mk(1.0), mk(0.3)
    gam = torch.from_numpy((1 + 0.1 * g.standard_normal(H)).astype(np.float32)).cuda()
    bet = torch.from_numpy((0.1 * g.standard_normal(H)).astype(np.float32)).cuda()
    out, fpo = torch.empty(M, H, dtype=t, device="cuda"), torch.empty(M, H, dtype=t, device="cuda")
    fused = torch.zeros(H, dtype=torch.float32, device="cuda")
    ref = torch.zeros(H, dtype=torch.float32, device="cuda")

    def run(xx):
        if flavour == "ln":
            h.hero_layernorm_quant(hero.tensor(xx), gam, bet, 1e-5, hero.tensor(out), out_col_absmax=fused)
            return out
        if flavour == "add_ln":
            h.hero_layernorm_quant(hero.tensor(xx), gam, bet, 1e-5, hero.tensor(out), branch=hero.tensor(br), out_col_absmax=fused)
            return out
        if flavour == "add_ln_fp":
            h.hero_layernorm_quant(hero.tensor(xx), gam, bet, 1e-5, hero.tensor(out), branch=hero.tensor(br),
                                   fp_out=hero.tensor(fpo), out_col_absmax=fused)
            return out
        h.hero_layernorm_quant(hero.tensor(xx), None, None, 1e-5, None, branch=hero.tensor(br), fp_out=hero.tensor(fpo),
                               out_col_absmax=fused)
        return fpo

    for xx in (x, (x * 0.5 + 2.0).contiguous()):                   # the second batch: running maxima
        seen = run(xx)
        h.hero_absmax_observe(hero.tensor(seen), ref, None)
        h.check()
        assert torch.equal(fused, ref)
    assert float(fused.min()) > 0
    # the observed call stores what the unobserved one stores
    plain = torch.empty_like(seen)
    if flavour == "bare_add":
        h.hero_layernorm_quant(hero.tensor(xx), None, None, 1e-5, None, branch=hero.tensor(br), fp_out=hero.tensor(plain))
    else:
        h.hero_layernorm_quant(hero.tensor(xx), gam, bet, 1e-5, hero.tensor(plain),
                               branch=None if flavour == "ln" else hero.tensor(br),
                               fp_out=hero.tensor(torch.empty_like(fpo)) if flavour == "add_ln_fp" else None)
    h.check()
    if flavour == "bare_add":
        assert torch.equal(plain.view(torch.int16), seen.view(torch.int16))
    else:                                                          # another kernel: the row sums may round differently
        assert torch.allclose(plain.float(), seen.float(), rtol=1e-2, atol=1e-2)


def test_layernorm_observer_refuses_an_int8_output(h):
    x = torch.zeros(64, 256, dtype=torch.float16, device="cuda")
    out = torch.empty(64, 256, dtype=torch.int8, device="cuda")
    sc = torch.ones(256, dtype=torch.float32, device="cuda")
    with pytest.raises(hero.HeroError) as e:
        h.hero_layernorm_quant(hero.tensor(x), sc, sc, 1e-5, hero.tensor(out, "fwq", sc), out_col_absmax=sc)
    assert e.value.status == hero.ERR_UNSUPPORTED


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("B,S,nh,dh,mask,klen", [(2, 128, 4, 64, "none", False), (3, 200, 2, 128, "causal", False),
                                                   (2, 333, 3, 64, "none", True), (1, 1000, 2, 64, "causal", False)])
def test_attention_observer_equals_the_streaming_observer(h, dt, B, S, nh, dh, mask, klen):
    g = W.rng(33, B * S + nh)
    t = TORCH_FP[dt]
    H = nh * dh
    qkv = torch.from_numpy(g.standard_normal((B * S, 3 * H)).astype(np.float32)).to(t).cuda()
    q, k, v = qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:]
    kl = torch.from_numpy(g.integers(1, S + 1, B).astype(np.int32)).cuda() if klen else None
    out = torch.empty(B * S, H, dtype=t, device="cuda")
    fused = torch.zeros(H, dtype=torch.float32, device="cuda")
    ref = torch.zeros(H, dtype=torch.float32, device="cuda")
    for scale in (1.0, 2.0):                                       # the second batch: running maxima
        vv = (qkv * scale).contiguous()
        h.hero_int8_attention(vv[:, :H], vv[:, H:2 * H], vv[:, 2 * H:], B, S, nh, dh, hero.tensor(out), mask=mask,
                              key_len=kl, out_col_absmax=fused)
        h.hero_absmax_observe(hero.tensor(out), ref, None)
        h.check()
        assert torch.equal(fused, ref)
    assert float(fused.min()) > 0


def test_attention_observer_refuses_the_int8_core(h):
    q = torch.zeros(128, 64, dtype=torch.int8, device="cuda")
    out = torch.empty(128, 64, dtype=torch.float16, device="cuda")
    sc = torch.zeros(64, dtype=torch.float32, device="cuda")
    with pytest.raises(hero.HeroError) as e:
        h.hero_int8_attention(q, q, q, 1, 128, 1, 64, hero.tensor(out), out_col_absmax=sc)
    assert e.value.status == hero.ERR_UNSUPPORTED


@pytest.mark.parametrize("K,N,fold", [(256, 192, "none"), (1024, 3072, "both"), (4096, 1024, "in"), (768, 768, "out")])
def test_quantize_weight_matches_fold_then_eq2(h, K, N, fold):
    rng = np.random.default_rng(K + N)
    Wm = rng.standard_normal((K, N)) * 0.02
    Wm[:, 3] = 0.0                                                 # a zero output feature: scale 1, codes 0
    b = rng.standard_normal(N) * 0.01
    s_in = np.exp(rng.standard_normal(K) * 0.5) * 0.03 if fold in ("in", "both") else None
    s_out = np.exp(rng.standard_normal(N) * 0.5) * 0.05 if fold in ("out", "both") else None
    Wq, ws, bo = CAL.fold_quantize_gpu(h, Wm, b, s_in, s_out)
    # the device reads FP32 master weights and FP32 scale vectors: give the oracle the same values
    f32 = lambda a: None if a is None else np.asarray(a, np.float64).astype(np.float32).astype(np.float64)
    W_i8, S_w, b_ref = OL.fold_and_quantize(f32(Wm), f32(b), f32(s_in), f32(s_out))
    assert_int8_close(Wq, np.ascontiguousarray(np.asarray(W_i8).T), 1e-4, "W_i8")
    np.testing.assert_allclose(ws, np.asarray(S_w, np.float64), rtol=1e-6)
    np.testing.assert_allclose(bo, b_ref, rtol=1e-6, atol=1e-12)
    assert ws[3] == 1.0 and not Wq[3].any()


@pytest.mark.parametrize("K,N,fold", [(256, 192, "none"), (1024, 3072, "both"), (4096, 1024, "in")])
def test_quantize_weight_f8_matches_fold_then_e4m3(h, K, N, fold):
    # the FP8 variant's weights prepared on the device: absmax / 448 scales, saturating round-to-nearest-even e4m3 codes
    rng = np.random.default_rng(7 * K + N)
    Wm = rng.standard_normal((K, N)) * 0.02
    Wm[:, 5] = 0.0
    b = rng.standard_normal(N) * 0.01
    s_in = np.exp(rng.standard_normal(K) * 0.5) * 0.03 if fold in ("in", "both") else None
    s_out = np.exp(rng.standard_normal(N) * 0.5) * 0.05 if fold == "both" else None
    Wq, ws, bo = CAL.fold_quantize_gpu(h, Wm, b, s_in, s_out, payload="f8")
    f32 = lambda a: None if a is None else np.asarray(a, np.float64).astype(np.float32).astype(np.float64)
    W_f8, S_w, b_ref = OL.fold_and_quantize(f32(Wm), f32(b), f32(s_in), f32(s_out), payload="f8")
    got = torch.from_numpy(Wq).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)        # [N][K] e4m3 values
    want = np.ascontiguousarray(np.asarray(W_f8).T)
    np.testing.assert_allclose(ws, np.asarray(S_w, np.float64), rtol=1e-6)
    np.testing.assert_allclose(bo, b_ref, rtol=1e-6, atol=1e-12)
    # identical codes except where fp32 and fp64 arithmetic fall on different sides of an e4m3 rounding tie: then the
    # neighbouring code (one step of 2^-3 relative at most)
    d = got != want
    assert d.mean() <= 1e-4, float(d.mean())
    assert np.all(np.abs(got - want)[d] <= np.abs(want[d]) * 0.126 + 2.0 ** -9)
    assert ws[5] == 1.0 and not got[5].any()
    assert np.abs(got).max() == 448.0                               # a column's largest weight lands on the largest code


SMALL = dict(B=2, S=128, H=256, nh=4, F=512)


def _case(arch, dt, mask):
    shape = W.tiny_shape(**SMALL, eps=1e-5, n_outlier=2, arch=arch, mask=mask, fp_dtype=dt)
    spec = OL.LayerSpec(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, arch=shape.arch, mask=shape.mask,
                        fp_dtype=shape.fp_dtype, eps=shape.eps)
    p = W.layer_params(shape, 77)
    x = W.activations(shape, 77)
    cal_in = O.layernorm(x, p["ln0_g"], p["ln0_b"], spec.eps) if arch == "post_ln" else x
    cfg = prep.LayerConfig(B=spec.B, S=spec.S, H=spec.H, nh=spec.nh, F=spec.F, arch=spec.arch, act=spec.act, eps=spec.eps,
                           mask=spec.mask, fp_dtype=spec.fp_dtype, mode=dict(spec.mode), gran_in=spec.gran_in,
                           gran_mid=spec.gran_mid, gran_attn=spec.gran_attn, gran_out=spec.gran_out)
    return shape, spec, cfg, p, x, cal_in


@pytest.mark.parametrize("arch,dt,mask", [("post_ln", "f16", "none"), ("pre_ln", "bf16", "causal"), ("pre_ln", "f16", "none")])
def test_device_calibration_matches_fp64_calibration(h, arch, dt, mask):
    shape, spec, cfg, p, x, cal_in = _case(arch, dt, mask)
    # both sides see the calibration input on the storage grid of the layer
    cal_q = O.fp_tensor(cal_in, dt).real()
    want = OL.calibrate(spec, p, cal_q, shape.B)
    got = CAL.calibrate_gpu(h, cfg, p, cal_q, shape.B)
    # every tensor of the device's layer is rounded to FP16 (11 bits) / BF16 (8 bits) where the fp64 layer is not
    tol = 4e-3 if dt == "f16" else 3e-2
    assert set(got) == set(want)
    for k in want:
        np.testing.assert_allclose(np.asarray(got[k], np.float64), np.asarray(want[k], np.float64), rtol=tol, err_msg=k)
    if arch == "post_ln":       # the tensor feeding QKV is the calibration input itself: identical values, exact statistics
        np.testing.assert_array_equal(np.asarray(got["S_in_f"]), np.asarray(want["S_in_f"], np.float32))


def test_int8_layer_prepared_on_the_device(h):
    """Calibrate, fold and quantize on the device, run the INT8 layer, and compare with the un-quantized fp64 layer:
    the error must be of the size the oracle's own calibration gives."""
    shape, spec, cfg, p, x, cal_in = _case("post_ln", "f16", "none")
    cal_q = O.fp_tensor(cal_in, "f16").real()
    C = CAL.calibrate_gpu(h, cfg, p, cal_q, shape.B)
    L = CAL.prepare_layer_gpu(h, cfg, p, C)
    L_host = prep.prepare_layer(cfg, p, C)
    for name in ("qkv", "o", "fc1", "fc2"):                        # device fold + Eq. 2 = host fold + Eq. 2 on the same scales
        assert_int8_close(L[name]["W"], L_host[name]["W"], 1e-4, name)
        np.testing.assert_allclose(L[name]["w_scale"], L_host[name]["w_scale"], rtol=1e-6)
    layer = Layer(h, L)
    # entry LN^quant (TWQ) feeds the layer, as in the benchmark
    Lo = OL.prepare_layer(spec, p, OL.calibrate(spec, p, cal_q, shape.B))
    x_in = OL.entry_ln(O.fp_tensor(x, "f16"), p["ln0_g"], p["ln0_b"], spec.eps, Lo["ln_in_out"])
    _, in_desc, _ = qt_to_device(x_in)
    out = torch.empty(shape.M, shape.H, dtype=torch.int8, device="cuda")
    sc = torch.zeros(shape.M, dtype=torch.float32, device="cuda")
    layer.forward(in_desc, hero.tensor(out, "twq", sc))
    h.check()
    got = out.cpu().numpy().astype(np.float64) * sc.cpu().numpy().astype(np.float64)[:, None]
    ref = OL.layer_fp64(spec, p, cal_in, B=shape.B)["x_out"]
    ora = OL.layer_forward(Lo, x_in)["x_out"].real()
    e_dev, e_ora = rel_err(got, ref), rel_err(ora, ref)
    assert e_dev < 0.1 and e_dev < 1.5 * e_ora + 1e-3, (e_dev, e_ora)
