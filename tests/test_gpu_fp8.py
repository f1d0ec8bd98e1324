"""The FP8 (e4m3) variant of LN^quant and GeMM^quant against the oracle: the same fusion points with an 8-bit
floating-point payload (scale = absmax / 448, saturating round-to-nearest-even conversion)."""
import numpy as np
import pytest
import torch

from oracle import ops as O
from oracle import quant as Q
from paper_2310_17723_b200 import hero, workloads as W
from gpu_util import f32, rel_err, assert_scales_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def h():
    hd = hero.Handle()
    yield hd
    hd.check()
    hd.close()


def to_f8(values):
    """e4m3 values (already on the grid) -> device tensor of that type (the cast is exact)."""
    return torch.from_numpy(np.asarray(values, np.float32)).to(torch.float8_e4m3fn).cuda()


def f8_vals(t):
    return t.float().cpu().numpy().astype(np.float64)


def assert_f8_close(got, want, frac, what):
    """Bit-exact except a step to the neighbouring e4m3 value on at most `frac` of the elements (an fp32-vs-fp64
    difference that moves a value across a rounding boundary)."""
    d = np.abs(got - want)
    step = np.maximum(np.abs(want), 2.0 ** -6) * 2.0 ** -3 * 1.0001     # spacing of the binade (one mantissa step)
    assert np.all(d <= step), "%s: more than one e4m3 step apart" % what
    f = float(np.mean(d > 0))
    assert f <= max(frac, 1.0 / want.size), "%s: %.3g of the elements differ" % (what, f)


@pytest.mark.parametrize("M,H", [(7, 768), (300, 1024), (65, 4096), (300, 768), (9, 1280)])
def test_ln_quant_fp16_to_e4m3_twq_and_static(h, M, H):
    g = W.rng(11, M + H)
    x = g.standard_normal((M, H)) * 2
    x[:, 5] *= 20
    gam, bet = 1 + 0.1 * g.standard_normal(H), 0.1 * g.standard_normal(H)
    xin = O.fp_tensor(x, "f16")
    want, _ = O.ln_quant([xin], gam, bet, 1e-5, O.OutSpec("twq", payload="f8"))
    xd = torch.from_numpy(xin.data).to(torch.float16).cuda()
    out = torch.empty(M, H, dtype=torch.float8_e4m3fn, device="cuda")
    sc = torch.zeros(M, dtype=torch.float32, device="cuda")
    h.hero_layernorm_quant(hero.tensor(xd), f32(gam), f32(bet), 1e-5, hero.tensor(out, "twq", sc))
    h.check()
    assert_scales_close(sc.cpu().numpy(), want.row_scale, 1e-6, "e4m3 LN row scales")
    assert_f8_close(f8_vals(out), want.data, 1e-4, "LN^quant e4m3 TWQ")
    # static feature-wise scale, half the needed range so that the largest entries saturate at 448
    S = np.abs(O.layernorm(xin.real(), gam, bet, 1e-5)).max(0) / 448 / 2
    want, _ = O.ln_quant([xin], gam, bet, 1e-5, O.OutSpec("fwq", scale=S.astype(np.float32).astype(np.float64), payload="f8"))
    h.hero_layernorm_quant(hero.tensor(xd), f32(gam), f32(bet), 1e-5, hero.tensor(out, "fwq", f32(S)))
    h.check()
    assert_f8_close(f8_vals(out), want.data, 1e-4, "LN^quant e4m3 FWQ")
    assert np.abs(f8_vals(out)).max() == 448.0


def test_ln_quant_e4m3_residual_plus_e4m3_branch(h):
    # Eq. 19 / 31 with e4m3 payloads: TWQ residual + FWQ branch -> TWQ
    M, H = 257, 1024
    g = W.rng(11, 3)
    res = O.emit(g.standard_normal((M, H)) * 3, O.OutSpec("twq", payload="f8"))
    S_o = (np.abs(g.standard_normal(H)) * 0.01 + 0.005).astype(np.float32).astype(np.float64)
    br = O.emit(g.standard_normal((M, H)) * 2, O.OutSpec("fwq", scale=S_o, payload="f8"))
    gam, bet = 1 + 0.1 * g.standard_normal(H), 0.1 * g.standard_normal(H)
    want, _ = O.ln_quant([res, br], gam, bet, 1e-5, O.OutSpec("twq", payload="f8"))
    out = torch.empty(M, H, dtype=torch.float8_e4m3fn, device="cuda")
    sc = torch.zeros(M, dtype=torch.float32, device="cuda")
    h.hero_layernorm_quant(hero.tensor(to_f8(res.data), "twq", f32(res.row_scale)), f32(gam), f32(bet), 1e-5,
                           hero.tensor(out, "twq", sc), branch=hero.tensor(to_f8(br.data), "fwq", f32(S_o)))
    h.check()
    assert_scales_close(sc.cpu().numpy(), want.row_scale, 1e-6, "e4m3 LN row scales")
    assert_f8_close(f8_vals(out), want.data, 1e-4, "LN^quant e4m3 + e4m3")


GEMM_CASES = [(200, 512, 256, "none"), (1024, 1024, 2048, "none"), (1024, 1024, 2048, "gelu_erf"), (129, 4096, 1024, "none"),
              (2000, 768, 3072, "gelu_erf"),
              # few rows: the kernel with the operands swapped on the tensor core and K split over a cluster
              (1, 4096, 1024, "none"), (16, 8192, 512, "gelu_erf"), (40, 16384, 1024, "none"), (128, 8192, 256, "gelu_erf")]


@pytest.mark.parametrize("M,K,N,act", GEMM_CASES)
def test_gemm_quant_e4m3(h, M, K, N, act):
    g = W.rng(12, M + K + N)
    x = g.standard_normal((M, K)) * 2
    Wm = g.standard_normal((K, N)) * 0.03
    b = g.standard_normal(N) * 0.1
    xq = O.emit(x, O.OutSpec("twq", payload="f8"))
    Wq, Sw = O.quant_weight_columnwise_f8(Wm)
    A = hero.tensor(to_f8(xq.data), "twq", f32(xq.row_scale))
    Wd = to_f8(np.ascontiguousarray(Wq.T))                            # [N][K]
    ref = O.gemm_quant_f8(xq, Wq, Sw, b, act, O.OutSpec("fp", dtype="f64")).data
    # FP16 output
    out = torch.empty(M, N, dtype=torch.float16, device="cuda")
    h.hero_w8a8_linear(A, Wd, hero.tensor(out), w_scale=f32(Sw), bias=f32(b), act=act)
    h.check()
    assert rel_err(out.float().cpu().numpy(), ref) < 2e-3
    # e4m3 output with a calibrated feature-wise scale (the quantizer is e4m3(v / S): post_scale carries 1 / S)
    S = (np.abs(ref).max(0) / 448).astype(np.float32).astype(np.float64)
    S[S == 0] = 1.0
    want = O.gemm_quant_f8(xq, Wq, Sw, b, act, O.OutSpec("fwq", scale=S, payload="f8"))
    o8 = torch.empty(M, N, dtype=torch.float8_e4m3fn, device="cuda")
    h.hero_w8a8_linear(A, Wd, hero.tensor(o8, "fwq", f32(S)), w_scale=f32(Sw), bias=f32(b), act=act, post_scale=f32(1.0 / S))
    h.check()
    # the tensor core accumulates in FP32 and the epilogue multiplies by the reciprocal scale: a value within ~1e-6 of
    # an e4m3 rounding boundary may land on the neighbouring code
    assert_f8_close(f8_vals(o8), want.data, 1e-3, "GeMM^quant e4m3")


def test_e4m3_rejections(h):
    x = torch.zeros(128, 256, dtype=torch.float8_e4m3fn, device="cuda")
    w = torch.zeros(256, 256, dtype=torch.int8, device="cuda")
    o = torch.zeros(128, 256, dtype=torch.int8, device="cuda")
    s = torch.ones(256, device="cuda")
    with pytest.raises(hero.HeroError):          # e4m3 operands cannot produce INT8
        h.hero_w8a8_linear(hero.tensor(x, "sq", s[:1]), w, hero.tensor(o, "sq", s[:1]), w_scale=s)
    with pytest.raises(hero.HeroError):          # a token-wise output needs a row reduction: not in a GEMM epilogue
        h.hero_w8a8_linear(hero.tensor(x, "sq", s[:1]), w, hero.tensor(x.clone(), "twq", torch.ones(128, device="cuda")), w_scale=s)


ATTN_CASES = [(1, 128, 2, 64, "none", 1.0), (2, 384, 4, 64, "none", 1.0), (1, 333, 2, 128, "causal", 1.0),
              (1, 1024, 1, 128, "causal", 1.0), (2, 200, 2, 64, "none", 0.25)]


@pytest.mark.parametrize("B,S,nh,dh,mask,clipf", ATTN_CASES)
def test_attention_e4m3(h, B, S, nh, dh, mask, clipf):
    """e4m3 Q, K, V and an e4m3 P against the oracle's FP8 attention; clipf < 1 makes s_p too small so that P saturates."""
    g = W.rng(13, S + dh)
    H = nh * dh
    qkv = Q.e4m3_round(g.standard_normal((B * S, 3 * H)) * 100)
    s = float(np.sqrt(1.5) / 100)
    s_q, s_k, s_v, s_p = s, s, 0.02, clipf / 448
    q, k, v = qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:]
    raw = O.attention_f8(q, k, v, B, S, nh, dh, s_q, s_k, s_v, s_p, O.OutSpec("fp", dtype="f64"), mask=mask).data
    t = to_f8(qkv)
    out = torch.full((B * S, H), float("nan"), dtype=torch.float16, device="cuda")
    h.hero_int8_attention(t[:, :H], t[:, H:2 * H], t[:, 2 * H:], B, S, nh, dh, hero.tensor(out), s_q=s_q, s_k=s_k, s_v=s_v, s_p=s_p,
                          mask=mask)
    h.check()
    assert rel_err(out.float().cpu().numpy(), raw) < 3e-3
    S_attn = Q.f8_scale(np.abs(raw).max(0))
    want = O.attention_f8(q, k, v, B, S, nh, dh, s_q, s_k, s_v, s_p, O.OutSpec("fwq", scale=S_attn, payload="f8"), mask=mask)
    o8 = torch.empty(B * S, H, dtype=torch.float8_e4m3fn, device="cuda")
    h.hero_int8_attention(t[:, :H], t[:, H:2 * H], t[:, 2 * H:], B, S, nh, dh, hero.tensor(o8, "fwq", f32(S_attn)), s_q=s_q, s_k=s_k,
                          s_v=s_v, s_p=s_p, mask=mask)
    h.check()
    # an e4m3 P code that flips on an fp32-vs-fp64 tie moves that probability by a whole mantissa step (6-12 % of its
    # value, against 1/255 of full scale for the unsigned 8-bit P of the INT8 core), so an output can move by a step or,
    # where one key dominates the row, two: almost all outputs identical, none further than two steps
    # (the shift is absolute, a fraction of one key's contribution, so next to an output near zero it spans several
    # of that value's fine steps: steps are counted at no less than 1/16 of the full range)
    got, d = f8_vals(o8), np.abs(f8_vals(o8) - want.data)
    step = np.maximum(np.abs(want.data), 448.0 / 16) * 2.0 ** -3 * 1.0001
    stats = (float(np.mean(d > 0)), float(np.mean(d > step)), float((d / step).max()))
    assert np.mean(d > 0) <= 5e-3 and np.mean(d > step) <= 2e-4 and np.all(d <= 2 * step), stats


# ------------------------------------------------------------------------------------------------------------------
# the whole layer with an e4m3 payload (hero_layer_desc.payload = HERO_F8)
# ------------------------------------------------------------------------------------------------------------------
from oracle import layer as OL
from paper_2310_17723_b200.layer import Layer
from gpu_util import qt_to_device, oracle_layer_to_prepared, TORCH_FP


def _f8_layer(shape, seed, **kw):
    spec = OL.LayerSpec(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, arch=shape.arch, mask=shape.mask,
                        fp_dtype=shape.fp_dtype, eps=shape.eps, payload="f8", **kw)
    p = W.layer_params(shape, seed)
    x = W.activations(shape, seed)
    cal = O.layernorm(x, p["ln0_g"], p["ln0_b"], spec.eps) if spec.arch == "post_ln" else x
    Lp = OL.prepare_layer(spec, p, OL.calibrate(spec, p, cal, shape.B))
    if spec.arch == "post_ln":
        x_in = OL.entry_ln(O.fp_tensor(x, spec.fp_dtype), p["ln0_g"], p["ln0_b"], spec.eps, Lp["ln_in_out"])
    else:
        x_in = O.fp_tensor(x, spec.fp_dtype)
    return spec, Lp, x_in


class _F8Borders:
    """Views of the operator-border tensors the layer left in its workspace (e4m3 values, fp32 scales, FP tensors)."""

    def __init__(self, h, layer, M):
        self.lay, self.ws, self.M = h.hero_layer_workspace_layout(layer.desc, M), layer.workspace, M

    def f8(self, name, cols):
        off = getattr(self.lay, name)
        return f8_vals(self.ws[off:off + self.M * cols].view(torch.float8_e4m3fn).view(self.M, cols))

    def f32(self, name):
        off = getattr(self.lay, name)
        return self.ws[off:off + self.M * 4].view(torch.float32).cpu().numpy().astype(np.float64)

    def fp(self, name, cols, dt):
        off = getattr(self.lay, name)
        return self.ws[off:off + self.M * cols * 2].view(TORCH_FP[dt]).view(self.M, cols).float().cpu().numpy().astype(np.float64)


def _like8(template, values, row_scale=None):
    return O.QT("f8", values, row_scale=row_scale if template.row_scale is not None else None, col_scale=template.col_scale)


def _attn_close(got, want, what):
    # the e4m3 P moves an output by up to two steps where one key dominates (see test_attention_e4m3)
    d = np.abs(got - want)
    step = np.maximum(np.abs(want), 448.0 / 16) * 2.0 ** -3 * 1.0001
    stats = (float(np.mean(d > 0)), float(np.mean(d > step)), float((d / step).max()))
    assert np.mean(d > 0) <= 5e-3 and np.mean(d > step) <= 2e-4 and np.all(d <= 2 * step), (what, stats)


# H = 1024 rows take the specialised LN^quant kernel, H = 256 the generic one
@pytest.mark.parametrize("gran_in,gran_attn,H,nh", [("twq", "fwq", 256, 4), ("fwq", "sq", 256, 4), ("twq", "fwq", 1024, 8),
                                                    ("fwq", "sq", 1024, 16)])
def test_post_ln_layer_e4m3_stage_by_stage(h, gran_in, gran_attn, H, nh):
    shape = W.tiny_shape(B=2, S=200, H=H, nh=nh, F=2 * H, eps=1e-5, n_outlier=2)      # ragged attention tiles
    spec, Lp, x_in = _f8_layer(shape, 31, gran_in=gran_in, gran_mid=gran_in, gran_attn=gran_attn)
    M, H, F = spec.M, spec.H, spec.F
    T = OL.layer_forward(Lp, x_in)
    layer = Layer(h, oracle_layer_to_prepared(Lp))
    _, in_desc, _ = qt_to_device(x_in)
    out = torch.empty(M, H, dtype=torch.float8_e4m3fn, device="cuda")
    sc = torch.zeros(M, dtype=torch.float32, device="cuda")
    n0 = h.launches
    layer.forward(in_desc, hero.tensor(out, "twq", sc))
    h.check()
    assert h.launches - n0 == 7
    bd = _F8Borders(h, layer, M)
    # ---- each oracle operator is fed what the device produced one stage earlier
    qkv = _like8(T["qkv"], bd.f8("qkv", 3 * H))
    assert_f8_close(qkv.data, T["qkv"].data, 1e-4, "qkv")
    x_attn = _like8(T["x_attn"], bd.f8("x_attn", H))
    _attn_close(x_attn.data, OL._attention(Lp, qkv, spec.B).data, "x_attn")
    x_o = _like8(T["x_o"], bd.f8("x_o", H))
    assert_f8_close(x_o.data, OL._linear(Lp["o"], x_attn, "none").data, 1e-4, "x_o")
    x_mid = _like8(T["x_mid"], bd.f8("x_mid", H), bd.f32("x_mid_scale"))
    want, _ = O.ln_quant([x_in, x_o], Lp["ln1_g"], Lp["ln1_b"], spec.eps, Lp["ln_mid_out"])
    assert_f8_close(x_mid.data, want.data, 1e-4, "x_mid")
    if gran_in == "twq":
        assert_scales_close(x_mid.row_scale, want.row_scale, 1e-6, "e4m3 x_mid scales")
    a = _like8(T["a"], bd.f8("a", F))
    assert_f8_close(a.data, OL._linear(Lp["fc1"], x_mid, spec.act).data, 2e-4, "a")
    x_2 = _like8(T["x_2"], bd.f8("x_2", H))
    assert_f8_close(x_2.data, OL._linear(Lp["fc2"], a, "none").data, 1e-4, "x_2")
    want, _ = O.ln_quant([x_mid, x_2], Lp["ln2_g"], Lp["ln2_b"], spec.eps, Lp["ln_final_out"])
    assert_f8_close(f8_vals(out), want.data, 1e-4, "x_out")
    assert_scales_close(sc.cpu().numpy(), want.row_scale, 1e-6, "e4m3 LN row scales")
    # ---- free-running against the oracle's own chain: an e4m3 value that flips moves by 6-12 % of itself
    got = f8_vals(out) * sc.cpu().numpy().astype(np.float64)[:, None]
    assert rel_err(got, T["x_out"].real()) < 6e-2
    assert float(np.abs(got - T["x_out"].real()).mean() / np.abs(T["x_out"].real()).mean()) < 5e-3


@pytest.mark.parametrize("preset,H", [("M2", 256), ("M3", 256), ("M3", 1024)])
def test_pre_ln_causal_layer_e4m3(h, preset, H):
    shape = W.tiny_shape(B=2, S=256, H=H, nh=H // 128, F=2 * H, arch="pre_ln", mask="causal", fp_dtype="bf16", eps=1e-5)
    spec, Lp, x_in = _f8_layer(shape, 33, mode=dict(OL.MODE_PRESETS[preset]))
    M, H, F, fd = spec.M, spec.H, spec.F, spec.fp_dtype
    T = OL.layer_forward(Lp, x_in)
    layer = Layer(h, oracle_layer_to_prepared(Lp))
    xd, in_desc, _ = qt_to_device(x_in)
    out = torch.empty(M, H, dtype=torch.bfloat16, device="cuda")
    layer.forward(in_desc, hero.tensor(out))
    h.check()
    bd = _F8Borders(h, layer, M)
    x_in8 = _like8(T["x_in"], bd.f8("x_in", H), bd.f32("x_in_scale"))
    assert_f8_close(x_in8.data, T["x_in"].data, 1e-4, "x_in")
    assert_scales_close(x_in8.row_scale, T["x_in"].row_scale, 1e-6, "e4m3 x_in scales")
    qkv = _like8(T["qkv"], bd.f8("qkv", 3 * H))
    assert_f8_close(qkv.data, OL._linear(Lp["qkv"], x_in8, "none").data, 1e-4, "qkv")
    x_attn = _like8(T["x_attn"], bd.f8("x_attn", H))
    _attn_close(x_attn.data, OL._attention(Lp, qkv, spec.B).data, "x_attn")
    x_o = _like8(T["x_o"], bd.f8("x_o", H))
    assert_f8_close(x_o.data, OL._linear(Lp["o"], x_attn, "none").data, 1e-4, "x_o")
    h_mid = O.QT("fp", bd.fp("h_mid", H, fd), dtype=fd)
    want2, _ = O.ln_quant([h_mid], Lp["ln2_g"], Lp["ln2_b"], spec.eps, Lp["ln_mid_out"])
    x_mid = _like8(T["x_mid"], bd.f8("x_mid", H), bd.f32("x_mid_scale"))
    assert_f8_close(x_mid.data, want2.data, 1e-4, "x_mid")
    want_a = OL._linear(Lp["fc1"], x_mid, spec.act)
    if preset == "M3":
        a = _like8(T["a"], bd.f8("a", F))
        assert_f8_close(a.data, want_a.data, 2e-4, "a")
        x_2 = _like8(T["x_2"], bd.f8("x_2", H))
        assert_f8_close(x_2.data, OL._linear(Lp["fc2"], a, "none").data, 1e-4, "x_2")
    else:                                                   # FC2 left in FP: A and X_2 are BF16 tensors
        a = O.QT("fp", bd.fp("a", F, fd), dtype=fd)
        assert rel_err(a.data, want_a.real()) < 2.0 ** -7
        x_2 = O.QT("fp", bd.fp("x_2", H, fd), dtype=fd)
        assert rel_err(x_2.data, OL._linear(Lp["fc2"], a, "none").real()) < 2.0 ** -7
    _, want_o = O.ln_quant([h_mid, x_2], None, None, spec.eps, None, fp_out_dtype=fd, normalize=False)
    got = out.float().cpu().numpy().astype(np.float64)
    do = np.abs(got - want_o.real())
    assert np.all(do <= 2.0 ** -7 * np.maximum(np.abs(want_o.real()), 2.0 ** -20)) and np.mean(do > 0) < 1e-3
    assert rel_err(got, T["h_out"].real()) < 3e-2


def test_layer_e4m3_rejections(h):
    shape = W.tiny_shape(B=1, S=128, H=256, nh=4, F=512, eps=1e-5)
    spec, Lp, x_in = _f8_layer(shape, 35)
    L = oracle_layer_to_prepared(Lp)
    _, in_desc, _ = qt_to_device(x_in)
    out = torch.empty(spec.M, spec.H, dtype=torch.float8_e4m3fn, device="cuda")
    sc = torch.zeros(spec.M, dtype=torch.float32, device="cuda")
    layer = Layer(h, L)
    layer.desc.p_mode = hero.P_MODE["rowmax"]
    with pytest.raises(hero.HeroError):
        layer.forward(in_desc, hero.tensor(out, "twq", sc))
    layer.desc.p_mode = hero.P_MODE["static"]
    layer.desc.mode[hero.MODULES.index("attn")] = hero.MODE_FP          # FP core feeding an 8-bit attention-output linear
    with pytest.raises(hero.HeroError):
        layer.forward(in_desc, hero.tensor(out, "twq", sc))
    layer.desc.mode[hero.MODULES.index("attn")] = hero.MODE_INT8
    i8 = torch.zeros(spec.M, spec.H, dtype=torch.int8, device="cuda")   # an INT8 input to an e4m3 layer
    with pytest.raises(hero.HeroError):
        layer.forward(hero.tensor(i8, "twq", sc), hero.tensor(out, "twq", sc))
    layer.desc.payload = 3
    with pytest.raises(hero.HeroError):
        layer.forward(in_desc, hero.tensor(out, "twq", sc))
    layer.desc.payload = hero.F8
    layer.forward(in_desc, hero.tensor(out, "twq", sc))
    h.check()
