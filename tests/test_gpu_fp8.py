"""The FP8 (e4m3) variant of LN^quant and GeMM^quant against the oracle: the same fusion points with an 8-bit
floating-point payload (scale = absmax / 448, saturating round-to-nearest-even conversion)."""
import numpy as np
import pytest
import torch

from oracle import ops as O
from oracle import quant as Q
from paper_2310_17723_b200 import hero, workloads as W
from gpu_util import f32, rel_err

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


@pytest.mark.parametrize("M,H", [(7, 768), (300, 1024), (65, 4096)])
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
    np.testing.assert_allclose(sc.cpu().numpy(), want.row_scale, rtol=2e-6)
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
    np.testing.assert_allclose(sc.cpu().numpy(), want.row_scale, rtol=2e-6)
    assert_f8_close(f8_vals(out), want.data, 1e-4, "LN^quant e4m3 + e4m3")


GEMM_CASES = [(200, 512, 256, "none"), (1024, 1024, 2048, "none"), (1024, 1024, 2048, "gelu_erf"), (129, 4096, 1024, "none"),
              (2000, 768, 3072, "gelu_erf")]


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
