"""Pins for oracle/ops.py: brute force, closed forms and library routines (CPU only)."""
import math
import os

import numpy as np
import pytest

from oracle import ops as O
from oracle import quant as Q

torch = pytest.importorskip("torch")
GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ integer contraction
def _brute(A, B):
    n, d = A.shape
    m = B.shape[1]
    out = [[0] * m for _ in range(n)]
    for i in range(n):
        for j in range(m):
            s = 0
            for c in range(d):
                s += int(A[i, c]) * int(B[c, j])
            out[i][j] = s
    return np.array(out, dtype=np.int64)


def test_int_matmul_brute_force_and_numpy_int64():
    g = np.random.default_rng(0)
    A = g.integers(-127, 128, (7, 19), dtype=np.int8)
    B = g.integers(-127, 128, (19, 5), dtype=np.int8)
    assert np.array_equal(O.int_matmul(A, B), _brute(A, B))
    U = g.integers(0, 256, (7, 19), dtype=np.uint8)                 # unsigned x signed (P V)
    assert np.array_equal(O.int_matmul(U, B), _brute(U, B))
    A = g.integers(-127, 128, (33, 4096), dtype=np.int8)
    B = g.integers(-127, 128, (4096, 17), dtype=np.int8)
    assert np.array_equal(O.int_matmul(A, B), A.astype(np.int64) @ B.astype(np.int64))
    # worst case magnitudes stay exact
    A = np.full((2, 16384), 127, np.int8)
    B = np.full((16384, 2), -127, np.int8)
    assert np.all(O.int_matmul(A, B) == -16384 * 127 * 127)


def test_int_matmul_is_not_transposed():
    A = np.array([[1, 2], [3, 4]], np.int8)
    B = np.array([[5, 6], [7, 8]], np.int8)
    assert np.array_equal(O.int_matmul(A, B), np.array([[19, 22], [43, 50]]))


# ------------------------------------------------------------------ LayerNorm
def test_layernorm_closed_forms():
    H = 768
    g = np.random.default_rng(1)
    gamma, beta = 1 + 0.1 * g.standard_normal(H), 0.1 * g.standard_normal(H)
    # constant row -> beta
    y = O.layernorm(np.full((1, H), 3.25), gamma, beta, 1e-12)
    assert np.allclose(y, beta, atol=1e-12)
    # arithmetic progression a + k t: mean a + t(H-1)/2, biased variance t^2 (H^2-1)/12
    a, t = 2.0, 0.5
    r = (a + t * np.arange(H))[None, :]
    mu, var = a + t * (H - 1) / 2, t * t * (H * H - 1) / 12
    want = (r - mu) / np.sqrt(var + 1e-5) * gamma + beta
    assert np.allclose(O.layernorm(r, gamma, beta, 1e-5), want, rtol=1e-12, atol=1e-12)
    # two-valued row +-c -> +-gamma + beta as eps -> 0
    r = np.where(np.arange(H) % 2 == 0, 4.0, -4.0)[None, :]
    assert np.allclose(O.layernorm(r, gamma, beta, 0.0), np.sign(r) * gamma + beta, atol=1e-12)


def test_layernorm_matches_library():
    g = np.random.default_rng(2)
    x = g.standard_normal((17, 96)) * 3 + 1
    gamma, beta = g.standard_normal(96), g.standard_normal(96)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(x), (96,), torch.from_numpy(gamma),
                                         torch.from_numpy(beta), 1e-5).numpy()
    assert np.allclose(O.layernorm(x, gamma, beta, 1e-5), ref, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ GELU
def test_gelu_identities_and_library():
    x = np.linspace(-8, 8, 2001)
    assert np.allclose(O.gelu_erf(x) - O.gelu_erf(-x), x, atol=1e-14)
    assert O.gelu_erf(np.array([0.0]))[0] == 0.0
    assert abs(O.gelu_erf(np.array([30.0]))[0] - 30.0) < 1e-12 and abs(O.gelu_erf(np.array([-30.0]))[0]) < 1e-12
    t = torch.from_numpy(x)
    assert np.allclose(O.gelu_erf(x), torch.nn.functional.gelu(t).numpy(), atol=1e-14)
    assert np.allclose(O.gelu_tanh(x), torch.nn.functional.gelu(t, approximate="tanh").numpy(), atol=1e-14)


# ------------------------------------------------------------------ softmax / attention
def test_softmax_rows_and_masks():
    g = np.random.default_rng(3)
    A = g.standard_normal((16, 16)) * 4
    P = O.softmax_masked(A, O.attention_mask(16, "none"))
    assert np.allclose(P.sum(-1), 1.0, atol=1e-15)
    Pc = O.softmax_masked(A, O.attention_mask(16, "causal"))
    assert np.all(np.triu(Pc, 1) == 0.0) and np.allclose(Pc.sum(-1), 1.0, atol=1e-15)
    assert Pc[0, 0] == 1.0
    Pk = O.softmax_masked(A, O.attention_mask(16, "none", key_len=5))
    assert np.all(Pk[:, 5:] == 0.0) and np.allclose(Pk.sum(-1), 1.0, atol=1e-15)
    assert np.all(O.softmax_masked(A, np.zeros((16, 16), bool)) == 0.0)   # fully masked rows -> 0
    ref = torch.softmax(torch.from_numpy(A), -1).numpy()
    assert np.allclose(P, ref, atol=1e-15)


def test_attention_fp_matches_library_sdpa():
    g = np.random.default_rng(4)
    B, S, nh, dh = 2, 24, 3, 8
    H = nh * dh
    q, k, v = (g.standard_normal((B * S, H)) for _ in range(3))
    for mask in ("none", "causal"):
        got = O.attention_fp(q, k, v, B, S, nh, dh, O.OutSpec("fp", dtype="f64"), mask=mask).data
        tq, tk, tv = (torch.from_numpy(a).view(B, S, nh, dh).transpose(1, 2) for a in (q, k, v))
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=(mask == "causal"))
        ref = ref.transpose(1, 2).reshape(B * S, H).numpy()
        assert np.allclose(got, ref, atol=1e-12)


def test_attention_int8_uniform_logits_closed_form():
    # q = 0 -> A = 0 -> P = 1/S -> P_u8 = RNE(255/S) (golden) -> acc = P_u8 * column sum of V
    g = np.random.default_rng(5)
    with open(os.path.join(GOLD, "uniform_softmax_u8.txt")) as f:
        gold = {int(a): int(b) for a, b in (l.split() for l in f if l.strip() and not l.startswith("#"))}
    for S in (128, 384, 512):
        nh, dh = 2, 8
        q = np.zeros((S, nh * dh), np.int8)
        k = g.integers(-127, 128, (S, nh * dh), dtype=np.int8)
        v = g.integers(-127, 128, (S, nh * dh), dtype=np.int8)
        s_v, s_p = 0.03, 1.0 / 255
        o, internals = O.attention_int8(q, k, v, 1, S, nh, dh, 0.1, 0.1, s_v, s_p,
                                        O.OutSpec("fp", dtype="f64"), return_internals=True)
        assert np.all(internals["P_u8"][(0, 0)] == gold[S])
        want = s_p * s_v * gold[S] * v.astype(np.int64).sum(0)
        assert np.allclose(o.data, np.broadcast_to(want, o.data.shape), rtol=1e-13)


def test_attention_int8_dominant_logit_and_causal_row0():
    g = np.random.default_rng(6)
    S, nh, dh = 16, 1, 8
    k = g.integers(-20, 21, (S, dh), dtype=np.int8)
    v = g.integers(-127, 128, (S, dh), dtype=np.int8)
    k[3] = 127                                   # key 3 dominates for a positive query
    q = np.full((S, dh), 127, np.int8)
    s_attn = np.full(dh, 0.05)
    o, it = O.attention_int8(q, k, v, 1, S, nh, dh, 0.05, 0.05, 0.02, 1.0 / 255,
                             O.OutSpec("fwq", scale=s_attn), return_internals=True)
    Pu = it["P_u8"][(0, 0)]
    assert np.all(Pu[:, 3] == 255) and np.all(np.delete(Pu, 3, axis=1) == 0)
    assert np.array_equal(o.data, np.broadcast_to(Q.quant_sym(0.02 * v[3].astype(float), 0.05), (S, dh)))
    # causal: row 0 sees only key 0 -> P = [1, 0, ...] -> X_attn[0] = Qs(s_v V[0]; S_attn)
    q = g.integers(-127, 128, (S, dh), dtype=np.int8)
    o = O.attention_int8(q, k, v, 1, S, nh, dh, 0.05, 0.05, 0.02, 1.0 / 255,
                         O.OutSpec("fwq", scale=s_attn), mask="causal")
    assert np.array_equal(o.data[0], Q.quant_sym(0.02 * v[0].astype(float), 0.05))


def test_attention_int8_tracks_fp_attention():
    # with fine scales the INT8 core approximates FP attention of the dequantized operands;
    # a missing sqrt(dh), a swapped scale or a transposed operand breaks this by far more than 5%
    g = np.random.default_rng(7)
    B, S, nh, dh = 1, 32, 2, 16
    H = nh * dh
    qf, kf, vf = (g.standard_normal((B * S, H)) for _ in range(3))
    s_q, s_k, s_v = (np.abs(a).max() / 127 for a in (qf, kf, vf))
    qi, ki, vi = Q.quant_sq(qf, s_q), Q.quant_sq(kf, s_k), Q.quant_sq(vf, s_v)
    got = O.attention_int8(qi, ki, vi, B, S, nh, dh, s_q, s_k, s_v, 1.0 / 255, O.OutSpec("fp", dtype="f64")).data
    ref = O.attention_fp(qi * s_q, ki * s_k, vi * s_v, B, S, nh, dh, O.OutSpec("fp", dtype="f64")).data
    assert np.max(np.abs(got - ref)) / np.max(np.abs(ref)) < 0.05


def test_attention_int8_rowmax_variant_closed_forms_and_brute_force():
    """The row-max-normalised P quantizer (the long-sequence-robust variant): closed forms and a scalar re-derivation."""
    g = np.random.default_rng(70)
    # uniform logits: e = 1 for every key -> P~ = 255, l = S -> X_attn = s_v * mean(V), for ANY S (the static
    # quantizer rounds 1/S to zero beyond 510 keys)
    for S in (128, 640, 1024):
        nh, dh = 1, 8
        q = np.zeros((S, dh), np.int8)
        k = g.integers(-127, 128, (S, dh), dtype=np.int8)
        v = g.integers(-127, 128, (S, dh), dtype=np.int8)
        o, it = O.attention_int8(q, k, v, 1, S, nh, dh, 0.1, 0.1, 0.03, 1.0 / 255, O.OutSpec("fp", dtype="f64"),
                                 return_internals=True, p_mode="rowmax")
        assert np.all(it["P_u8"][(0, 0)] == 255)
        assert np.allclose(o.data, np.broadcast_to(0.03 * v.astype(np.float64).mean(0), o.data.shape), rtol=1e-13)
    stat = O.attention_int8(q, k, v, 1, S, nh, dh, 0.1, 0.1, 0.03, 1.0 / 255, O.OutSpec("fp", dtype="f64")).data
    assert not stat.any()                           # the paper-literal quantizer has lost all the mass at S = 1024
    # causal row 0 sees only key 0: P~ = [255, 0, ...], l = 1 -> X_attn[0] = s_v V[0]
    S, dh = 16, 8
    q, k, v = (g.integers(-127, 128, (S, dh), dtype=np.int8) for _ in range(3))
    o = O.attention_int8(q, k, v, 1, S, 1, dh, 0.05, 0.05, 0.02, 1.0, O.OutSpec("fp", dtype="f64"), mask="causal", p_mode="rowmax")
    assert np.allclose(o.data[0], 0.02 * v[0].astype(np.float64), rtol=1e-13)
    # scalar re-derivation, key lengths included
    S, nh, dh, klen = 12, 2, 4, 9
    q, k, v = (g.integers(-127, 128, (S, nh * dh), dtype=np.int8) for _ in range(3))
    s_q, s_k, s_v = 0.021, 0.017, 0.013
    o = O.attention_int8(q, k, v, 1, S, nh, dh, s_q, s_k, s_v, 1.0, O.OutSpec("fp", dtype="f64"), mask="causal",
                         key_len=np.array([klen]), p_mode="rowmax").data
    for i in range(S):
        for h in range(nh):
            keys = [j for j in range(S) if j <= i and j < klen]
            a = [s_q * s_k / math.sqrt(dh) * sum(int(q[i, h * dh + d]) * int(k[j, h * dh + d]) for d in range(dh)) for j in keys]
            m = max(a)
            e = [math.exp(x - m) for x in a]
            pu = [min(255, max(0, round(255 * x))) for x in e]          # no ties at these magnitudes
            for d in range(dh):
                want = s_v * sum(p_ * int(v[j, h * dh + d]) for p_, j in zip(pu, keys)) / (255 * sum(e))
                assert abs(o[i, h * dh + d] - want) <= 1e-12 * max(1.0, abs(want))


def test_attention_int8_rowmax_tracks_fp_attention_better_at_long_sequences():
    g = np.random.default_rng(71)
    B, S, nh, dh = 1, 768, 1, 16
    qf, kf, vf = (g.standard_normal((B * S, dh)) * c for c in (0.3, 0.3, 1.0))      # flat attention over many keys
    s_q, s_k, s_v = (np.abs(a).max() / 127 for a in (qf, kf, vf))
    qi, ki, vi = Q.quant_sq(qf, s_q), Q.quant_sq(kf, s_k), Q.quant_sq(vf, s_v)
    ref = O.attention_fp(qi * s_q, ki * s_k, vi * s_v, B, S, nh, dh, O.OutSpec("fp", dtype="f64")).data
    err = {}
    for mode in ("static", "rowmax"):
        got = O.attention_int8(qi, ki, vi, B, S, nh, dh, s_q, s_k, s_v, 1.0 / 255, O.OutSpec("fp", dtype="f64"), p_mode=mode).data
        err[mode] = np.max(np.abs(got - ref)) / np.max(np.abs(ref))
    assert err["rowmax"] < 0.02 and err["rowmax"] < 0.2 * err["static"], err


def test_fp8_variant_gemm_and_ln_against_plain_definitions():
    """FP8 GeMM^quant = the fp64 product of the dequantized e4m3 operands pushed through the same epilogue; the output
    quantizer is e4m3 rounding of v / S; LN^quant with an e4m3 TWQ output reconstructs the LayerNorm to 2^-4 relative."""
    g = np.random.default_rng(80)
    n, d, m = 9, 64, 12
    x = g.standard_normal((n, d)) * 2
    Wm = g.standard_normal((d, m)) * 0.05
    b = g.standard_normal(m) * 0.1
    xq = O.emit(x, O.OutSpec("twq", payload="f8"))
    assert xq.kind == "f8" and np.all(np.abs(xq.data).max(1) == 448.0)
    Wq, Sw = O.quant_weight_columnwise_f8(Wm)
    out = O.gemm_quant_f8(xq, Wq, Sw, b, "none", O.OutSpec("fp", dtype="f64"))
    ref = xq.real() @ (Wq * Sw[None, :]) + b
    assert np.allclose(out.data, ref, rtol=1e-13, atol=1e-13)
    # quantized output with a feature-wise scale: e4m3(v / S) exactly, including saturation
    S = np.abs(ref).max(0) / 448 / 2                       # half the needed range: the largest entries saturate
    o8 = O.gemm_quant_f8(xq, Wq, Sw, b, "none", O.OutSpec("fwq", scale=S, payload="f8"))
    assert np.array_equal(o8.data, Q.e4m3_round(ref / S[None, :])) and np.abs(o8.data).max() == 448.0
    # closeness to the un-quantized product: e4m3 keeps 4 significant bits per operand
    assert np.max(np.abs(out.data - (x @ Wm + b))) / np.max(np.abs(x @ Wm + b)) < 0.1
    # LN^quant -> e4m3 TWQ
    gam, bet = 1 + 0.1 * g.standard_normal(d), 0.1 * g.standard_normal(d)
    y, _ = O.ln_quant([O.fp_tensor(x, "f16")], gam, bet, 1e-5, O.OutSpec("twq", payload="f8"))
    ln = O.layernorm(O.fp_tensor(x, "f16").real(), gam, bet, 1e-5)
    big = np.abs(ln) > np.abs(ln).max(1, keepdims=True) * 2.0 ** -6
    assert np.all(np.abs(y.real() - ln)[big] <= np.abs(ln)[big] * 2.0 ** -4 * (1 + 1e-6))


def test_fp8_attention_closed_forms_and_closeness():
    g = np.random.default_rng(81)
    # uniform logits: P = 1/S, P_f8 = e4m3(448 / S) for every key -> X_attn = s_p s_v e4m3(1 / (S s_p)) * column sum of V
    S, dh = 96, 16
    q = np.zeros((S, dh))
    k = Q.e4m3_round(g.standard_normal((S, dh)) * 50)
    v = Q.e4m3_round(g.standard_normal((S, dh)) * 50)
    s_p = (1.0 / S) / 448
    o = O.attention_f8(q, k, v, 1, S, 1, dh, 0.01, 0.01, 0.02, s_p, O.OutSpec("fp", dtype="f64")).data
    assert np.allclose(o, np.broadcast_to(s_p * 0.02 * 448.0 * v.sum(0), o.shape), rtol=1e-13)
    # causal row 0 sees key 0 only: P = 1 -> saturates at 448 when s_p < 1 / 448 -> X_attn[0] = s_p s_v 448 V[0]
    q = Q.e4m3_round(g.standard_normal((S, dh)) * 50)
    o = O.attention_f8(q, k, v, 1, S, 1, dh, 0.01, 0.01, 0.02, 1.0 / 448, O.OutSpec("fp", dtype="f64"), mask="causal").data
    assert np.allclose(o[0], 0.02 * v[0], rtol=1e-13)
    o2 = O.attention_f8(q, k, v, 1, S, 1, dh, 0.01, 0.01, 0.02, 0.5 / 448, O.OutSpec("fp", dtype="f64"), mask="causal").data
    assert np.allclose(o2[0], 0.5 * 0.02 * v[0], rtol=1e-13)                    # clipped at 448: half the mass survives
    # close to FP attention of the dequantized operands (4 significant bits in P)
    qf, kf, vf = (g.standard_normal((64, 32)) for _ in range(3))
    s_q, s_k, s_v = (np.abs(a).max() / 448 for a in (qf, kf, vf))
    qi, ki, vi = Q.quant_f8(qf, s_q), Q.quant_f8(kf, s_k), Q.quant_f8(vf, s_v)
    got = O.attention_f8(qi, ki, vi, 1, 64, 2, 16, s_q, s_k, s_v, 1.0 / 448, O.OutSpec("fp", dtype="f64")).data
    ref = O.attention_fp(qi * s_q, ki * s_k, vi * s_v, 1, 64, 2, 16, O.OutSpec("fp", dtype="f64")).data
    assert np.max(np.abs(got - ref)) / np.max(np.abs(ref)) < 0.05


# ------------------------------------------------------------------ GeMM^quant
def test_gemm_quant_equals_fake_quant_path():
    # exact INT32 + scale epilogue == fp64 product of the dequantized operands (before rounding)
    g = np.random.default_rng(8)
    n, d, m = 9, 64, 12
    x = g.standard_normal((n, d)) * 2
    W = g.standard_normal((d, m)) * 0.02
    b = g.standard_normal(m) * 0.01
    xq, sx = Q.quant_twq(x)
    Wq, sw = Q.quant_weight_columnwise(W)
    o, acc = O.gemm_quant(O.QT("i8", xq, row_scale=sx), Wq, sw, b, "none", O.OutSpec("fp", dtype="f64"), return_acc=True)
    fake = (sx[:, None] * xq) @ (Wq * sw[None, :]) + b
    assert np.allclose(o.data, fake, rtol=1e-12, atol=1e-14)
    assert np.array_equal(acc, _brute(xq, Wq))
    # and the quantized product is close to the FP product (catches an axis mix-up of the scales)
    assert np.max(np.abs(fake - (x @ W + b))) / np.max(np.abs(x @ W + b)) < 0.03


def test_gemm_quant_epilogue_order_bias_then_act_then_quant():
    x = O.QT("i8", np.array([[10, -10]], np.int8), row_scale=np.array([0.5]))
    W = np.array([[1, 2], [3, -4]], np.int8)          # acc = [-20, 60]
    cs = np.array([0.1, 0.2])
    b = np.array([0.25, -1.0])
    v = np.array([[-20 * 0.5 * 0.1 + 0.25, 60 * 0.5 * 0.2 - 1.0]])     # [-0.75, 5.0]
    o = O.gemm_quant(x, W, cs, b, "gelu_erf", O.OutSpec("fwq", scale=np.array([0.01, 0.1])))
    want = Q.quant_sym(O.gelu_erf(v), np.array([[0.01, 0.1]]))
    assert np.array_equal(o.data, want) and int(o.data[0, 1]) == 50
    o = O.gemm_quant(x, W, cs, b, "none", O.OutSpec("round"))
    assert o.data.tolist() == [[-1, 5]]               # RNE(-0.75) = -1, RNE(5.0) = 5


# ------------------------------------------------------------------ LN^quant
def test_ln_quant_residual_sum_and_embedding_flavour():
    g = np.random.default_rng(9)
    n, H = 6, 32
    gamma, beta = 1 + 0.1 * g.standard_normal(H), 0.1 * g.standard_normal(H)
    xin, sin = Q.quant_twq(g.standard_normal((n, H)))
    so = np.abs(g.standard_normal(H)) * 0.01 + 0.01
    xo = g.integers(-127, 128, (n, H), dtype=np.int8)
    out, _ = O.ln_quant([O.QT("i8", xin, row_scale=sin), O.QT("i8", xo, col_scale=so)], gamma, beta, 1e-12,
                        O.OutSpec("twq"))
    r = sin[:, None] * xin + xo * so[None, :]                       # Eq. 19's two operands
    ref = torch.nn.functional.layer_norm(torch.from_numpy(r), (H,), torch.from_numpy(gamma),
                                         torch.from_numpy(beta), 1e-12).numpy()
    q, s = Q.quant_twq(ref)
    assert np.array_equal(out.data, q) and np.allclose(out.row_scale, s, rtol=1e-7)
    # embedding flavour == plain flavour on the explicitly gathered and summed input
    V, P, T, S = 11, 4, 2, 4
    tok = g.integers(-127, 128, (V, H), dtype=np.int8)
    ts = np.abs(g.standard_normal(V)) * 0.01 + 0.001
    pos = Q.round_to_storage(g.standard_normal((P, H)) * 0.02, "f16")
    typ = Q.round_to_storage(g.standard_normal((T, H)) * 0.02, "f16")
    ids = g.integers(0, V, 8)
    tids = g.integers(0, T, 8)
    e = O.embedding_ln_quant(ids, tids, tok, ts, pos, typ, S, gamma, beta, 1e-12, O.OutSpec("twq"))
    summed = ts[ids][:, None] * tok[ids] + pos[np.arange(8) % S] + typ[tids]
    q, s = Q.quant_twq(O.layernorm(summed, gamma, beta, 1e-12))
    assert np.array_equal(e.data, q) and np.array_equal(e.row_scale, s)


def test_ln_quant_fp_out_and_bare_add():
    g = np.random.default_rng(10)
    h = O.fp_tensor(g.standard_normal((4, 16)), "bf16")
    br = O.QT("i8", g.integers(-127, 128, (4, 16), dtype=np.int8), col_scale=np.full(16, 0.01))
    out, r = O.ln_quant([h, br], np.ones(16), np.zeros(16), 1e-5, O.OutSpec("twq"), fp_out_dtype="bf16")
    assert np.array_equal(r.data, Q.round_to_storage(h.data + br.real(), "bf16"))
    q, s = Q.quant_twq(O.layernorm(r.data, np.ones(16), np.zeros(16), 1e-5))
    assert np.array_equal(out.data, q)
    none, r2 = O.ln_quant([h, br], None, None, 0.0, None, fp_out_dtype="bf16", normalize=False)
    assert none is None and np.array_equal(r2.data, r.data)


@pytest.mark.parametrize("p_mode", ["static", "rowmax"])
def test_attention_int8_decode_is_the_last_causal_row_and_brute_force(p_mode):
    # a decode step at position t computes row t of the causal prefill over the first t + 1 tokens (the prefill is
    # pinned above); plus a pure-Python evaluation of the definition on one head
    g = np.random.default_rng(40)
    B, S, nh, dh = 3, 37, 2, 8
    H = nh * dh
    q = g.integers(-127, 128, (B * S, H), dtype=np.int8)
    k = g.integers(-127, 128, (B * S, H), dtype=np.int8)
    v = g.integers(-127, 128, (B * S, H), dtype=np.int8)
    s_q, s_k, s_v, s_p = 0.011, 0.013, 0.02, 1.0 / 255
    out = O.OutSpec("fp", dtype="f64")
    full = O.attention_int8(q, k, v, B, S, nh, dh, s_q, s_k, s_v, s_p, out, mask="causal", p_mode=p_mode).data
    kc, vc = k.reshape(B, S, H), v.reshape(B, S, H)
    lens = np.array([S, 1, 20])
    qd = np.stack([q[b * S + lens[b] - 1] for b in range(B)])
    got = O.attention_int8_decode(qd, kc, vc, lens, nh, dh, s_q, s_k, s_v, s_p, out, p_mode=p_mode).data
    for b in range(B):
        assert np.allclose(got[b], full[b * S + lens[b] - 1], rtol=1e-12, atol=1e-15), b
    # entries of the cache beyond lens[b] are never read
    kc2, vc2 = kc.copy(), vc.copy()
    kc2[2, 20:], vc2[2, 20:] = 99, -99
    got2 = O.attention_int8_decode(qd, kc2, vc2, lens, nh, dh, s_q, s_k, s_v, s_p, out, p_mode=p_mode).data
    assert np.array_equal(got, got2)
    # brute force, sequence 2 head 1
    import math
    b, h, L = 2, 1, 20
    A = [s_q * s_k / math.sqrt(dh) * sum(int(qd[b, h * dh + d]) * int(kc[b, t, h * dh + d]) for d in range(dh)) for t in range(L)]
    m = max(A)
    e = [math.exp(a - m) for a in A]
    l = sum(e)
    for d in range(dh):
        if p_mode == "static":
            acc = sum(min(255, max(0, round(e[t] / l / s_p))) * int(vc[b, t, h * dh + d]) for t in range(L))
            want = s_p * s_v * acc
        else:
            acc = sum(min(255, round(255 * e[t])) * int(vc[b, t, h * dh + d]) for t in range(L))
            want = s_v * acc / (255 * l)
        assert math.isclose(got[b, h * dh + d], want, rel_tol=1e-12, abs_tol=1e-15)
    # an empty sequence yields zeros; a single key yields that key's value row (P = 1 -> 255 s_p s_v V)
    z = O.attention_int8_decode(qd, kc, vc, np.array([0, 1, 1]), nh, dh, s_q, s_k, s_v, s_p, out, p_mode=p_mode).data
    assert np.all(z[0] == 0)
    assert np.allclose(z[1], s_v * vc[1, 0].astype(float), rtol=1e-12)
