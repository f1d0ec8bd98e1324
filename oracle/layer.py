"""Offline preparation and the layer forward of Sec. 2.2-2.3 (oracle; test infrastructure only).

Master (FP) parameters use the paper's layout: a linear layer is Y = X W + b with W [d, m].
    params = {Wq, Wk, Wv, Wo: [H, H]; W1: [H, F]; W2: [F, H]; bq, bk, bv, bo, b2: [H]; b1: [F];
              ln1_g, ln1_b, ln2_g, ln2_b: [H]}
Post-LN (the paper's equations):  x_mid = LN1(x_in + Attn(x_in)),  x_out = LN2(x_mid + MLP(x_mid)).
Pre-LN (GPT-shaped; the paper names GPT but prints only post-LN equations, so this is a reading):
    h' = h + Attn(LN1(h)),  h'' = h' + MLP(LN2(h')), residual stream h kept in FP16/BF16.
"""
from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

from . import quant as Q
from .ops import (QT, OutSpec, fp_tensor, layernorm, ACTIVATIONS, softmax_masked, attention_mask,
                  ln_quant, gemm_quant, gemm_quant_f8, gemm_fp, attention_int8, attention_f8, attention_fp,
                  quant_weight_columnwise_f8)

MODULES = ("qkv", "attn", "attn_out", "fc1", "fc2")

# Table 1: which modules run INT8 under each preset (Embedding is INT8 in all three).
MODE_PRESETS = {
    "M1": dict(qkv="int8", attn="fp", attn_out="fp", fc1="int8", fc2="fp"),
    "M2": dict(qkv="int8", attn="int8", attn_out="int8", fc1="int8", fc2="fp"),
    "M3": dict(qkv="int8", attn="int8", attn_out="int8", fc1="int8", fc2="int8"),
    "FP": dict(qkv="fp", attn="fp", attn_out="fp", fc1="fp", fc2="fp"),
}


@dataclass
class LayerSpec:
    B: int
    S: int
    H: int
    nh: int
    F: int
    arch: str = "post_ln"            # 'post_ln' | 'pre_ln'
    act: str = "gelu_erf"
    eps: float = 1e-12
    mask: str = "none"               # 'none' | 'causal'
    fp_dtype: str = "f16"            # storage type of every FP tensor at a module border
    mode: Dict[str, str] = field(default_factory=lambda: dict(MODE_PRESETS["M3"]))
    gran_in: str = "twq"             # granularity of the INT8 tensor feeding QKV  (twq | fwq | sq)
    gran_mid: str = "twq"            # granularity of the INT8 tensor feeding FC1  (twq | fwq | sq)
    gran_attn: str = "fwq"           # granularity of X_attn                        (fwq | sq)
    gran_out: str = "twq"            # post-LN layer output: twq | fwq | sq | fp
    p_mode: str = "static"           # P quantizer of the INT8 attention core: 'static' (Eq. 16) | 'rowmax'
    payload: str = "i8"              # 8-bit type of the modules in 'int8' mode: 'i8' (the paper) | 'f8' (e4m3 variant)

    @property
    def dh(self):
        return self.H // self.nh

    @property
    def M(self):
        return self.B * self.S


# --------------------------------------------------------------------------------------
# un-quantized fp64 layer + calibration (Sec. 3: forward-only passes, absmax, no truncation tuning)
# --------------------------------------------------------------------------------------
def layer_fp64(spec: LayerSpec, params, x, B=None):
    """The textbook layer (Eq. 8-13, 24-27) in fp64 with no rounding anywhere.  Returns every
    intermediate named in the paper.  `x` is [B*S, H]."""
    p = {k: np.asarray(v, np.float64) for k, v in params.items()}
    B = spec.B if B is None else B
    S, nh, dh, H = spec.S, spec.nh, spec.dh, spec.H
    t = {}
    act = ACTIVATIONS[spec.act]

    def attn_block(x_in):
        t["x_in"] = x_in
        q = x_in @ p["Wq"] + p["bq"]
        k = x_in @ p["Wk"] + p["bk"]
        v = x_in @ p["Wv"] + p["bv"]
        t["q"], t["k"], t["v"] = q, k, v
        xa = np.zeros_like(q)
        pmax = 0.0
        allowed = attention_mask(S, spec.mask)
        for b in range(B):
            rows = slice(b * S, (b + 1) * S)
            for h in range(nh):
                cols = slice(h * dh, (h + 1) * dh)
                P = softmax_masked(q[rows, cols] @ k[rows, cols].T / np.sqrt(float(dh)), allowed)
                pmax = max(pmax, float(P.max()))
                xa[rows, cols] = P @ v[rows, cols]
        t["p_max"] = pmax
        t["x_attn"] = xa
        t["x_o"] = xa @ p["Wo"] + p["bo"]
        return t["x_o"]

    def mlp_block(x_mid):
        t["x_mid"] = x_mid
        t["x_1"] = x_mid @ p["W1"] + p["b1"]
        t["a"] = act(t["x_1"])
        t["x_2"] = t["a"] @ p["W2"] + p["b2"]
        return t["x_2"]

    x = np.asarray(x, np.float64)
    if spec.arch == "post_ln":
        x_o = attn_block(x)
        x_mid = layernorm(x + x_o, p["ln1_g"], p["ln1_b"], spec.eps)
        x_2 = mlp_block(x_mid)
        t["x_out"] = layernorm(x_mid + x_2, p["ln2_g"], p["ln2_b"], spec.eps)
    else:
        x_o = attn_block(layernorm(x, p["ln1_g"], p["ln1_b"], spec.eps))
        h1 = x + x_o
        x_2 = mlp_block(layernorm(h1, p["ln2_g"], p["ln2_b"], spec.eps))
        t["x_out"] = h1 + x_2
    return t


def calibrate(spec: LayerSpec, params, x_cal, B_cal):
    """Static scales from absmax statistics of the un-quantized forward on calibration data.

    Per-feature (FWQ) scales are vectors, per-tensor (SQ) scales are scalars; S_p = max P / 255.
    """
    t = layer_fp64(spec, params, x_cal, B=B_cal)
    am_f = lambda a: np.max(np.abs(a), axis=0)
    am_t = lambda a: np.max(np.abs(a))
    f8 = spec.payload == "f8"
    cs = (lambda a: Q.calib_scale(a, Q.F8MAX)) if f8 else Q.calib_scale       # absmax / 448 for an e4m3 payload
    return {
        "S_in_f": cs(am_f(t["x_in"])), "S_in_t": float(cs(am_t(t["x_in"]))),
        "S_q": float(cs(am_t(t["q"]))), "S_k": float(cs(am_t(t["k"]))),
        "S_v": float(cs(am_t(t["v"]))),
        "S_p": float(Q.calib_scale(t["p_max"], Q.F8MAX if f8 else Q.PMAX)),
        "S_attn_f": cs(am_f(t["x_attn"])), "S_attn_t": float(cs(am_t(t["x_attn"]))),
        "S_o": cs(am_f(t["x_o"])),
        "S_mid_f": cs(am_f(t["x_mid"])), "S_mid_t": float(cs(am_t(t["x_mid"]))),
        "S_a": cs(am_f(t["a"])),
        "S_x2": cs(am_f(t["x_2"])),
        "S_out_f": cs(am_f(t["x_out"])), "S_out_t": float(cs(am_t(t["x_out"]))),
    }


# --------------------------------------------------------------------------------------
# folding + weight quantization (Eq. 20-23, 32)
# --------------------------------------------------------------------------------------
def _vec(gran, S_f, S_t, n):
    """The per-feature scale vector an INT8 tensor of granularity `gran` carries (None for TWQ)."""
    if gran == "fwq":
        return np.asarray(S_f, np.float64)
    if gran == "sq":
        return np.full(n, float(S_t))
    return None


def fold_and_quantize(W, b, in_scale=None, out_scale=None, payload="i8"):
    """W~ = Diag(in_scale) W Diag(1/out_scale), b~ = b / out_scale, then Eq. 2 column-wise INT8.

    in_scale : FWQ/SQ scale vector of the GEMM's INT8 input (consumer-side fold, Eq. 23, 32)
    out_scale: FWQ/SQ scale vector of the GEMM's INT8 output (producer-side fold, Eq. 20-21),
               after which the output quantizer is a bare Round (Eq. 22).
    The fold precedes quantization: the INT8 weights of the folded matrix are what is stored.
    """
    W = np.asarray(W, np.float64).copy()
    b = None if b is None else np.asarray(b, np.float64).copy()
    if in_scale is not None:
        W = np.asarray(in_scale, np.float64)[:, None] * W
    if out_scale is not None:
        W = W / np.asarray(out_scale, np.float64)[None, :]
        if b is not None:
            b = b / np.asarray(out_scale, np.float64)[None, :].reshape(-1)
    if payload == "f8":
        W_i8, S_w = quant_weight_columnwise_f8(W)           # e4m3 values, scales absmax / 448
    else:
        W_i8, S_w = Q.quant_weight_columnwise(W)
    if b is not None:
        b = b.astype(np.float32).astype(np.float64)     # biases are stored in fp32
    return W_i8, S_w, b


def prepare_layer(spec: LayerSpec, params, C):
    """Everything the forward needs besides activations: INT8 (or FP-stored) weights, column
    scales, folded biases and the output stage of every operator, from master parameters and the
    calibrated scales C.  The rule for types: a producer emits what its consumer's mode needs
    (Table 1); an INT8 module always contracts INT8 x INT8 whatever it emits."""
    p = {k: np.asarray(v, np.float64) for k, v in params.items()}
    H, F, m, fd = spec.H, spec.F, spec.mode, spec.fp_dtype
    for k in MODULES:
        assert m[k] in ("int8", "fp")
    L = {"spec": spec, "C": C}
    pay = spec.payload
    assert pay in ("i8", "f8")
    assert pay == "i8" or spec.p_mode == "static", "the e4m3 attention core has the static P quantizer only"

    def out_spec(kind, **kw):                                   # every 8-bit output stage of the layer carries the payload
        return OutSpec(kind, payload=pay, **kw)

    def fold_and_quantize_(W, b, i, o):
        return fold_and_quantize(W, b, i, o, payload=pay)
    fpW = lambda W: Q.round_to_storage(W, fd)
    f32 = lambda b: np.asarray(b, np.float64).astype(np.float32).astype(np.float64)

    in_vec = _vec(spec.gran_in, C["S_in_f"], C["S_in_t"], H)
    mid_vec = _vec(spec.gran_mid, C["S_mid_f"], C["S_mid_t"], H)
    attn_vec = _vec(spec.gran_attn, C["S_attn_f"], C["S_attn_t"], H)
    assert attn_vec is not None, "X_attn is FWQ or SQ (a GEMM epilogue cannot do TWQ, Sec. 2.1)"
    qkv_vec = np.concatenate([np.full(H, C["S_q"]), np.full(H, C["S_k"]), np.full(H, C["S_v"])])

    # what the LN feeding QKV / FC1 must emit
    def ln_spec(mode, gran, S_f, S_t):
        if mode == "fp":
            return out_spec("fp", dtype=fd)
        return {"twq": out_spec("twq"), "fwq": out_spec("fwq", scale=S_f), "sq": out_spec("sq", scale=S_t)}[gran]

    L["ln_in_out"] = ln_spec(m["qkv"], spec.gran_in, C["S_in_f"], C["S_in_t"])
    L["ln_mid_out"] = ln_spec(m["fc1"], spec.gran_mid, C["S_mid_f"], C["S_mid_t"])
    L["ln_final_out"] = (out_spec("fp", dtype=fd) if spec.gran_out == "fp" else
                         ln_spec("int8", spec.gran_out, C["S_out_f"], C["S_out_t"]))

    # QKV (Eq. 14, 20-22)
    Wqkv = np.concatenate([p["Wq"], p["Wk"], p["Wv"]], axis=1)
    bqkv = np.concatenate([p["bq"], p["bk"], p["bv"]])
    g = {"mode": m["qkv"]}
    if m["qkv"] == "int8":
        out_fold = qkv_vec if m["attn"] == "int8" else None
        g["W_i8"], g["cs"], g["bias"] = fold_and_quantize_(Wqkv, bqkv, in_vec, out_fold)
        g["out"] = out_spec("round") if m["attn"] == "int8" else out_spec("fp", dtype=fd)
        g["carried"] = out_fold
    else:
        g["W"], g["bias"] = fpW(Wqkv), f32(bqkv)
        g["out"] = out_spec("fwq", scale=qkv_vec) if m["attn"] == "int8" else out_spec("fp", dtype=fd)
        g["carried"] = None
    L["qkv"] = g

    # attention output stage (Eq. 17): INT8 FWQ/SQ when the attention-output linear is INT8
    if m["attn_out"] == "int8":
        L["attn_out_spec"] = (out_spec("fwq", scale=C["S_attn_f"]) if spec.gran_attn == "fwq"
                              else out_spec("sq", scale=C["S_attn_t"]))
    else:
        L["attn_out_spec"] = out_spec("fp", dtype=fd)

    # attention-output linear (Eq. 18, 23)
    g = {"mode": m["attn_out"]}
    if m["attn_out"] == "int8":
        g["W_i8"], g["cs"], g["bias"] = fold_and_quantize_(p["Wo"], p["bo"], attn_vec, C["S_o"])
        g["out"], g["carried"] = out_spec("round"), np.asarray(C["S_o"], np.float64)
    else:
        g["W"], g["bias"] = fpW(p["Wo"]), f32(p["bo"])
        g["out"], g["carried"] = out_spec("fp", dtype=fd), None
    L["o"] = g

    # FC1 + GELU^quant (Eq. 28-29): X_1 is never quantized; A is FWQ when FC2 is INT8
    g = {"mode": m["fc1"]}
    a_spec = out_spec("fwq", scale=C["S_a"]) if m["fc2"] == "int8" else out_spec("fp", dtype=fd)
    if m["fc1"] == "int8":
        g["W_i8"], g["cs"], g["bias"] = fold_and_quantize_(p["W1"], p["b1"], mid_vec, None)
    else:
        g["W"], g["bias"] = fpW(p["W1"]), f32(p["b1"])
    g["out"], g["carried"] = a_spec, None
    L["fc1"] = g

    # FC2 (Eq. 30, 32)
    g = {"mode": m["fc2"]}
    if m["fc2"] == "int8":
        g["W_i8"], g["cs"], g["bias"] = fold_and_quantize_(p["W2"], p["b2"], C["S_a"], C["S_x2"])
        g["out"], g["carried"] = out_spec("round"), np.asarray(C["S_x2"], np.float64)
    else:
        g["W"], g["bias"] = fpW(p["W2"]), f32(p["b2"])
        g["out"], g["carried"] = out_spec("fp", dtype=fd), None
    L["fc2"] = g

    for k in ("ln1_g", "ln1_b", "ln2_g", "ln2_b"):
        L[k] = f32(p[k])
    return L


# --------------------------------------------------------------------------------------
# forward
# --------------------------------------------------------------------------------------
def _linear(g, x: QT, act, return_acc=False):
    if g["mode"] == "int8" and x.kind == "f8":
        o = gemm_quant_f8(x, g["W_i8"], g["cs"], g["bias"], act, g["out"], g["carried"])
        return (o, None) if return_acc else o
    if g["mode"] == "int8":
        return gemm_quant(x, g["W_i8"], g["cs"], g["bias"], act, g["out"], g["carried"], return_acc=return_acc)
    o = gemm_fp(x, g["W"], g["bias"], act, g["out"], g["carried"])
    return (o, None) if return_acc else o


def _attention(L, qkv: QT, B):
    spec, C = L["spec"], L["C"]
    H = spec.H
    if spec.mode["attn"] == "int8" and spec.payload == "f8":
        assert qkv.kind == "f8" and spec.p_mode == "static"
        d = qkv.data
        return attention_f8(d[:, :H], d[:, H:2 * H], d[:, 2 * H:], B, spec.S, spec.nh, spec.dh,
                            C["S_q"], C["S_k"], C["S_v"], C["S_p"], L["attn_out_spec"], mask=spec.mask)
    if spec.mode["attn"] == "int8":
        assert qkv.kind == "i8"
        d = qkv.data
        return attention_int8(d[:, :H], d[:, H:2 * H], d[:, 2 * H:], B, spec.S, spec.nh, spec.dh,
                              C["S_q"], C["S_k"], C["S_v"], C["S_p"], L["attn_out_spec"], mask=spec.mask,
                              p_mode=spec.p_mode)
    assert qkv.kind == "fp"
    d = qkv.real()
    return attention_fp(d[:, :H], d[:, H:2 * H], d[:, 2 * H:], B, spec.S, spec.nh, spec.dh,
                        L["attn_out_spec"], mask=spec.mask)


def layer_forward(L, x: QT, B=None, pending: Optional[QT] = None):
    """One layer on `x` ([B*S, H]); returns a dict of every tensor at an operator border
    (QT objects) plus the INT32 accumulators of the INT8 GEMMs.

    post_ln: x is the layer input X_in (INT8 TWQ/FWQ/SQ, or FP); result key 'x_out'.
    pre_ln : x is the FP residual stream h; `pending` is an optional branch still to be added to
             it (the previous layer's X_2, added inside LN1's kernel); result keys 'h_mid', 'x_2'
             and 'h_out' = h_mid + X_2 (the lone-layer closing add).
    """
    spec = L["spec"]
    B = spec.B if B is None else B
    T = {}
    if spec.arch == "post_ln":
        T["x_in"] = x
        T["qkv"], T["acc_qkv"] = _linear(L["qkv"], x, "none", return_acc=True)
        T["x_attn"] = _attention(L, T["qkv"], B)
        T["x_o"], T["acc_o"] = _linear(L["o"], T["x_attn"], "none", return_acc=True)
        T["x_mid"], _ = ln_quant([x, T["x_o"]], L["ln1_g"], L["ln1_b"], spec.eps, L["ln_mid_out"])
        T["a"], T["acc_fc1"] = _linear(L["fc1"], T["x_mid"], spec.act, return_acc=True)
        T["x_2"], T["acc_fc2"] = _linear(L["fc2"], T["a"], "none", return_acc=True)
        T["x_out"], _ = ln_quant([T["x_mid"], T["x_2"]], L["ln2_g"], L["ln2_b"], spec.eps, L["ln_final_out"])
    else:
        fd = spec.fp_dtype
        ins = [x] if pending is None else [x, pending]
        T["x_in"], h0 = ln_quant(ins, L["ln1_g"], L["ln1_b"], spec.eps, L["ln_in_out"],
                                 fp_out_dtype=None if pending is None else fd)
        T["h_in"] = x if h0 is None else h0
        T["qkv"], T["acc_qkv"] = _linear(L["qkv"], T["x_in"], "none", return_acc=True)
        T["x_attn"] = _attention(L, T["qkv"], B)
        T["x_o"], T["acc_o"] = _linear(L["o"], T["x_attn"], "none", return_acc=True)
        T["x_mid"], T["h_mid"] = ln_quant([T["h_in"], T["x_o"]], L["ln2_g"], L["ln2_b"], spec.eps,
                                          L["ln_mid_out"], fp_out_dtype=fd)
        T["a"], T["acc_fc1"] = _linear(L["fc1"], T["x_mid"], spec.act, return_acc=True)
        T["x_2"], T["acc_fc2"] = _linear(L["fc2"], T["a"], "none", return_acc=True)
        _, T["h_out"] = ln_quant([T["h_mid"], T["x_2"]], None, None, spec.eps, None, fp_out_dtype=fd,
                                 normalize=False)
        T["x_out"] = T["h_out"]
    return T


def entry_ln(x_fp: QT, gamma, beta, eps, out: OutSpec):
    """The entry LN^quant that turns an FP16 activation into the layer's INT8 input (the role the
    embedding LayerNorm plays in Eq. 6-7 for a lone layer fed FP activations)."""
    return ln_quant([x_fp], gamma, beta, eps, out)[0]
