"""Offline, host-side preparation for the W8A8 layer (paper Sec. 2.1, Eq. 2; Sec. 2.2.2, Eq. 20-23;
Sec. 2.2.3, Eq. 32; calibration as in Sec. 3): runs once per model, before inference, on the CPU.

Nothing here is on the hot path.  It turns FP master weights and calibration activations into what
libhero.so consumes: INT8 weights laid out [N][K] (the paper's column-major W[d, m]), one fp32 scale per
output column, folded fp32 biases, calibrated feature-wise / static activation scales and the epilogue
reciprocal vectors.  The arithmetic is float64 numpy.
"""
from dataclasses import dataclass, field
from typing import Dict

import numpy as np

MODULES = ("qkv", "attn", "attn_out", "fc1", "fc2")
PRESETS = {
    "M1": dict(qkv="int8", attn="fp", attn_out="fp", fc1="int8", fc2="fp"),
    "M2": dict(qkv="int8", attn="int8", attn_out="int8", fc1="int8", fc2="fp"),
    "M3": dict(qkv="int8", attn="int8", attn_out="int8", fc1="int8", fc2="int8"),
    "FP": dict(qkv="fp", attn="fp", attn_out="fp", fc1="fp", fc2="fp"),
}


@dataclass
class LayerConfig:
    B: int
    S: int
    H: int
    nh: int
    F: int
    arch: str = "post_ln"
    act: str = "gelu_erf"
    eps: float = 1e-12
    mask: str = "none"
    fp_dtype: str = "f16"
    mode: Dict[str, str] = field(default_factory=lambda: dict(PRESETS["M3"]))
    gran_in: str = "twq"
    gran_mid: str = "twq"
    gran_attn: str = "fwq"
    gran_out: str = "twq"
    p_mode: str = "static"          # P quantizer of the INT8 attention core: "static" (the paper) | "rowmax"
    payload: str = "i8"             # 8-bit type of the modules in "int8" mode: "i8" (the paper) | "f8" (e4m3 variant)

    @property
    def dh(self):
        return self.H // self.nh

    @property
    def M(self):
        return self.B * self.S


def _f32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64).astype(np.float32))


def scale_from_absmax(amax, qmax=127.0):
    """absmax / qmax with a zero statistic mapped to 1; fp32 (the storage type of every scale)."""
    amax = np.asarray(amax, dtype=np.float64)
    return np.where(amax > 0, amax / qmax, 1.0).astype(np.float32)


def quantize_columns(W):
    """Eq. 2 on W[d, m]: per-output-column symmetric INT8.  Returns (W_int8 laid out [m][d], S_w[m])."""
    W = np.asarray(W, dtype=np.float64)
    s = scale_from_absmax(np.abs(W).max(axis=0)).astype(np.float64)
    q = np.clip(np.rint(W / s[None, :]), -127, 127).astype(np.int8)
    return np.ascontiguousarray(q.T), s.astype(np.float32)


F8_MAX = 448.0          # largest finite e4m3 value


def e4m3_encode(x):
    """Saturating round-to-nearest-even of real values to e4m3 (4 exponent bits, bias 7, 3 mantissa bits, subnormals
    down to 2^-9, no infinities).  Returns (bytes uint8, values float64)."""
    x = np.clip(np.asarray(x, dtype=np.float64), -F8_MAX, F8_MAX)
    a = np.abs(x)
    _, ex = np.frexp(a)                                    # a = m * 2^ex, m in [0.5, 1)
    e = np.maximum(ex - 1, -6)                             # binade exponent; everything below 2^-6 is subnormal
    step = np.ldexp(1.0, e - 3)
    v = np.rint(a / step) * step                           # ties to even; may carry into the next binade
    _, ex = np.frexp(v)
    e = np.maximum(ex - 1, -6)
    normal = v >= 2.0 ** -6
    field = np.where(normal, e + 7, 0).astype(np.int64)
    mant = np.where(normal, np.rint((v / np.ldexp(1.0, e) - 1.0) * 8.0), np.rint(v * 512.0)).astype(np.int64)
    byte = (np.signbit(x).astype(np.int64) << 7) | (field << 3) | mant
    return byte.astype(np.uint8), np.copysign(v, x)


def quantize_columns_f8(W):
    """Eq. 2 with an e4m3 payload on W[d, m]: per-output-column scale absmax / 448.  Returns (bytes [m][d], S_w[m])."""
    W = np.asarray(W, dtype=np.float64)
    s = scale_from_absmax(np.abs(W).max(axis=0), F8_MAX).astype(np.float64)
    q, _ = e4m3_encode(W / s[None, :])
    return np.ascontiguousarray(q.T), s.astype(np.float32)


def fold_quantize(W, b, in_scale=None, out_scale=None, payload="i8"):
    """W~ = Diag(in_scale) W Diag(1 / out_scale), b~ = b / out_scale, then column-wise INT8 (fold first);
    payload "f8" quantizes the folded matrix to e4m3 instead."""
    W = np.asarray(W, dtype=np.float64)
    if in_scale is not None:
        W = W * np.asarray(in_scale, np.float64)[:, None]
    b = None if b is None else np.asarray(b, np.float64)
    if out_scale is not None:
        o = np.asarray(out_scale, np.float64)
        W = W / o[None, :]
        if b is not None:
            b = b / o
    Wq, s = quantize_columns_f8(W) if payload == "f8" else quantize_columns(W)
    return Wq, s, (None if b is None else _f32(b))


def _gelu(x, kind):
    if kind == "gelu_tanh":
        return 0.5 * x * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (x + 0.044715 * x ** 3)))
    from scipy.special import erf
    return 0.5 * x * (1.0 + erf(x / np.sqrt(2.0)))


def _ln(x, g, b, eps):
    mu = x.mean(-1, keepdims=True)
    c = x - mu
    return c / np.sqrt((c * c).mean(-1, keepdims=True) + eps) * g + b


def calibrate(cfg: LayerConfig, params, x_cal, n_seq, return_output=False):
    """Forward-only pass of the un-quantized layer over calibration data, recording absmax statistics
    (no truncation tuning).  `x_cal` is what enters the layer: for post-LN the tensor feeding QKV, for
    pre-LN the residual stream.  Returns the calibrated scales."""
    p = {k: np.asarray(v, np.float64) for k, v in params.items()}
    x = np.asarray(x_cal, np.float64)
    S, nh, dh, H = cfg.S, cfg.nh, cfg.dh, cfg.H
    stat = {}

    def attn(x_in):
        stat["in_f"], stat["in_t"] = np.abs(x_in).max(0), np.abs(x_in).max()
        q, k, v = (x_in @ p["W" + n] + p["b" + n] for n in "qkv")
        stat["q"], stat["k"], stat["v"] = (np.abs(t).max() for t in (q, k, v))
        xa = np.empty_like(q)
        pmax = 0.0
        causal = np.tril(np.ones((S, S), bool)) if cfg.mask == "causal" else None
        for b in range(n_seq):
            r = slice(b * S, (b + 1) * S)
            for h in range(nh):
                c = slice(h * dh, (h + 1) * dh)
                a = q[r, c] @ k[r, c].T / np.sqrt(dh)
                if causal is not None:
                    a = np.where(causal, a, -np.inf)
                e = np.exp(a - a.max(-1, keepdims=True))
                P = e / e.sum(-1, keepdims=True)
                pmax = max(pmax, float(P.max()))
                xa[r, c] = P @ v[r, c]
        stat["p"] = pmax
        stat["attn_f"], stat["attn_t"] = np.abs(xa).max(0), np.abs(xa).max()
        xo = xa @ p["Wo"] + p["bo"]
        stat["o"] = np.abs(xo).max(0)
        return xo

    def mlp(x_mid):
        stat["mid_f"], stat["mid_t"] = np.abs(x_mid).max(0), np.abs(x_mid).max()
        a = _gelu(x_mid @ p["W1"] + p["b1"], cfg.act)
        stat["a"] = np.abs(a).max(0)
        x2 = a @ p["W2"] + p["b2"]
        stat["x2"] = np.abs(x2).max(0)
        return x2

    if cfg.arch == "post_ln":
        xm = _ln(x + attn(x), p["ln1_g"], p["ln1_b"], cfg.eps)
        out = _ln(xm + mlp(xm), p["ln2_g"], p["ln2_b"], cfg.eps)
    else:
        h1 = x + attn(_ln(x, p["ln1_g"], p["ln1_b"], cfg.eps))
        out = h1 + mlp(_ln(h1, p["ln2_g"], p["ln2_b"], cfg.eps))
    stat["out_f"], stat["out_t"] = np.abs(out).max(0), np.abs(out).max()
    qmax, pmax = (F8_MAX, F8_MAX) if cfg.payload == "f8" else (127.0, 255.0)
    sc = lambda a, q=qmax: scale_from_absmax(a, q)
    scales = {
        "S_in_f": sc(stat["in_f"]), "S_in_t": float(sc(stat["in_t"])),
        "S_q": float(sc(stat["q"])), "S_k": float(sc(stat["k"])), "S_v": float(sc(stat["v"])),
        "S_p": float(sc(stat["p"], pmax)),
        "S_attn_f": sc(stat["attn_f"]), "S_attn_t": float(sc(stat["attn_t"])),
        "S_o": sc(stat["o"]),
        "S_mid_f": sc(stat["mid_f"]), "S_mid_t": float(sc(stat["mid_t"])),
        "S_a": sc(stat["a"]), "S_x2": sc(stat["x2"]),
        "S_out_f": sc(stat["out_f"]), "S_out_t": float(sc(stat["out_t"])),
    }
    return (scales, out) if return_output else scales


def _gran_vec(gran, S_f, S_t, n):
    if gran == "fwq":
        return np.asarray(S_f, np.float64)
    if gran == "sq":
        return np.full(n, float(S_t))
    return None


def _store_fp(W, fp_dtype):
    """FP-mode weights: [N][K] in the module's storage type (as uint16 bit patterns for bf16)."""
    Wt = np.ascontiguousarray(np.asarray(W, np.float32).T)
    if fp_dtype == "f16":
        return Wt.astype(np.float16)
    u = Wt.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return u.astype(np.uint16)          # bfloat16 bit patterns


def prepare_layer(cfg: LayerConfig, params, C, fold_quantize_fn=None):
    """Host arrays for one layer: per linear module {W, w_scale, bias, post_scale}, LN parameters, and the
    activation scales the kernels read.  `C` comes from `calibrate`.  `fold_quantize_fn(W, b, in_scale, out_scale)`
    replaces the host-side fold + Eq. 2 quantization (the device version lives in calibrate.py)."""
    if cfg.payload not in ("i8", "f8"):
        raise ValueError("payload %r" % (cfg.payload,))
    if cfg.payload == "f8":
        if cfg.p_mode != "static":
            raise ValueError("the e4m3 attention core has the static P quantizer only")
        if cfg.mode["attn"] != "int8" and cfg.mode["attn_out"] == "int8":
            raise ValueError("e4m3 payload: an FP attention core cannot feed an 8-bit attention-output linear")
        fq = fold_quantize_fn or (lambda W, b, i, o: fold_quantize(W, b, i, o, payload="f8"))
    else:
        fq = fold_quantize_fn or fold_quantize
    p = {k: np.asarray(v, np.float64) for k, v in params.items()}
    H, m = cfg.H, cfg.mode
    in_vec = _gran_vec(cfg.gran_in, C["S_in_f"], C["S_in_t"], H)
    mid_vec = _gran_vec(cfg.gran_mid, C["S_mid_f"], C["S_mid_t"], H)
    attn_vec = _gran_vec(cfg.gran_attn, C["S_attn_f"], C["S_attn_t"], H)
    if attn_vec is None:
        raise ValueError("X_attn must be FWQ or SQ")
    qkv_vec = np.concatenate([np.full(H, C["S_q"]), np.full(H, C["S_k"]), np.full(H, C["S_v"])]).astype(np.float64)
    L = {"cfg": cfg, "C": C}

    def linear(W, b, int8, in_scale, out_fold, post):
        g = {"int8": int8, "post_scale": None if post is None else _f32(post)}
        if int8:
            g["W"], g["w_scale"], g["bias"] = fq(W, b, in_scale, out_fold)
        else:
            g["W"], g["w_scale"], g["bias"] = _store_fp(W, cfg.fp_dtype), None, _f32(b)
        return g

    Wqkv = np.concatenate([p["Wq"], p["Wk"], p["Wv"]], axis=1)
    bqkv = np.concatenate([p["bq"], p["bk"], p["bv"]])
    attn8, o8, fc28 = m["attn"] == "int8", m["attn_out"] == "int8", m["fc2"] == "int8"
    if m["qkv"] == "int8":
        L["qkv"] = linear(Wqkv, bqkv, True, in_vec, qkv_vec if attn8 else None, None)
    else:
        L["qkv"] = linear(Wqkv, bqkv, False, None, None, (1.0 / qkv_vec) if attn8 else None)
    if o8:
        L["o"] = linear(p["Wo"], p["bo"], True, attn_vec, np.asarray(C["S_o"], np.float64), None)
    else:
        L["o"] = linear(p["Wo"], p["bo"], False, None, None, None)
    post_a = (1.0 / np.asarray(C["S_a"], np.float64)) if fc28 else None
    if m["fc1"] == "int8":
        L["fc1"] = linear(p["W1"], p["b1"], True, mid_vec, None, post_a)
    else:
        L["fc1"] = linear(p["W1"], p["b1"], False, None, None, post_a)
    if fc28:
        L["fc2"] = linear(p["W2"], p["b2"], True, np.asarray(C["S_a"], np.float64), np.asarray(C["S_x2"], np.float64), None)
    else:
        L["fc2"] = linear(p["W2"], p["b2"], False, None, None, None)
    for k in ("ln1_g", "ln1_b", "ln2_g", "ln2_b"):
        L[k] = _f32(p[k])
    L["s_in"] = None if in_vec is None else _f32(in_vec if cfg.gran_in == "fwq" else in_vec[:1])
    L["s_mid"] = None if mid_vec is None else _f32(mid_vec if cfg.gran_mid == "fwq" else mid_vec[:1])
    L["s_attn"] = _f32(attn_vec if cfg.gran_attn == "fwq" else attn_vec[:1])
    L["s_o"], L["s_x2"] = _f32(C["S_o"]), _f32(C["S_x2"])
    L["s_out"] = None
    if cfg.gran_out == "fwq":
        L["s_out"] = _f32(C["S_out_f"])
    elif cfg.gran_out == "sq":
        L["s_out"] = _f32([C["S_out_t"]])
    return L
