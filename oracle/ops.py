"""Quantization-aware operators of Sec. 2.2 in fp64 / exact integers (oracle; test infrastructure only).

Every real-valued step is fp64; every integer contraction is exact.  Nothing here is blocked,
fused or reordered beyond what the equations state.
"""
from dataclasses import dataclass
from typing import Optional

import numpy as np
from scipy.special import erf as _erf

from . import quant as Q


# --------------------------------------------------------------------------------------
# tensors at operator borders
# --------------------------------------------------------------------------------------
@dataclass
class QT:
    """A tensor at an operator border: INT8 payload + scale (Eq. 3-5), or an FP tensor.

    kind 'i8': data int8 [n, d]; row_scale [n] (TWQ) and/or col_scale [d] (FWQ; SQ is a
               constant vector) give the real value row_scale[i] * data[i, j] * col_scale[j].
    kind 'f8': the same with an e4m3 payload (FP8 variant): data holds the e4m3 VALUES in fp64.
    kind 'fp': data fp64 holding values already rounded to the storage grid `dtype`.
    """
    kind: str
    data: np.ndarray
    row_scale: Optional[np.ndarray] = None
    col_scale: Optional[np.ndarray] = None
    dtype: str = "f16"

    def real(self):
        if self.kind == "fp":
            return np.asarray(self.data, dtype=np.float64)
        return Q.dequant(self.data, self.row_scale, self.col_scale)


def fp_tensor(x, dtype):
    return QT("fp", Q.round_to_storage(x, dtype), dtype=dtype)


# --------------------------------------------------------------------------------------
# plain definitions
# --------------------------------------------------------------------------------------
def int_matmul(A, B):
    """Exact integer product A[n, d] @ B[d, m] of 8-bit operands, returned as int64.

    The contraction runs through the fp64 matrix product: every partial sum is an integer of
    magnitude < d * 255 * 127 << 2^53, so each fp64 operation is exact whatever the summation
    order.  The result must fit INT32 (the accumulator type of the method).
    """
    A = np.asarray(A)
    B = np.asarray(B)
    assert A.dtype in (np.int8, np.uint8) and B.dtype in (np.int8, np.uint8)
    assert A.shape[1] * 255 * 127 < 2 ** 31, "INT32 accumulator would overflow"
    acc = A.astype(np.float64) @ B.astype(np.float64)
    out = acc.astype(np.int64)
    assert np.array_equal(out.astype(np.float64), acc)
    return out


def layernorm(r, gamma, beta, eps):
    """LN over the last axis: (r - mean) / sqrt(biased variance + eps) * gamma + beta, two-pass."""
    r = np.asarray(r, dtype=np.float64)
    mu = np.mean(r, axis=-1, keepdims=True)
    c = r - mu
    var = np.mean(c * c, axis=-1, keepdims=True)
    return c / np.sqrt(var + eps) * np.asarray(gamma, np.float64) + np.asarray(beta, np.float64)


def gelu_erf(x):
    x = np.asarray(x, dtype=np.float64)
    return x * 0.5 * (1.0 + _erf(x / np.sqrt(2.0)))


def gelu_tanh(x):
    x = np.asarray(x, dtype=np.float64)
    return 0.5 * x * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (x + 0.044715 * x ** 3)))


ACTIVATIONS = {"none": lambda x: np.asarray(x, dtype=np.float64), "gelu_erf": gelu_erf, "gelu_tanh": gelu_tanh}


def softmax_masked(A, allowed):
    """Row softmax over the allowed keys; masked entries are exactly 0; a fully masked row is 0."""
    A = np.asarray(A, dtype=np.float64)
    neg = np.where(allowed, A, -np.inf)
    m = np.max(neg, axis=-1, keepdims=True)
    m = np.where(np.isfinite(m), m, 0.0)
    e = np.where(allowed, np.exp(neg - m), 0.0)
    s = np.sum(e, axis=-1, keepdims=True)
    return np.where(s > 0.0, e / np.where(s > 0.0, s, 1.0), 0.0)


def attention_mask(S, kind="none", key_len=None):
    """allowed[i, k] for one sequence: 'none', 'causal' (k <= i), optionally k < key_len."""
    allowed = np.ones((S, S), dtype=bool)
    if kind == "causal":
        allowed &= np.tril(np.ones((S, S), dtype=bool))
    elif kind != "none":
        raise ValueError(kind)
    if key_len is not None:
        allowed &= (np.arange(S)[None, :] < int(key_len))
    return allowed


# --------------------------------------------------------------------------------------
# output stage shared by the operators: what the consumer wants decides the type
# --------------------------------------------------------------------------------------
@dataclass
class OutSpec:
    """How an operator's real-valued result leaves it.

    kind 'twq'  : INT8 + per-row scale computed on the fly (only legal for LN^quant, Sec. 2.1)
    kind 'fwq'  : INT8 with the given per-feature scale [d]   (Eq. 4)
    kind 'sq'   : INT8 with the given scalar scale            (Eq. 5)
    kind 'round': INT8 = clip(Round(v)); the scale was folded into the producer (Eq. 20-22)
    kind 'fp'   : stored in `dtype` ('f16' / 'bf16' / 'f32')
    payload 'f8' (FP8 variant): the same kinds with an e4m3 payload instead of INT8; a scale computed on the fly is
    absmax / 448 and the quantizer is the saturating e4m3 rounding instead of clip(Round(.)).
    """
    kind: str
    scale: Optional[np.ndarray] = None
    dtype: str = "f16"
    payload: str = "i8"


def emit(v, spec: OutSpec, carried_col_scale=None):
    """Apply the output stage.  `carried_col_scale` is the scale vector the INT8 result stands
    for when it was folded away upstream (kind 'round')."""
    if spec.kind == "fp":
        return fp_tensor(v, spec.dtype)
    if spec.payload == "f8":
        v = np.asarray(v, dtype=np.float64)
        if spec.kind == "twq":
            s = Q.f8_scale(np.max(np.abs(v), axis=1))
            return QT("f8", Q.quant_f8(v, s[:, None]), row_scale=s)
        if spec.kind == "fwq":
            s = np.asarray(spec.scale, dtype=np.float64).reshape(-1)
            return QT("f8", Q.quant_f8(v, s[None, :]), col_scale=s)
        if spec.kind == "sq":
            s = float(np.asarray(spec.scale).reshape(()))
            return QT("f8", Q.quant_f8(v, s), col_scale=np.full(v.shape[1], s))
        if spec.kind == "round":
            return QT("f8", Q.quant_f8(v, 1.0), col_scale=carried_col_scale)
        raise ValueError(spec.kind)
    if spec.kind == "twq":
        q, s = Q.quant_twq(v)
        return QT("i8", q, row_scale=s)
    if spec.kind == "fwq":
        s = np.asarray(spec.scale, dtype=np.float64).reshape(-1)
        return QT("i8", Q.quant_fwq(v, s), col_scale=s)
    if spec.kind == "sq":
        s = float(np.asarray(spec.scale).reshape(()))
        return QT("i8", Q.quant_sq(v, s), col_scale=np.full(v.shape[1], s))
    if spec.kind == "round":
        return QT("i8", Q.quant_sym(v, 1.0), col_scale=carried_col_scale)
    raise ValueError(spec.kind)


# --------------------------------------------------------------------------------------
# LN^quant (Eq. 7, Eq. 19, Eq. 31)
# --------------------------------------------------------------------------------------
def ln_quant(inputs, gamma, beta, eps, out: OutSpec, fp_out_dtype=None, normalize=True):
    """LN^quant: LayerNorm of the SUM of its inputs (each a QT), then the output quantizer.

    Returns (out QT or None, r QT or None) where r is the pre-LN sum stored in `fp_out_dtype`
    (the FP residual stream of a pre-LN layer).  When r is stored, the normalisation reads the
    stored (rounded) value, since that is the tensor the layer carries on.
    normalize=False gives the bare residual add (last add of a lone pre-LN layer).
    """
    r = sum(t.real() for t in inputs)
    r_t = None
    if fp_out_dtype is not None:
        r_t = fp_tensor(r, fp_out_dtype)
        r = r_t.real()
    if not normalize:
        return None, r_t
    y = layernorm(r, gamma, beta, eps)
    return emit(y, out), r_t


def embedding_ln_quant(ids, type_ids, tok_i8, tok_scale, pos_table, type_table, S, gamma, beta, eps, out):
    """Eq. 7: S_emb X_emb,int8 = LN^quant(S_xt X_t,int8, X_p, X_s).

    tok_i8 [V, H] int8 with per-row scale tok_scale [V] (TWQ table); pos_table [P, H] and
    type_table [T, H] hold FP16 values; token i sits at position i mod S.
    """
    ids = np.asarray(ids).reshape(-1)
    pos = np.arange(ids.size) % S
    x_t = QT("i8", tok_i8[ids], row_scale=np.asarray(tok_scale, np.float64)[ids])
    x_p = fp_tensor(np.asarray(pos_table, np.float64)[pos], "f16")
    x_s = fp_tensor(np.asarray(type_table, np.float64)[np.asarray(type_ids).reshape(-1)], "f16")
    return ln_quant([x_t, x_p, x_s], gamma, beta, eps, out)[0]


# --------------------------------------------------------------------------------------
# GeMM^quant (Eq. 14/18/22/28-30) and its FP counterpart
# --------------------------------------------------------------------------------------
def gemm_quant(x: QT, W_i8, col_scale, bias, act, out: OutSpec, carried=None, return_acc=False):
    """INT8 GEMM with the fused epilogue.

    acc = X_int8 W_int8                      exact INT32                      (Eq. 1-2)
    v   = acc * rs[i] * cs[j] + b[j]         rs = TWQ row scale of X or 1     (Eq. 14, 22)
    a   = act(v)                             GELU for FC1                     (Eq. 29)
    out = emit(a)                            Round only when the scale is folded (Eq. 22), else
                                             the FWQ / SQ quantizer (GELU^quant) or an FP store

    W_i8 is [d, m] (the paper's layout), col_scale/bias [m].  A feature-wise/static scale of X
    never appears here: it was folded into the rows of W before quantization (Eq. 23, 32).
    """
    assert x.kind == "i8"
    acc = int_matmul(x.data, W_i8)
    v = acc.astype(np.float64)
    if x.row_scale is not None:
        v = v * np.asarray(x.row_scale, np.float64)[:, None]
    v = v * np.asarray(col_scale, np.float64)[None, :]
    if bias is not None:
        v = v + np.asarray(bias, np.float64)[None, :]
    a = ACTIVATIONS[act](v)
    o = emit(a, out, carried)
    return (o, acc) if return_acc else o


def gemm_quant_f8(x: QT, W_f8, col_scale, bias, act, out: OutSpec, carried=None):
    """The FP8 variant of GeMM^quant: e4m3 operands, the same epilogue.

    acc = X_f8 W_f8 (every product of two e4m3 values and every partial sum is exact in fp64 for d <= 2^17),
    v = acc * rs[i] * cs[j] + b[j], a = act(v), out = emit(a).  W_f8 [d, m] holds e4m3 values, col_scale [m] the
    column scales of Eq. 2 taken with 448 in place of 127.
    """
    assert x.kind == "f8"
    assert x.data.shape[1] <= 2 ** 17
    acc = np.asarray(x.data, np.float64) @ np.asarray(W_f8, np.float64)
    v = acc
    if x.row_scale is not None:
        v = v * np.asarray(x.row_scale, np.float64)[:, None]
    v = v * np.asarray(col_scale, np.float64)[None, :]
    if bias is not None:
        v = v + np.asarray(bias, np.float64)[None, :]
    return emit(ACTIVATIONS[act](v), out, carried)


def quant_weight_columnwise_f8(W):
    """Eq. 2 with an e4m3 payload: per-output-column scale absmax / 448.  Returns (e4m3 values [d, m], S_w [m])."""
    W = np.asarray(W, dtype=np.float64)
    S_w = Q.f8_scale(np.max(np.abs(W), axis=0))
    return Q.quant_f8(W, S_w[None, :]), S_w


def gemm_fp(x: QT, W, bias, act, out: OutSpec, carried=None):
    """FP-mode linear (Table 1, a module left in FP16/BF16): textbook X W + b in fp64 on the
    stored operands, then the same output stage."""
    assert x.kind == "fp"
    v = x.real() @ np.asarray(W, np.float64)
    if bias is not None:
        v = v + np.asarray(bias, np.float64)[None, :]
    a = ACTIVATIONS[act](v)
    return emit(a, out, carried)


# --------------------------------------------------------------------------------------
# attention core (Eq. 15-17)
# --------------------------------------------------------------------------------------
def attention_int8(q_i8, k_i8, v_i8, B, S, nh, dh, s_q, s_k, s_v, s_p, out: OutSpec,
                   mask="none", key_len=None, return_internals=False, p_mode="static"):
    """INT8 attention.  q_i8/k_i8/v_i8: [B*S, nh*dh] int8 (SQ, scalar scales s_q, s_k, s_v).

    per (b, h):  A = d~ (Q K^T),  d~ = s_q s_k / sqrt(dh)   -- never quantized
                 P = softmax(A) over the allowed keys
                 P_u8 = clip(Round(P / s_p), 0, 255)       -- asymmetric (unsigned) INT8
                 acc = P_u8 V_int8                          -- exact INT32
                 X_attn = s_p s_v acc                       -> output stage (FWQ / SQ / FP)

    p_mode="rowmax" (not in the paper; the long-sequence-robust variant): the un-normalised probabilities are
    quantized against their row maximum instead of the normalised ones against a static scale,
                 e = exp(A - max_row A) over the allowed keys (masked: 0),   l = sum_row e
                 P~_u8 = clip(Round(255 e), 0, 255)        -- the largest key of every row gets 255
                 acc = P~_u8 V_int8,   X_attn = s_v acc / (255 l)
    so nothing underflows however many keys share the mass; s_p is unused.
    """
    assert p_mode in ("static", "rowmax")
    H = nh * dh
    d_tilde = float(s_q) * float(s_k) / np.sqrt(float(dh))
    x_attn = np.zeros((B * S, H), dtype=np.float64)
    internals = {"P_u8": {}, "acc": {}}
    for b in range(B):
        allowed = attention_mask(S, mask, None if key_len is None else key_len[b])
        rows = slice(b * S, (b + 1) * S)
        for h in range(nh):
            cols = slice(h * dh, (h + 1) * dh)
            A = d_tilde * int_matmul(q_i8[rows, cols], k_i8[rows, cols].T).astype(np.float64)
            if p_mode == "static":
                P = softmax_masked(A, allowed)
                P_u8 = Q.quant_unsigned(P, s_p)
                acc = int_matmul(P_u8, v_i8[rows, cols])
                x_attn[rows, cols] = float(s_p) * float(s_v) * acc.astype(np.float64)
            else:
                neg = np.where(allowed, A, -np.inf)
                m = np.max(neg, axis=-1, keepdims=True)
                m = np.where(np.isfinite(m), m, 0.0)
                e = np.where(allowed, np.exp(neg - m), 0.0)
                l = np.sum(e, axis=-1, keepdims=True)
                P_u8 = Q.quant_unsigned(e, 1.0 / Q.PMAX)
                acc = int_matmul(P_u8, v_i8[rows, cols])
                x_attn[rows, cols] = np.where(l > 0.0, float(s_v) * acc.astype(np.float64) / (Q.PMAX * np.where(l > 0.0, l, 1.0)), 0.0)
            if return_internals:
                internals["P_u8"][(b, h)] = P_u8
                internals["acc"][(b, h)] = acc
    o = emit(x_attn, out)
    return (o, internals) if return_internals else o


def attention_int8_decode(q_i8, k_cache, v_cache, lens, nh, dh, s_q, s_k, s_v, s_p, out: OutSpec, p_mode="static"):
    """One decode step of the INT8 attention core (Eq. 15-17 for a single query row per sequence, the generation
    workload the method names) over an INT8 key / value cache.

    q_i8 [B, nh*dh] int8: the current token's query; k_cache, v_cache [B, S_max, nh*dh] int8 (SQ scales s_k, s_v), of
    which sequence b holds lens[b] valid entries, the current token's own key / value included (it attends to itself
    and to everything before it, which is what the causal mask gives its row in a prefill).  Per (b, h):
        A[k] = d~ (q . K[k]),  d~ = s_q s_k / sqrt(dh),  k < lens[b];   P = softmax(A);
        P_u8 = clip(Round(P / s_p), 0, 255);   acc = sum_k P_u8[k] V[k]  (exact INT32);   X_attn = s_p s_v acc
    then the output stage.  p_mode="rowmax": e = exp(A - max A), P~_u8 = Round(255 e), X_attn = s_v acc / (255 sum e).
    A sequence with lens[b] = 0 yields zeros.
    """
    assert p_mode in ("static", "rowmax")
    q_i8, k_cache, v_cache = np.asarray(q_i8), np.asarray(k_cache), np.asarray(v_cache)
    assert q_i8.dtype == np.int8 and k_cache.dtype == np.int8 and v_cache.dtype == np.int8
    B, H = q_i8.shape
    assert H == nh * dh
    d_tilde = float(s_q) * float(s_k) / np.sqrt(float(dh))
    x_attn = np.zeros((B, H), dtype=np.float64)
    for b in range(B):
        L = int(lens[b])
        if L == 0:
            continue
        for h in range(nh):
            cols = slice(h * dh, (h + 1) * dh)
            A = d_tilde * int_matmul(q_i8[b:b + 1, cols], k_cache[b, :L, cols].T).astype(np.float64)[0]
            e = np.exp(A - np.max(A))
            if p_mode == "static":
                P_u8 = Q.quant_unsigned(e / np.sum(e), s_p)
                acc = int_matmul(P_u8[None, :], v_cache[b, :L, cols])[0]
                x_attn[b, cols] = float(s_p) * float(s_v) * acc.astype(np.float64)
            else:
                P_u8 = Q.quant_unsigned(e, 1.0 / Q.PMAX)
                acc = int_matmul(P_u8[None, :], v_cache[b, :L, cols])[0]
                x_attn[b, cols] = float(s_v) * acc.astype(np.float64) / (Q.PMAX * np.sum(e))
    return emit(x_attn, out)


def attention_f8(q_f8, k_f8, v_f8, B, S, nh, dh, s_q, s_k, s_v, s_p, out: OutSpec, mask="none", key_len=None):
    """The FP8 variant of the attention core: e4m3 Q, K, V (values, SQ scales s_q, s_k, s_v) and an e4m3 P.

    per (b, h):  A = d~ (Q K^T),  d~ = s_q s_k / sqrt(dh);  P = softmax(A) over the allowed keys;
                 P_f8 = e4m3(P / s_p)  (s_p = max P / 448 from calibration; saturating);
                 acc = P_f8 V_f8;  X_attn = s_p s_v acc -> output stage.
    Every product of two e4m3 values and every partial sum here is exact in fp64.
    """
    H = nh * dh
    d_tilde = float(s_q) * float(s_k) / np.sqrt(float(dh))
    x_attn = np.zeros((B * S, H), dtype=np.float64)
    for b in range(B):
        allowed = attention_mask(S, mask, None if key_len is None else key_len[b])
        rows = slice(b * S, (b + 1) * S)
        for h in range(nh):
            cols = slice(h * dh, (h + 1) * dh)
            A = d_tilde * (np.asarray(q_f8[rows, cols], np.float64) @ np.asarray(k_f8[rows, cols], np.float64).T)
            P = softmax_masked(A, allowed)
            P_f8 = Q.quant_f8(P, s_p)
            x_attn[rows, cols] = float(s_p) * float(s_v) * (P_f8 @ np.asarray(v_f8[rows, cols], np.float64))
    return emit(x_attn, out)


def attention_fp(q, k, v, B, S, nh, dh, out: OutSpec, mask="none", key_len=None):
    """FP-mode attention (Eq. 9-11): softmax(Q K^T / sqrt(dh)) V in fp64 on the stored operands."""
    H = nh * dh
    x_attn = np.zeros((B * S, H), dtype=np.float64)
    for b in range(B):
        allowed = attention_mask(S, mask, None if key_len is None else key_len[b])
        rows = slice(b * S, (b + 1) * S)
        for h in range(nh):
            cols = slice(h * dh, (h + 1) * dh)
            A = (q[rows, cols] @ k[rows, cols].T) / np.sqrt(float(dh))
            x_attn[rows, cols] = softmax_masked(A, allowed) @ v[rows, cols]
    return emit(x_attn, out)
