"""Quantizers of Sec. 2.1 in fp64 (oracle; test infrastructure only).

Conventions fixed where the paper is silent:
  * Round(.) is IEEE round-half-to-even (Sec. 2.2.2, "round to the integer operator").
  * "symmetric uniform INT8" uses the range [-127, 127]; -128 is never produced.
  * a scale derived from data is absmax/127; an all-zero row/column/tensor gets scale 1.
  * scales are stored in fp32, so a computed scale is rounded to fp32 before it is used.
"""
import numpy as np

QMAX = 127
PMAX = 255


def rne(v):
    """Round half to even, elementwise, in fp64."""
    return np.rint(np.asarray(v, dtype=np.float64))


def quant_sym(v, scale):
    """Qs(v; s) = clip(RNE(v / s), -127, 127) -> int8.  `scale` broadcasts against v."""
    q = rne(np.asarray(v, dtype=np.float64) / np.asarray(scale, dtype=np.float64))
    return np.clip(q, -QMAX, QMAX).astype(np.int8)


def quant_unsigned(p, scale):
    """Qu(p; s) = clip(RNE(p / s), 0, 255) -> uint8 (the asymmetric softmax output, Sec. 2.2.2)."""
    q = rne(np.asarray(p, dtype=np.float64) / np.asarray(scale, dtype=np.float64))
    return np.clip(q, 0, PMAX).astype(np.uint8)


def _absmax_scale(absmax, qmax=QMAX):
    """scale = absmax / qmax, zero statistic -> 1, rounded to its fp32 storage type."""
    absmax = np.asarray(absmax, dtype=np.float64)
    s = np.where(absmax > 0.0, absmax / qmax, 1.0)
    return s.astype(np.float32).astype(np.float64)


def quant_weight_columnwise(W):
    """Eq. 2: W[d, m] = W_int8 Diag(S_w), one scale per output column.

    Returns (W_int8 [d, m] int8, S_w [m] fp64 holding fp32-representable values).
    """
    W = np.asarray(W, dtype=np.float64)
    S_w = _absmax_scale(np.max(np.abs(W), axis=0))
    return quant_sym(W, S_w[None, :]), S_w


def quant_twq(Y):
    """Eq. 3: token-wise.  X = S_x X_int8 with S_x in R^{n x 1} computed from each row."""
    Y = np.asarray(Y, dtype=np.float64)
    S = _absmax_scale(np.max(np.abs(Y), axis=1))
    return quant_sym(Y, S[:, None]), S


def quant_fwq(Y, S):
    """Eq. 4: feature-wise with a calibrated S_x in R^{1 x d}; values beyond 127 S saturate."""
    S = np.asarray(S, dtype=np.float64).reshape(1, -1)
    return quant_sym(Y, S)


def quant_sq(Y, S):
    """Eq. 5: static, a single calibrated real scale."""
    return quant_sym(Y, float(S))


def dequant(q, row_scale=None, col_scale=None):
    """Reconstruct S_x X_int8 (row scale) and/or X_int8 S_x (column / scalar scale)."""
    x = np.asarray(q).astype(np.float64)
    if row_scale is not None:
        x = x * np.asarray(row_scale, dtype=np.float64).reshape(-1, 1)
    if col_scale is not None:
        x = x * np.asarray(col_scale, dtype=np.float64).reshape(1, -1)
    return x


# --------------------------------------------------------------------------------------
# FP8 (e4m3) variant: the same fusion points with an 8-bit floating-point payload
# --------------------------------------------------------------------------------------
F8MAX = 448.0            # largest finite e4m3 value (1.75 * 2^8); no infinities in this format


def e4m3_round(v):
    """Nearest e4m3 value (1 sign, 4 exponent bits with bias 7, 3 mantissa bits), ties to even, saturating at
    +-448 (the 'satfinite' conversion).  Normal values 2^e (1 + k/8), e in [-6, 8]; below 2^-6 the grid is the
    subnormal one with spacing 2^-9.  Returned in fp64."""
    x = np.asarray(v, dtype=np.float64)
    a = np.minimum(np.abs(x), F8MAX)
    e = np.floor(np.log2(np.where(a > 0.0, a, 1.0)))
    e = np.clip(e, -6.0, 8.0)                   # subnormals share the spacing of the smallest normal binade
    q = np.exp2(e - 3.0)                        # grid spacing inside the binade
    r = np.rint(a / q) * q                      # rint: half to even; a value that rounds up to 2^(e+1) is on the next grid too
    return np.sign(x) * np.minimum(r, F8MAX)


def quant_f8(v, scale):
    """Qf8(v; s) = e4m3(v / s): the 8-bit floating-point counterpart of Qs.  Returns the e4m3 VALUES in fp64."""
    return e4m3_round(np.asarray(v, dtype=np.float64) / np.asarray(scale, dtype=np.float64))


def f8_scale(absmax):
    """absmax / 448 (so that the largest magnitude lands on the largest finite code), zero statistic -> 1, fp32."""
    return _absmax_scale(absmax, F8MAX)


def calib_scale(absmax, qmax=QMAX):
    """Calibrated FWQ / SQ scale from an absmax statistic (no truncation tuning, Sec. 3)."""
    return _absmax_scale(absmax, qmax)


def round_to_storage(x, dtype):
    """Round fp64 values to the grid of a storage type ('f16', 'bf16', 'f32', 'f64'), RNE."""
    x = np.asarray(x, dtype=np.float64)
    if dtype == "f64":
        return x
    if dtype == "f32":
        return x.astype(np.float32).astype(np.float64)
    if dtype == "f16":
        return x.astype(np.float16).astype(np.float64)
    if dtype == "bf16":
        # 8 significant bits (1 implicit + 7 stored); exponent range of fp32, which these
        # activations never leave.
        m, e = np.frexp(x)                      # x = m * 2^e, 0.5 <= |m| < 1
        return np.ldexp(np.rint(m * 256.0), e - 8)
    raise ValueError(dtype)
