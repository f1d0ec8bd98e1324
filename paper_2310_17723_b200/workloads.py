"""Seeded synthetic inputs shaped like the BERT / GPT layers the method targets.

This module only draws random numbers and names shapes.  It contains none of the method's
arithmetic (no quantizer, no LayerNorm, no folding): both the CUDA path and the CPU checker are
handed what it returns.  Real checkpoints and GLUE batches are not available offline, so these
inputs stand in for them: N(0,1) activations with a few outlier channels (the structure that
motivates feature-wise scales), N(0, 0.02) weights, N(0, 0.01) biases, LayerNorm gains near 1.
"""
from dataclasses import dataclass

import numpy as np

BASE_SEED = 231017723


@dataclass(frozen=True)
class Shape:
    name: str
    B: int
    S: int
    H: int
    nh: int
    F: int
    arch: str = "post_ln"
    mask: str = "none"
    fp_dtype: str = "f16"
    eps: float = 1e-12
    n_outlier: int = 4
    outlier_gain: float = 20.0

    @property
    def dh(self):
        return self.H // self.nh

    @property
    def M(self):
        return self.B * self.S


# The layer shapes of the benchmark configurations.
C1 = Shape("bert_base_b1_s128", B=1, S=128, H=768, nh=12, F=3072)
C3 = Shape("bert_large_b32_s384", B=32, S=384, H=1024, nh=16, F=4096, n_outlier=10, outlier_gain=30.0)
C4 = Shape("gpt_prefill_b8_s2048", B=8, S=2048, H=4096, nh=32, F=16384, arch="pre_ln", mask="causal",
           fp_dtype="bf16", eps=1e-5, n_outlier=0)
C5 = Shape("bert_large_b64_s512", B=64, S=512, H=1024, nh=16, F=4096, n_outlier=10, outlier_gain=30.0)
SHAPES = {s.name: s for s in (C1, C3, C4, C5)}

LN_SWEEP_M = (128, 256, 512, 1024, 2048, 4096, 8192, 16384, 32768, 65536)
LN_SWEEP_H = (768, 1024, 4096, 8192)
GEMM_SWEEP_M = (16, 128, 1024, 8192, 32768)
GEMM_SWEEP_KN = ((1024, 4096), (4096, 4096), (4096, 16384), (16384, 4096))


def rng(config: int, tensor: int = 0):
    return np.random.default_rng(BASE_SEED + 1000 * config + tensor)


def tiny_shape(B=2, S=48, H=128, nh=2, F=256, **kw):
    """A small layer for tests that the CPU checker finishes instantly."""
    return Shape("tiny", B=B, S=S, H=H, nh=nh, F=F, **kw)


def layer_params(shape: Shape, config: int, dtype=np.float32, unit_ln=False):
    """Master (FP) parameters of one transformer layer, paper layout W[d_in, d_out]."""
    H, F = shape.H, shape.F
    g = rng(config, 1)
    n = lambda *s: g.standard_normal(s, dtype=np.float32).astype(dtype)
    p = {}
    for k, s in (("Wq", (H, H)), ("Wk", (H, H)), ("Wv", (H, H)), ("Wo", (H, H)), ("W1", (H, F)), ("W2", (F, H))):
        p[k] = n(*s) * dtype(0.02)
    for k, s in (("bq", H), ("bk", H), ("bv", H), ("bo", H), ("b1", F), ("b2", H)):
        p[k] = n(s) * dtype(0.01)
    for k in ("ln0", "ln1", "ln2"):
        if unit_ln:
            p[k + "_g"], p[k + "_b"] = np.ones(H, dtype), np.zeros(H, dtype)
        else:
            p[k + "_g"] = dtype(1.0) + n(H) * dtype(0.1)
            p[k + "_b"] = n(H) * dtype(0.1)
    return p


def activations(shape: Shape, config: int, n_seq=None, tensor=2):
    """FP activations [n_seq*S, H] ~ N(0,1); a seeded set of channels is scaled up on every token.
    Returned as float32 holding values already representable in float16 (bfloat16 for bf16 shapes)."""
    n_seq = shape.B if n_seq is None else n_seq
    g = rng(config, tensor)
    x = g.standard_normal((n_seq * shape.S, shape.H), dtype=np.float32)
    if shape.n_outlier:
        ch = rng(config, 3).choice(shape.H, size=shape.n_outlier, replace=False)
        x[:, ch] *= np.float32(shape.outlier_gain)
    return to_storage_grid(x, shape.fp_dtype)


def to_storage_grid(x, fp_dtype):
    """Snap float32 values to the float16 / bfloat16 grid (a storage cast, not method arithmetic)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if fp_dtype == "f16":
        return x.astype(np.float16).astype(np.float32)
    if fp_dtype == "bf16":
        u = x.view(np.uint32).astype(np.uint64)
        u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
        return u.astype(np.uint32).view(np.float32)
    raise ValueError(fp_dtype)


def ln_case(M, H, config=2, with_outliers=True):
    """LayerNorm+quant sweep point: X fp16 [M, H], gamma ~ 1+N(0,0.1), beta ~ N(0,0.1)."""
    g = rng(config, 10 + (M % 997) + H)
    x = g.standard_normal((M, H), dtype=np.float32)
    if with_outliers:
        ch = rng(config, 3).choice(H, size=4, replace=False)
        x[:, ch] *= np.float32(20.0)
    gamma = (1.0 + 0.1 * g.standard_normal(H)).astype(np.float32)
    beta = (0.1 * g.standard_normal(H)).astype(np.float32)
    return to_storage_grid(x, "f16"), gamma, beta


def gemm_case(M, K, N, config=2):
    """W8A8 GEMM sweep point: INT8 operands uniform in [-127, 127]; row/column scales sized so
    that the requantized output has a standard deviation of about 30 LSB; bias ~ N(0,1) LSB."""
    g = rng(config, 20 + (M % 991) + K + N)
    A = g.integers(-127, 128, size=(M, K), dtype=np.int8)
    W = g.integers(-127, 128, size=(N, K), dtype=np.int8)      # [N, K]: reduction dim contiguous
    rc = 30.0 / (5376.0 * np.sqrt(K))
    rs = (g.uniform(0.5, 1.5, M) * np.sqrt(rc)).astype(np.float32)
    cs = (g.uniform(0.5, 1.5, N) * np.sqrt(rc)).astype(np.float32)
    bias = g.standard_normal(N).astype(np.float32)
    return A, W, rs, cs, bias


def embedding_tables(V, P, T, H, config=0):
    g = rng(config, 40)
    tok = g.standard_normal((V, H), dtype=np.float32) * np.float32(0.05)
    pos = to_storage_grid(g.standard_normal((P, H), dtype=np.float32) * np.float32(0.02), "f16")
    typ = to_storage_grid(g.standard_normal((T, H), dtype=np.float32) * np.float32(0.02), "f16")
    return tok, pos, typ
