"""Calibration on the device (Sec. 2.1): the un-quantized layer runs in FP16 / BF16 through the library's own
operators; every border tensor is observed by the kernel that produces it (the out_col_absmax option of the linear,
LayerNorm and attention calls; the softmax probabilities through p_absmax), only the input of a post-LN layer, which no
kernel of the layer produces, with hero_absmax_observe, and the weights are folded and quantized column-wise by hero_quantize_weight
(Eq. 2, Eq. 20-23, Eq. 32).  Same statistics and the same result layout as the host-side `prep.calibrate` /
`prep.fold_quantize`; only argument marshalling happens here."""
import numpy as np
import torch

from . import hero, prep


def _fp_weight(W, fp_dtype):
    """[K, N] fp64 -> device [N][K] in the storage type."""
    a = prep._store_fp(W, fp_dtype)
    t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a)
    return (t.view(torch.bfloat16) if fp_dtype == "bf16" else t).cuda()


def _vec(a):
    return torch.from_numpy(np.ascontiguousarray(np.asarray(a, np.float64).astype(np.float32))).cuda()


def calibrate_gpu(h, cfg, params, x_cal, n_seq, return_output=False):
    """Device counterpart of `prep.calibrate`: x_cal ([n_seq * S, H], numpy or torch) is what enters the layer (post-LN:
    the tensor feeding QKV; pre-LN: the residual stream).  Returns the same dict of calibrated scales."""
    S, nh, dh, H, F = cfg.S, cfg.nh, cfg.dh, cfg.H, cfg.F
    M = n_seq * S
    fpt = hero.TORCH_FP[cfg.fp_dtype]
    x = (torch.from_numpy(np.asarray(x_cal)) if not torch.is_tensor(x_cal) else x_cal).to(fpt).cuda().contiguous()
    assert x.shape == (M, H)
    p = {k: np.asarray(v, np.float64) for k, v in params.items()}
    Wqkv = _fp_weight(np.concatenate([p["Wq"], p["Wk"], p["Wv"]], axis=1), cfg.fp_dtype)
    bqkv = _vec(np.concatenate([p["bq"], p["bk"], p["bv"]]))
    Wo, W1, W2 = (_fp_weight(p[n], cfg.fp_dtype) for n in ("Wo", "W1", "W2"))
    bo, b1, b2 = _vec(p["bo"]), _vec(p["b1"]), _vec(p["b2"])
    g1, be1, g2, be2 = _vec(p["ln1_g"]), _vec(p["ln1_b"]), _vec(p["ln2_g"]), _vec(p["ln2_b"])
    new = lambda cols: torch.empty(M, cols, dtype=fpt, device="cuda")
    stat = {}

    def observe(name, t, per_feature=True, per_tensor=True):
        cf = torch.zeros(t.shape[1], dtype=torch.float32, device="cuda") if per_feature else None
        ct = torch.zeros(1, dtype=torch.float32, device="cuda") if per_tensor else None
        h.hero_absmax_observe(hero.tensor(t), cf, ct)
        if per_feature:
            stat[name + "_f"] = cf
        if per_tensor:
            stat[name + "_t"] = ct

    def colmax(n):
        return torch.zeros(n, dtype=torch.float32, device="cuda")

    def fused(name, n):
        """Registers the per-feature statistic `name`, to be filled by its producer; the per-tensor one is its maximum."""
        stat[name + "_f"] = colmax(n)
        return stat[name + "_f"]

    def attn(x_in):
        qkv = new(3 * H)
        # the outputs of the linear modules are observed by their own epilogues (per-column running maxima; Q, K and V
        # want one static scale each: the maximum over their column ranges)
        qkv_f = colmax(3 * H)
        h.hero_w8a8_linear(hero.tensor(x_in), Wqkv, hero.tensor(qkv), bias=bqkv, out_col_absmax=qkv_f)
        q, k, v = qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:]
        for i, n in enumerate("qkv"):
            stat[n + "_t"] = qkv_f[i * H:(i + 1) * H].max().reshape(1)
        xa = new(H)
        stat["p_t"] = torch.zeros(1, dtype=torch.float32, device="cuda")
        h.hero_int8_attention(q, k, v, n_seq, S, nh, dh, hero.tensor(xa), mask=cfg.mask, p_absmax=stat["p_t"],
                              out_col_absmax=fused("attn", H))
        xo = new(H)
        stat["o_f"] = colmax(H)
        h.hero_w8a8_linear(hero.tensor(xa), Wo, hero.tensor(xo), bias=bo, out_col_absmax=stat["o_f"])
        return xo

    def mlp(x_mid):
        a = new(F)
        stat["a_f"] = colmax(F)
        h.hero_w8a8_linear(hero.tensor(x_mid), W1, hero.tensor(a), bias=b1, act=cfg.act, out_col_absmax=stat["a_f"])
        x2 = new(H)
        stat["x2_f"] = colmax(H)
        h.hero_w8a8_linear(hero.tensor(a), W2, hero.tensor(x2), bias=b2, out_col_absmax=stat["x2_f"])
        return x2

    out = new(H)
    if cfg.arch == "post_ln":
        observe("in", x, per_tensor=False)
        xo = attn(x)
        xm = new(H)
        h.hero_layernorm_quant(hero.tensor(x), g1, be1, cfg.eps, hero.tensor(xm), branch=hero.tensor(xo),
                               out_col_absmax=fused("mid", H))
        x2 = mlp(xm)
        h.hero_layernorm_quant(hero.tensor(xm), g2, be2, cfg.eps, hero.tensor(out), branch=hero.tensor(x2),
                               out_col_absmax=fused("out", H))
    else:
        xl = new(H)
        h.hero_layernorm_quant(hero.tensor(x), g1, be1, cfg.eps, hero.tensor(xl), out_col_absmax=fused("in", H))
        xo = attn(xl)
        xm, h1 = new(H), new(H)
        h.hero_layernorm_quant(hero.tensor(x), g2, be2, cfg.eps, hero.tensor(xm), branch=hero.tensor(xo), fp_out=hero.tensor(h1),
                               out_col_absmax=fused("mid", H))
        x2 = mlp(xm)
        h.hero_layernorm_quant(hero.tensor(h1), None, None, cfg.eps, None, branch=hero.tensor(x2), fp_out=hero.tensor(out),
                               out_col_absmax=fused("out", H))
    for n in ("in", "attn", "mid", "out"):
        stat[n + "_t"] = stat[n + "_f"].max().reshape(1)
    h.check()
    torch.cuda.synchronize()
    g = lambda k: stat[k].cpu().numpy().astype(np.float64)
    sc = prep.scale_from_absmax
    scales = {
        "S_in_f": sc(g("in_f")), "S_in_t": float(sc(g("in_t"))[0]),
        "S_q": float(sc(g("q_t"))[0]), "S_k": float(sc(g("k_t"))[0]), "S_v": float(sc(g("v_t"))[0]),
        "S_p": float(sc(g("p_t"), 255.0)[0]),
        "S_attn_f": sc(g("attn_f")), "S_attn_t": float(sc(g("attn_t"))[0]),
        "S_o": sc(g("o_f")),
        "S_mid_f": sc(g("mid_f")), "S_mid_t": float(sc(g("mid_t"))[0]),
        "S_a": sc(g("a_f")), "S_x2": sc(g("x2_f")),
        "S_out_f": sc(g("out_f")), "S_out_t": float(sc(g("out_t"))[0]),
    }
    return (scales, out) if return_output else scales


def fold_quantize_gpu(h, W, b, in_scale=None, out_scale=None, payload="i8"):
    """Device counterpart of `prep.fold_quantize` (same arguments and return layout): W is [K, N] (the paper's W[d, m]).
    payload "f8": e4m3 codes (returned as their bytes, uint8) and absmax / 448 scales, through hero_quantize_weight_f8."""
    Wt = torch.from_numpy(np.ascontiguousarray(np.asarray(W, np.float64).T.astype(np.float32))).cuda()   # [N][K]
    N, K = Wt.shape
    Wq = torch.empty(N, K, dtype=torch.float8_e4m3fn if payload == "f8" else torch.int8, device="cuda")
    ws = torch.empty(N, dtype=torch.float32, device="cuda")
    bo = torch.empty(N, dtype=torch.float32, device="cuda") if b is not None else None
    h.hero_quantize_weight(Wt, Wq, ws, in_scale=None if in_scale is None else _vec(in_scale),
                           out_scale=None if out_scale is None else _vec(out_scale),
                           bias=None if b is None else _vec(b), bias_out=bo)
    h.check()
    torch.cuda.synchronize()
    if payload == "f8":
        Wq = Wq.view(torch.uint8)
    return Wq.cpu().numpy(), ws.cpu().numpy(), (None if bo is None else bo.cpu().numpy())


def prepare_layer_gpu(h, cfg, params, C):
    """`prep.prepare_layer` with the weight folding and quantization done on the device."""
    return prep.prepare_layer(cfg, params, C, fold_quantize_fn=lambda W, b, i, o: fold_quantize_gpu(h, W, b, i, o, cfg.payload))
