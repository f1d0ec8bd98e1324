"""Helpers for the GPU parity tests: move oracle tensors to the device, compare within the stated bars."""
import os

import numpy as np
import torch

from paper_2310_17723_b200 import hero

TORCH_FP = {"f16": torch.float16, "bf16": torch.bfloat16}


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def f32(a):
    return dev(np.asarray(a, np.float32))


def qt_to_device(qt):
    """Oracle QT -> (torch tensor, hero.Tensor).  INT8: payload + its scale; FP: cast to the storage type
    (exact: the oracle already rounded the values to that grid)."""
    if qt.kind == "fp":
        t = dev(qt.data, TORCH_FP[qt.dtype])
        return t, hero.tensor(t), None
    t = dev(qt.data) if qt.kind == "i8" else dev(np.asarray(qt.data, np.float32), torch.float8_e4m3fn)
    if qt.row_scale is not None:
        s = f32(qt.row_scale)
        return t, hero.tensor(t, "twq", s), s
    if qt.col_scale is not None:
        cs = np.asarray(qt.col_scale)
        if np.all(cs == cs[0]):                      # a static scale travels as one value (Eq. 5)
            s = f32(cs[:1])
            return t, hero.tensor(t, "sq", s), s
        s = f32(cs)
        return t, hero.tensor(t, "fwq", s), s
    return t, hero.tensor(t, "none"), None


def int8_mismatch(got, want):
    """(fraction of elements that differ, max abs difference) between two INT8 arrays."""
    g = np.asarray(got).astype(np.int32)
    w = np.asarray(want).astype(np.int32)
    d = np.abs(g - w)
    return float(np.mean(d != 0)), int(d.max()) if d.size else 0


def report(what, text):
    """One line per passed parity check (shown by `pytest -s`; appended to the file HERO_PARITY_LOG names, if set),
    so that every bar's headroom is on record."""
    line = "parity %-44s %s" % (what or "(unnamed)", text)
    print(line)
    path = os.environ.get("HERO_PARITY_LOG")
    if path:
        with open(path, "a") as f:
            f.write(line + "\n")


def assert_int8_close(got, want, frac=1e-4, what=""):
    """The INT8 bar: bit-exact except at most 1 LSB on at most `frac` of the elements.  The measured mismatch
    fraction and largest difference are reported on success too."""
    f, m = int8_mismatch(got, want)
    assert m <= 1, "%s: max INT8 difference %d LSB" % (what, m)
    # rounding ties arrive like a Poisson count (measured rates: 1e-6 .. 6e-5): a tensor so small that frac * size is
    # below two may still show two of them
    assert f <= max(frac, 2.0 / max(np.asarray(want).size, 1)), "%s: %.3g of elements differ" % (what, f)
    report(what, "mismatch %.3g of %d elements (bar %.1g), max %d LSB" % (f, np.asarray(want).size, frac, m))


def assert_scales_close(got, want, rtol=1e-6, what="row scales"):
    """Token-wise scales (absmax / 127 or / 448, stored FP32) against the oracle's, relative; reports the largest gap."""
    g, w = np.asarray(got, np.float64), np.asarray(want, np.float64)
    gap = float(np.max(np.abs(g - w) / np.abs(w))) if w.size else 0.0
    assert gap <= rtol, "%s: relative gap %.3g (bar %.1g)" % (what, gap, rtol)
    report(what, "largest relative gap %.3g over %d scales (bar %.1g)" % (gap, w.size, rtol))


def rel_err(got, want):
    """max |g - o| / max |o| over the tensor."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    den = np.max(np.abs(want))
    return float(np.max(np.abs(got - want)) / (den if den > 0 else 1.0))


def oracle_layer_to_prepared(Lp):
    """Re-express the oracle's prepared layer (paper layout, fp64) as the host arrays the library's Layer
    uploads: weights transposed to [N][K], fp32 vectors, reciprocal epilogue scales.  Teacher-forcing: the
    CUDA path then runs on exactly the oracle's weights and scales."""
    from paper_2310_17723_b200 import prep
    spec, C = Lp["spec"], Lp["C"]
    cfg = prep.LayerConfig(B=spec.B, S=spec.S, H=spec.H, nh=spec.nh, F=spec.F, arch=spec.arch, act=spec.act,
                           eps=spec.eps, mask=spec.mask, fp_dtype=spec.fp_dtype, mode=dict(spec.mode),
                           gran_in=spec.gran_in, gran_mid=spec.gran_mid, gran_attn=spec.gran_attn,
                           gran_out=spec.gran_out, p_mode=getattr(spec, "p_mode", "static"),
                           payload=getattr(spec, "payload", "i8"))
    f = lambda a: None if a is None else np.ascontiguousarray(np.asarray(a, np.float64).astype(np.float32))
    L = {"cfg": cfg, "C": C}
    for name in ("qkv", "o", "fc1", "fc2"):
        g = Lp[name]
        post = None
        if g["out"].kind == "fwq":
            post = 1.0 / np.asarray(g["out"].scale, np.float64)
        if g["mode"] == "int8":
            Wq = np.ascontiguousarray(g["W_i8"].T)
            if cfg.payload == "f8":               # e4m3 values -> their bytes (the values are on the grid: exact)
                Wq = torch.from_numpy(Wq.astype(np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
            L[name] = {"int8": True, "W": Wq, "w_scale": f(g["cs"]), "bias": f(g["bias"]),
                       "post_scale": f(post)}
        else:
            L[name] = {"int8": False, "W": prep._store_fp(g["W"], spec.fp_dtype), "w_scale": None, "bias": f(g["bias"]),
                       "post_scale": f(post)}
    for k in ("ln1_g", "ln1_b", "ln2_g", "ln2_b"):
        L[k] = f(Lp[k])
    vec = lambda gran, sf, st: None if gran == "twq" else f(sf if gran == "fwq" else [st])
    L["s_in"] = vec(spec.gran_in, C["S_in_f"], C["S_in_t"])
    L["s_mid"] = vec(spec.gran_mid, C["S_mid_f"], C["S_mid_t"])
    L["s_attn"] = vec(spec.gran_attn, C["S_attn_f"], C["S_attn_t"])
    L["s_o"], L["s_x2"] = f(C["S_o"]), f(C["S_x2"])
    L["s_out"] = None if spec.gran_out in ("twq", "fp") else vec(spec.gran_out, C["S_out_f"], C["S_out_t"])
    return L
