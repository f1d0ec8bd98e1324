"""Pins for oracle/layer.py: folding identities (Eq. 20-23, 32), Table 1, and the layer forward
against a library transformer layer (all-FP) and against the un-quantized layer (INT8)."""
import os

import numpy as np
import pytest

from oracle import layer as L
from oracle import ops as O
from oracle import quant as Q
from paper_2310_17723_b200 import workloads as W

torch = pytest.importorskip("torch")
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _spec(shape, **kw):
    return L.LayerSpec(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, arch=shape.arch,
                       mask=shape.mask, fp_dtype=shape.fp_dtype, eps=shape.eps, **kw)


def test_mode_presets_match_table1():
    with open(os.path.join(GOLD, "mode_presets.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for name, emb, *flags in rows:
        assert emb == "1"
        got = [L.MODE_PRESETS[name][m] for m in L.MODULES]
        assert got == ["int8" if f == "1" else "fp" for f in flags], name


def test_producer_fold_leaves_int8_weights_unchanged():
    # Eq. 20-21: per-column absmax quantization is invariant to a per-column rescale, so the INT8
    # weights of W / S_out equal those of W and the column scale is S_w / S_out.
    g = np.random.default_rng(0)
    Wm, b = g.standard_normal((48, 24)) * 0.02, g.standard_normal(24) * 0.01
    s_out = np.abs(g.standard_normal(24)) * 0.05 + 0.01
    W0, sw0, _ = L.fold_and_quantize(Wm, b)
    W1, sw1, b1 = L.fold_and_quantize(Wm, b, None, s_out)
    assert np.array_equal(W0, W1)
    assert np.allclose(sw1, sw0 / s_out, rtol=2e-7)
    assert np.allclose(b1, b / s_out, rtol=1e-7)


def test_consumer_fold_is_exact_in_real_arithmetic_and_precedes_quantization():
    # Eq. 23 / 32: (X_int8 Diag(S)) W == X_int8 (Diag(S) W); the INT8 weights DO change.
    g = np.random.default_rng(1)
    Wm = g.standard_normal((40, 16)) * 0.02
    s_in = np.abs(g.standard_normal(40)) * 0.05 + 0.001
    x = g.integers(-127, 128, (5, 40), dtype=np.int8)
    lhs = (x * s_in[None, :]) @ Wm
    rhs = x.astype(float) @ (s_in[:, None] * Wm)
    assert np.allclose(lhs, rhs, rtol=1e-13)
    Wf, swf, _ = L.fold_and_quantize(Wm, None, s_in, None)
    Wp, swp, _ = L.fold_and_quantize(Wm, None, None, None)
    assert np.mean(Wf != Wp) > 0.5
    # the folded-then-quantized GEMM approximates the real product
    approx = x.astype(float) @ (Wf * swf[None, :])
    assert np.max(np.abs(approx - lhs)) / np.max(np.abs(lhs)) < 0.02


def _torch_layer(spec, p, x, B):
    """A transformer layer assembled from library routines in float64."""
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    X = t(x)
    H, nh, dh, S = spec.H, spec.nh, spec.dh, spec.S
    lin = torch.nn.functional.linear
    ln = lambda v, g, b: torch.nn.functional.layer_norm(v, (H,), t(p[g]), t(p[b]), spec.eps)

    def attn(v):
        q, k, vv = (lin(v, t(p["W" + n]).T, t(p["b" + n])).view(B, S, nh, dh).transpose(1, 2) for n in "qkv")
        a = torch.nn.functional.scaled_dot_product_attention(q, k, vv, is_causal=(spec.mask == "causal"))
        return lin(a.transpose(1, 2).reshape(B * S, H), t(p["Wo"]).T, t(p["bo"]))

    def mlp(v):
        return lin(torch.nn.functional.gelu(lin(v, t(p["W1"]).T, t(p["b1"]))), t(p["W2"]).T, t(p["b2"]))

    if spec.arch == "post_ln":
        m = ln(X + attn(X), "ln1_g", "ln1_b")
        return ln(m + mlp(m), "ln2_g", "ln2_b").numpy()
    h = X + attn(ln(X, "ln1_g", "ln1_b"))
    return (h + mlp(ln(h, "ln2_g", "ln2_b"))).numpy()


@pytest.mark.parametrize("arch,mask", [("post_ln", "none"), ("pre_ln", "causal")])
def test_unquantized_layer_matches_library(arch, mask):
    shape = W.tiny_shape(arch=arch, mask=mask, eps=1e-5)
    spec = _spec(shape)
    p = W.layer_params(shape, 7)
    x = W.activations(shape, 7)
    got = L.layer_fp64(spec, p, x)["x_out"]
    assert np.allclose(got, _torch_layer(spec, p, x, shape.B), rtol=1e-10, atol=1e-10)


@pytest.mark.parametrize("arch,mask", [("post_ln", "none"), ("pre_ln", "causal")])
def test_all_fp_mode_layer_tracks_library_layer(arch, mask):
    # every module in FP mode: the only difference from the library layer is FP16 storage rounding
    shape = W.tiny_shape(arch=arch, mask=mask, eps=1e-5)
    spec = _spec(shape, mode=dict(L.MODE_PRESETS["FP"]), gran_out="fp")
    p = W.layer_params(shape, 8)
    x = W.activations(shape, 8)
    C = L.calibrate(spec, p, x, shape.B)
    Lp = L.prepare_layer(spec, p, C)
    T = L.layer_forward(Lp, O.fp_tensor(x, spec.fp_dtype))
    ref = _torch_layer(spec, p, x, shape.B)
    assert T["x_out"].kind == "fp"
    assert np.max(np.abs(T["x_out"].real() - ref)) / np.max(np.abs(ref)) < 5e-3


@pytest.mark.parametrize("preset", ["M1", "M2", "M3"])
@pytest.mark.parametrize("arch", ["post_ln", "pre_ln"])
def test_int8_layer_is_close_to_unquantized_layer_and_types_follow_table1(preset, arch):
    shape = W.tiny_shape(arch=arch, mask="causal" if arch == "pre_ln" else "none", eps=1e-5, n_outlier=2)
    spec = _spec(shape, mode=dict(L.MODE_PRESETS[preset]))
    p = W.layer_params(shape, 9)
    x = W.activations(shape, 9)
    xc = x      # calibrated on the data it is checked on: a static S_p from 96 foreign tokens clips P
    C = L.calibrate(spec, p, xc if arch == "pre_ln" else O.layernorm(xc, p["ln0_g"], p["ln0_b"], spec.eps), shape.B)
    Lp = L.prepare_layer(spec, p, C)
    if arch == "post_ln":
        x_in = L.entry_ln(O.fp_tensor(x, "f16"), p["ln0_g"], p["ln0_b"], spec.eps, Lp["ln_in_out"])
        ref_in = O.layernorm(x, p["ln0_g"], p["ln0_b"], spec.eps)
    else:
        x_in, ref_in = O.fp_tensor(x, spec.fp_dtype), x
    T = L.layer_forward(Lp, x_in)
    R = L.layer_fp64(spec, p, ref_in)
    ref = R["x_out"]
    err = np.max(np.abs(T["x_out"].real() - ref)) / np.max(np.abs(ref))
    assert err < 0.05, err
    # the branches (small beside the residual, so checked on their own): a few percent; a wrong
    # scale axis, a missing sqrt(dh) or a transposed weight gives O(1)
    for key in ("x_attn", "x_o", "a", "x_2"):
        e = np.max(np.abs(T[key].real() - R[key])) / np.max(np.abs(R[key]))
        assert e < 0.08, (key, e)
    m = L.MODE_PRESETS[preset]
    kind = lambda k: T[k].kind
    assert kind("x_in") == "i8" and kind("x_mid") == "i8"                       # QKV, FC1 INT8 in all presets
    assert kind("qkv") == ("i8" if m["attn"] == "int8" else "fp")
    assert kind("x_attn") == ("i8" if m["attn_out"] == "int8" else "fp")
    assert kind("x_o") == ("i8" if m["attn_out"] == "int8" else "fp")
    assert kind("a") == ("i8" if m["fc2"] == "int8" else "fp")
    assert kind("x_2") == ("i8" if m["fc2"] == "int8" else "fp")
    # INT32 accumulators exist exactly for the INT8 GEMMs
    for key, mod in (("acc_qkv", "qkv"), ("acc_o", "attn_out"), ("acc_fc1", "fc1"), ("acc_fc2", "fc2")):
        assert (T[key] is not None) == (m[mod] == "int8")


# Largest |difference| / largest |value| allowed per border when a library routine recomputes the stage from the oracle's
# own (dequantized) input border: the stage's quantization steps (8-bit weights, 8-bit output, 8-bit P) and nothing else.
# Measured on these seeds: 0.0004 - 0.023; a dropped bias, a scale on the wrong axis, a missing 1 / sqrt(dh) or a
# transposed weight gives 0.1 or more.
_STAGE_BAR = {"qkv": 0.02, "x_attn": 0.05, "x_o": 0.025, "h_mid": 0.002, "x_mid": 0.008, "a": 0.04, "x_2": 0.035,
              "x_out": 0.008, "h_out": 0.002}


@pytest.mark.parametrize("preset", ["M1", "M2", "M3"])
@pytest.mark.parametrize("arch", ["post_ln", "pre_ln"])
def test_every_stage_of_the_layer_matches_a_library_routine_fed_its_own_input_border(preset, arch):
    # teacher-forced: each operator of layer_forward, whatever its mode, must agree with the float64 library routine of the
    # same operator applied to the dequantized tensor the oracle itself fed it, to within that operator's quantization
    # steps.  This pins the wiring of the whole quantized layer (which border feeds which operator, every folded scale,
    # bias and dequantization factor) to something other than the oracle.
    shape = W.tiny_shape(arch=arch, mask="causal" if arch == "pre_ln" else "none", eps=1e-5, n_outlier=2)
    spec = _spec(shape, mode=dict(L.MODE_PRESETS[preset]))
    p = W.layer_params(shape, 9)
    x = W.activations(shape, 9)
    C = L.calibrate(spec, p, x if arch == "pre_ln" else O.layernorm(x, p["ln0_g"], p["ln0_b"], spec.eps), shape.B)
    Lp = L.prepare_layer(spec, p, C)
    x_in = (L.entry_ln(O.fp_tensor(x, "f16"), p["ln0_g"], p["ln0_b"], spec.eps, Lp["ln_in_out"]) if arch == "post_ln"
            else O.fp_tensor(x, spec.fp_dtype))
    T = L.layer_forward(Lp, x_in)
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    r = lambda k: t(T[k].real())
    H, nh, dh, S, B = spec.H, spec.nh, spec.dh, spec.S, shape.B
    lin = torch.nn.functional.linear
    ln = lambda v, g, b: torch.nn.functional.layer_norm(v, (H,), t(p[g]), t(p[b]), spec.eps)
    want = {}
    want["qkv"] = lin(r("x_in"), t(np.concatenate([p["Wq"], p["Wk"], p["Wv"]], axis=1)).T,
                      t(np.concatenate([p["bq"], p["bk"], p["bv"]])))
    q, k, v = (r("qkv")[:, i * H:(i + 1) * H].reshape(B, S, nh, dh).transpose(1, 2) for i in range(3))
    want["x_attn"] = torch.nn.functional.scaled_dot_product_attention(
        q, k, v, is_causal=(spec.mask == "causal")).transpose(1, 2).reshape(B * S, H)
    want["x_o"] = lin(r("x_attn"), t(p["Wo"]).T, t(p["bo"]))
    if arch == "post_ln":
        want["x_mid"] = ln(r("x_in") + r("x_o"), "ln1_g", "ln1_b")
    else:
        want["h_mid"] = r("h_in") + r("x_o")
        want["x_mid"] = ln(r("h_mid"), "ln2_g", "ln2_b")
    want["a"] = torch.nn.functional.gelu(lin(r("x_mid"), t(p["W1"]).T, t(p["b1"])))
    want["x_2"] = lin(r("a"), t(p["W2"]).T, t(p["b2"]))
    if arch == "post_ln":
        want["x_out"] = ln(r("x_mid") + r("x_2"), "ln2_g", "ln2_b")
    else:
        want["h_out"] = r("h_mid") + r("x_2")
    for key, w in want.items():
        e = float((r(key) - w).abs().max() / w.abs().max())
        assert e < _STAGE_BAR[key], (key, e)


def test_granularity_options_fwq_input_and_sq_attn():
    # FWQ on the LN output feeding QKV (scale folded into the QKV weight rows) and SQ on X_attn
    shape = W.tiny_shape(n_outlier=3, eps=1e-5)
    p = W.layer_params(shape, 10)
    x = W.activations(shape, 10)
    ref_in = O.layernorm(x, p["ln0_g"], p["ln0_b"], 1e-5)
    errs = {}
    for gi, ga in (("twq", "fwq"), ("fwq", "sq"), ("sq", "fwq")):
        spec = _spec(shape, gran_in=gi, gran_attn=ga, gran_mid=gi)
        C = L.calibrate(spec, p, ref_in, shape.B)
        Lp = L.prepare_layer(spec, p, C)
        x_in = L.entry_ln(O.fp_tensor(x, "f16"), p["ln0_g"], p["ln0_b"], spec.eps, Lp["ln_in_out"])
        assert (x_in.row_scale is not None) == (gi == "twq")
        T = L.layer_forward(Lp, x_in)
        ref = L.layer_fp64(spec, p, ref_in)["x_out"]
        errs[gi] = np.max(np.abs(T["x_out"].real() - ref)) / np.max(np.abs(ref))
        assert errs[gi] < 0.25, (gi, errs[gi])
    # with outlier channels a single static scale is the coarsest choice
    assert errs["sq"] >= errs["fwq"] * 0.5


def test_a_and_x1_are_never_rounded_to_8_bits():
    # "For A, no quantization is applied"; "For X_1, no quantization is used": quantizing them
    # would change the result, so the forward must differ from a variant that does.
    shape = W.tiny_shape(eps=1e-5)
    spec = _spec(shape)
    p = W.layer_params(shape, 11)
    x = W.activations(shape, 11)
    ref_in = O.layernorm(x, p["ln0_g"], p["ln0_b"], 1e-5)
    C = L.calibrate(spec, p, ref_in, shape.B)
    Lp = L.prepare_layer(spec, p, C)
    x_in = L.entry_ln(O.fp_tensor(x, "f16"), p["ln0_g"], p["ln0_b"], spec.eps, Lp["ln_in_out"])
    T = L.layer_forward(Lp, x_in)
    g = Lp["fc1"]
    acc = O.int_matmul(T["x_mid"].data, g["W_i8"])
    x1 = acc * T["x_mid"].row_scale[:, None] * g["cs"][None, :] + g["bias"][None, :]
    assert np.array_equal(T["a"].data, Q.quant_fwq(O.gelu_erf(x1), C["S_a"]))
    s1 = np.abs(x1).max() / 127
    assert not np.array_equal(T["a"].data, Q.quant_fwq(O.gelu_erf(Q.quant_sq(x1, s1) * s1), C["S_a"]))


@pytest.mark.parametrize("preset", ["M2", "M3"])
@pytest.mark.parametrize("arch", ["post_ln", "pre_ln"])
def test_f8_payload_layer_is_close_to_unquantized_layer_and_every_border_is_e4m3(preset, arch):
    # the FP8 variant of the layer: every 8-bit border holds e4m3 values (3 mantissa bits: relative step 2^-4 per
    # element, averaged down by the contractions), scales are absmax / 448.  Pinned against the un-quantized layer.
    shape = W.tiny_shape(arch=arch, mask="causal" if arch == "pre_ln" else "none", eps=1e-5, n_outlier=2)
    spec = _spec(shape, mode=dict(L.MODE_PRESETS[preset]), payload="f8")
    p = W.layer_params(shape, 9)
    x = W.activations(shape, 9)
    C = L.calibrate(spec, p, x if arch == "pre_ln" else O.layernorm(x, p["ln0_g"], p["ln0_b"], spec.eps), shape.B)
    Ci = L.calibrate(_spec(shape, mode=dict(L.MODE_PRESETS[preset])), p,
                     x if arch == "pre_ln" else O.layernorm(x, p["ln0_g"], p["ln0_b"], spec.eps), shape.B)
    assert np.isclose(C["S_q"] * 448.0, Ci["S_q"] * 127.0, rtol=1e-6)          # same absmax, other full range
    assert np.isclose(C["S_p"] * 448.0, Ci["S_p"] * 255.0, rtol=1e-6)
    Lp = L.prepare_layer(spec, p, C)
    if arch == "post_ln":
        x_in = L.entry_ln(O.fp_tensor(x, "f16"), p["ln0_g"], p["ln0_b"], spec.eps, Lp["ln_in_out"])
        ref_in = O.layernorm(x, p["ln0_g"], p["ln0_b"], spec.eps)
    else:
        x_in, ref_in = O.fp_tensor(x, spec.fp_dtype), x
    T = L.layer_forward(Lp, x_in)
    R = L.layer_fp64(spec, p, ref_in)
    err = np.max(np.abs(T["x_out"].real() - R["x_out"])) / np.max(np.abs(R["x_out"]))
    assert err < 0.08, err
    for key in ("x_attn", "x_o", "a", "x_2"):
        e = np.max(np.abs(T[key].real() - R[key])) / np.max(np.abs(R[key]))
        assert e < 0.12, (key, e)
    m = L.MODE_PRESETS[preset]
    for key, mod in (("x_in", "qkv"), ("qkv", "attn"), ("x_attn", "attn_out"), ("x_o", "attn_out"),
                     ("x_mid", "fc1"), ("a", "fc2"), ("x_2", "fc2")):
        want = "f8" if m[mod] == "int8" else "fp"
        assert T[key].kind == want, key
        if want == "f8":
            d = T[key].data
            assert np.array_equal(Q.e4m3_round(d), d) and np.max(np.abs(d)) <= 448.0, key
    for mod in ("qkv", "o", "fc1", "fc2"):
        if Lp[mod]["mode"] == "int8":
            Wq = Lp[mod]["W_i8"]
            assert np.array_equal(Q.e4m3_round(Wq), Wq)
            assert np.allclose(np.max(np.abs(Wq), axis=0), 448.0)                  # every column uses the full range


@pytest.mark.parametrize("preset", ["M2", "M3"])
def test_pre_ln_pending_branch_equals_the_closing_add(preset):
    # Two chained pre-LN layers.  Layer 1 closes with h_out = Round_fp(h_mid + X_2) (the lone-layer add).  Layer 2 can
    # be fed either that h_out, or the un-added pair (h_mid, pending = X_2), in which case its LN1 step forms the same
    # sum itself.  The residual stream is rounded to the storage type exactly once either way, so every tensor of
    # layer 2 must be bit-identical between the two forms; and the `pending` form must report the sum as its h_in.
    shape = W.tiny_shape(arch="pre_ln", mask="causal", eps=1e-5, n_outlier=2)
    spec = _spec(shape, mode=dict(L.MODE_PRESETS[preset]))
    p1, p2 = W.layer_params(shape, 21), W.layer_params(shape, 22)
    x = W.activations(shape, 21)
    L1 = L.prepare_layer(spec, p1, L.calibrate(spec, p1, x, shape.B))
    T1 = L.layer_forward(L1, O.fp_tensor(x, spec.fp_dtype))
    h1 = T1["h_out"]
    assert h1.kind == "fp" and np.array_equal(Q.round_to_storage(T1["h_mid"].real() + T1["x_2"].real(), spec.fp_dtype), h1.data)
    assert np.max(np.abs(T1["x_2"].real())) > 0            # the pending branch is not trivially zero
    L2 = L.prepare_layer(spec, p2, L.calibrate(spec, p2, L.layer_fp64(spec, p1, x)["x_out"], shape.B))
    Ta = L.layer_forward(L2, h1)                                        # closing-add form
    Tb = L.layer_forward(L2, T1["h_mid"], pending=T1["x_2"])            # pending form
    assert np.array_equal(Tb["h_in"].data, h1.data)
    for key in ("x_in", "qkv", "x_attn", "x_o", "x_mid", "h_mid", "a", "x_2", "h_out"):
        a, b = Ta[key], Tb[key]
        assert a.kind == b.kind, key
        assert np.array_equal(a.data, b.data), key
        for sa, sb in ((a.row_scale, b.row_scale), (a.col_scale, b.col_scale)):
            assert (sa is None) == (sb is None) and (sa is None or np.array_equal(sa, sb)), key
    # and the branch matters: dropping it changes the layer's input
    Tc = L.layer_forward(L2, T1["h_mid"])
    assert not np.array_equal(Tc["x_in"].data, Ta["x_in"].data)
