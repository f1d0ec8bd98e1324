"""The library's offline preparation (host numpy) against the oracle's independent one: same master
parameters and calibration batch must give the same INT8 weights, scales and folded biases."""
import numpy as np
import pytest

from oracle import layer as OL
from oracle import ops as O
from paper_2310_17723_b200 import prep, workloads as W


@pytest.mark.parametrize("arch,preset,gi,ga", [("post_ln", "M3", "twq", "fwq"), ("post_ln", "M3", "fwq", "sq"),
                                               ("pre_ln", "M3", "twq", "fwq"), ("post_ln", "M2", "sq", "fwq"),
                                               ("post_ln", "M1", "twq", "fwq"), ("post_ln", "FP", "twq", "fwq")])
def test_prepared_layer_matches_oracle(arch, preset, gi, ga):
    shape = W.tiny_shape(arch=arch, mask="causal" if arch == "pre_ln" else "none", eps=1e-5, n_outlier=2)
    p = W.layer_params(shape, 31)
    x = W.activations(shape, 31).astype(np.float64)
    cal = O.layernorm(x, p["ln0_g"], p["ln0_b"], 1e-5) if arch == "post_ln" else x
    spec = OL.LayerSpec(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, arch=arch, mask=shape.mask, eps=1e-5,
                        mode=dict(OL.MODE_PRESETS[preset]), gran_in=gi, gran_mid=gi, gran_attn=ga)
    cfg = prep.LayerConfig(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, arch=arch, mask=shape.mask, eps=1e-5,
                           mode=dict(prep.PRESETS[preset]), gran_in=gi, gran_mid=gi, gran_attn=ga)
    Co = OL.calibrate(spec, p, cal, shape.B)
    Cp = prep.calibrate(cfg, p, cal, shape.B)
    for k in Co:
        assert np.allclose(np.asarray(Cp[k], np.float64), np.asarray(Co[k], np.float64), rtol=1e-6), k
    Lo = OL.prepare_layer(spec, p, Co)
    Lp = prep.prepare_layer(cfg, p, Cp)
    for name in ("qkv", "o", "fc1", "fc2"):
        go, gp = Lo[name], Lp[name]
        assert gp["int8"] == (go["mode"] == "int8")
        if gp["int8"]:
            diff = gp["W"].astype(int) - go["W_i8"].T.astype(int)
            assert np.abs(diff).max() <= 1 and np.mean(diff != 0) < 1e-4, name     # a code may flip on a tie of the fold
            assert np.allclose(gp["w_scale"], go["cs"], rtol=1e-6)
        assert np.allclose(gp["bias"], go["bias"], rtol=1e-6, atol=1e-12)
        if go["out"].kind == "fwq":
            assert np.allclose(gp["post_scale"], 1.0 / np.asarray(go["out"].scale, np.float64), rtol=1e-6)
        else:
            assert gp["post_scale"] is None
    assert prep.PRESETS == {k: v for k, v in OL.MODE_PRESETS.items()}
