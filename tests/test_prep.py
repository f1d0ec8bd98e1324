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


def test_e4m3_encode_matches_the_library_cast_and_saturates():
    # the host-side e4m3 quantizer against torch's float8_e4m3fn cast (round-to-nearest-even) on values that float32
    # holds exactly, all 256 byte patterns as fixed points, ties, subnormals and saturation
    import torch
    from paper_2310_17723_b200 import prep
    g = np.random.default_rng(5)
    x = np.concatenate([g.standard_normal(4000) * 100, g.standard_normal(4000) * 0.01, g.uniform(-448, 448, 4000),
                        [0.0, -0.0, 2.0 ** -9, 2.0 ** -10, 3 * 2.0 ** -10, 2.0 ** -6, 17.0, 18.0, 19.0, 447.9, 464.0]])
    x = x.astype(np.float32).astype(np.float64)
    x = x[np.abs(x) <= 464.0]                      # beyond that the library cast yields NaN; the quantizer saturates
    b, v = prep.e4m3_encode(x)
    want = torch.from_numpy(x.astype(np.float32)).to(torch.float8_e4m3fn)
    assert np.array_equal(v, want.float().numpy().astype(np.float64))
    nz = v != 0
    assert np.array_equal(b[nz], want.view(torch.uint8).numpy()[nz])
    # every finite byte pattern decodes to a value that encodes back to itself
    allb = np.array([i for i in range(256) if (i & 0x7F) != 0x7F], dtype=np.uint8)
    vals = torch.from_numpy(allb).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    b2, v2 = prep.e4m3_encode(vals)
    assert np.array_equal(v2, vals) and np.array_equal(b2[vals != 0], allb[vals != 0])
    b3, v3 = prep.e4m3_encode(np.array([1e9, -1e9, 449.0]))
    assert np.array_equal(v3, [448.0, -448.0, 448.0]) and list(b3) == [0x7E, 0xFE, 0x7E]
    Wq, s = prep.quantize_columns_f8(g.standard_normal((64, 8)) * 0.02)
    dec = torch.from_numpy(Wq).view(torch.float8_e4m3fn).float().numpy()
    assert Wq.shape == (8, 64) and np.allclose(np.abs(dec).max(axis=1), 448.0)
