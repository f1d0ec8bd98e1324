"""hero_layer_forward_static (the entry point for callers that may not allocate device memory) against
hero_layer_forward, through the C ABI, on two calls in a row.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2310_17723_b200 import hero, prep, workloads as W
from paper_2310_17723_b200.layer import Layer

pytestmark = pytest.mark.gpu


def _layer_and_input(seed):
    shape = W.tiny_shape(B=2, S=128, H=256, nh=4, F=512, eps=1e-5, n_outlier=2)
    p = W.layer_params(shape, seed)
    x = W.activations(shape, seed)
    cfg = prep.LayerConfig(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, eps=shape.eps)
    ln0 = prep._ln(np.asarray(x, np.float64), p["ln0_g"].astype(np.float64), p["ln0_b"].astype(np.float64), cfg.eps)
    h = hero.Handle()
    layer = Layer(h, prep.prepare_layer(cfg, p, prep.calibrate(cfg, p, ln0, shape.B)))
    x_in = torch.empty(shape.M, shape.H, dtype=torch.int8, device="cuda")
    s_in = torch.empty(shape.M, dtype=torch.float32, device="cuda")
    g0, b0 = (torch.from_numpy(np.asarray(p[k], np.float32)).cuda() for k in ("ln0_g", "ln0_b"))
    h.hero_layernorm_quant(hero.tensor(torch.from_numpy(x).to(torch.float16).cuda()), g0, b0, cfg.eps,
                           hero.tensor(x_in, "twq", s_in))
    h.check()
    return h, layer, shape, x_in, s_in


def test_static_scratch_entry_point_matches_the_workspace_one_twice():
    h, layer, shape, x_in, s_in = _layer_and_input(91)
    M, H = shape.M, shape.H
    ref = torch.empty(M, H, dtype=torch.int8, device="cuda")
    ref_s = torch.empty(M, dtype=torch.float32, device="cuda")
    layer.forward(hero.tensor(x_in, "twq", s_in), hero.tensor(ref, "twq", ref_s))
    h.check()
    for call in range(2):
        # a different input on the second call: the scratch still holds the first call's intermediates
        if call == 1:
            x_in = torch.roll(x_in, 7, dims=0).contiguous()
            s_in = torch.roll(s_in, 7, dims=0).contiguous()
            layer.forward(hero.tensor(x_in, "twq", s_in), hero.tensor(ref, "twq", ref_s))
            h.check()
        out = torch.full((M, H), -100, dtype=torch.int8, device="cuda")
        out_s = torch.zeros(M, dtype=torch.float32, device="cuda")
        x_d, o_d = hero.tensor(x_in, "twq", s_in), hero.tensor(out, "twq", out_s)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        hero.hero_layer_forward_static(layer.desc, x_d, o_d)
        hero.hero_static_check()                 # synchronizes; raises if a bounded device-side wait gave up
        free_after = torch.cuda.mem_get_info()[0]
        if call == 1:
            # the entry point's promise: the device's free memory is what it was before the call (the first call
            # may still make the driver load kernels; by the second everything is in place)
            assert free_after == free_before, "device free memory moved by %d bytes" % (free_before - free_after)
        # same kernels on the same inputs: identical INT8 codes and scales, not merely within the 1-LSB bar
        assert torch.equal(out, ref), "call %d: INT8 output differs" % call
        assert torch.equal(out_s, ref_s), "call %d: row scales differ" % call
    h.close()


def test_static_scratch_entry_point_refuses_layers_beyond_its_64_mib():
    h, layer, shape, x_in, s_in = _layer_and_input(92)
    big = hero.LayerDesc.from_buffer_copy(layer.desc)
    big.B, big.S = 64, 1024                       # 65536 tokens: far more scratch than the built-in array holds
    M = 64 * 1024
    x = torch.empty(M, shape.H, dtype=torch.int8, device="cuda")
    s = torch.empty(M, dtype=torch.float32, device="cuda")
    o = torch.empty(M, shape.H, dtype=torch.int8, device="cuda")
    with pytest.raises(hero.HeroError) as e:
        hero.hero_layer_forward_static(big, hero.tensor(x, "twq", s), hero.tensor(o, "twq", s))
    assert e.value.status == hero.ERR_WORKSPACE
    h.close()
