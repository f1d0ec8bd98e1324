"""GPU parity of a chained stack of layers (model.Stack: what the multi-layer benchmark drives) against the oracle's
chain: mixed granularities, one layer left in FP16, every hand-off between layers typed by the consumer."""
import numpy as np
import pytest
import torch

from oracle import layer as OL
from oracle import ops as O
from paper_2310_17723_b200 import hero, prep, workloads as W
from paper_2310_17723_b200.model import Stack
from gpu_util import rel_err

pytestmark = pytest.mark.gpu


def _cfgs(shape):
    m3, fp = dict(prep.PRESETS["M3"]), dict(prep.PRESETS["FP"])
    base = dict(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, arch=shape.arch, eps=shape.eps, mask=shape.mask,
                fp_dtype=shape.fp_dtype)
    cfgs = [prep.LayerConfig(**base, mode=dict(m3)),                        # TWQ everywhere
            prep.LayerConfig(**base, mode=dict(m3), gran_in="fwq"),         # FWQ on the LN output feeding QKV
            prep.LayerConfig(**base, mode=dict(fp)),                        # a layer left in FP16
            prep.LayerConfig(**base, mode=dict(m3), gran_attn="sq"),        # SQ on X_attn
            prep.LayerConfig(**base, mode=dict(m3), gran_in="sq", gran_mid="fwq")]
    for li, c in enumerate(cfgs):                                           # a layer emits what the next layer's QKV consumes
        c.gran_out = "fp" if li + 1 == len(cfgs) else ("fp" if cfgs[li + 1].mode["qkv"] == "fp" else cfgs[li + 1].gran_in)
    return cfgs


def test_stack_of_mixed_layers_against_the_oracle_chain():
    shape = W.tiny_shape(B=2, S=128, H=256, nh=4, F=512, eps=1e-5, n_outlier=2)
    cid, n_cal = 7, 2
    cfgs = _cfgs(shape)
    h = hero.Handle()
    stack = Stack(h, shape, cid, cfgs, n_cal_seq=n_cal)
    x = W.activations(shape, cid)
    stack.set_input(torch.from_numpy(x).to(torch.float16).cuda())
    n0 = h.launches
    stack.forward()
    h.check()
    assert h.launches - n0 == 7 * len(cfgs)
    got = stack.output[0].float().cpu().numpy().astype(np.float64)

    # ---- the oracle's chain: its own calibration on the same seeded calibration inputs, its own folding and quantization
    x_cal = W.activations(shape, cid, n_seq=n_cal, tensor=7).astype(np.float64)
    layers, cur = [], None
    for li, cfg in enumerate(cfgs):
        spec = OL.LayerSpec(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, arch=shape.arch, act=cfg.act, eps=cfg.eps,
                            mask=cfg.mask, fp_dtype=cfg.fp_dtype, mode=dict(cfg.mode), gran_in=cfg.gran_in, gran_mid=cfg.gran_mid,
                            gran_attn=cfg.gran_attn, gran_out=cfg.gran_out)
        p = W.layer_params(shape, cid * 100 + li)
        if li == 0:
            ln0 = (p["ln0_g"], p["ln0_b"])
            cur = O.layernorm(x_cal, p["ln0_g"], p["ln0_b"], spec.eps)
        C = OL.calibrate(spec, p, cur, n_cal)
        cur = OL.layer_fp64(spec, p, cur, B=n_cal)["x_out"]
        layers.append(OL.prepare_layer(spec, p, C))
    t = OL.entry_ln(O.fp_tensor(x, "f16"), ln0[0], ln0[1], cfgs[0].eps, layers[0]["ln_in_out"])
    kinds = []
    for Lp in layers:
        t = OL.layer_forward(Lp, t)["x_out"]
        kinds.append(t.kind)
    assert kinds == ["i8", "fp", "i8", "i8", "fp"]                          # the hand-offs: into the FP layer and out of the stack
    want = t.real()
    # free-running through five layers: codes that flip on a tie perturb everything downstream, so the check is statistical
    assert rel_err(got, want) < 5e-2
    assert float(np.abs(got - want).mean() / np.abs(want).mean()) < 1e-2
    h.close()
