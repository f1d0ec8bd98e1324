"""Device-resident prepared layer: uploads what `prep.prepare_layer` produced, fills the C layer
descriptor and owns the workspace.  `forward` is one call of hero_layer_forward."""
import numpy as np
import torch

from . import hero


def _up(a, dtype=None):
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.view(dtype) if t.dtype in (torch.uint16, torch.int16) else t.to(dtype)
    return t.cuda()


class Layer:
    def __init__(self, handle, L, workspace=None):
        cfg = L["cfg"]
        C = L["C"]
        self.h, self.cfg = handle, cfg
        self.fp_torch = hero.TORCH_FP[cfg.fp_dtype]
        self._bufs = {}
        d = hero.LayerDesc()
        d.arch = hero.PRE_LN if cfg.arch == "pre_ln" else hero.POST_LN
        d.B, d.S, d.H, d.nh, d.F = cfg.B, cfg.S, cfg.H, cfg.nh, cfg.F
        d.act, d.eps, d.mask, d.fp_dtype = hero.ACT[cfg.act], cfg.eps, hero.MASK[cfg.mask], hero.FPDT[cfg.fp_dtype]
        for i, mname in enumerate(hero.MODULES):
            d.mode[i] = hero.MODE_INT8 if cfg.mode[mname] == "int8" else hero.MODE_FP
        d.gran_in, d.gran_mid = hero.GRAN[cfg.gran_in], hero.GRAN[cfg.gran_mid]
        d.gran_attn, d.gran_out = hero.GRAN[cfg.gran_attn], hero.GRAN[cfg.gran_out]
        d.p_mode = hero.P_MODE[getattr(cfg, "p_mode", "static")]
        d.payload = hero.F8 if getattr(cfg, "payload", "i8") == "f8" else hero.I8
        for name in ("s_in", "s_mid", "s_attn", "s_o", "s_x2", "s_out", "ln1_g", "ln1_b", "ln2_g", "ln2_b"):
            t = _up(L.get(name))
            self._bufs[name] = t
            setattr(d, name, None if t is None else t.data_ptr())
        d.s_q, d.s_k, d.s_v, d.s_p = C["S_q"], C["S_k"], C["S_v"], C["S_p"]
        for name in ("qkv", "o", "fc1", "fc2"):
            g = L[name]
            lp = hero.LinearParams()
            W = g["W"]
            if g["int8"]:
                tW = _up(W)
            else:
                tW = _up(W.view(np.int16) if W.dtype == np.uint16 else W, self.fp_torch)
            ts, tb, tp = _up(g["w_scale"]), _up(g["bias"]), _up(g["post_scale"])
            self._bufs[name] = (tW, ts, tb, tp)
            lp.W = tW.data_ptr()
            lp.w_scale = None if ts is None else ts.data_ptr()
            lp.bias = None if tb is None else tb.data_ptr()
            lp.post_scale = None if tp is None else tp.data_ptr()
            setattr(d, name, lp)
        self.desc = d
        self.workspace_bytes = handle.hero_layer_workspace_bytes(d, cfg.M)
        if workspace is not None and workspace.numel() >= self.workspace_bytes:
            self.workspace = workspace            # layers of a stack run one after another and can share scratch
        else:
            self.workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device="cuda")

    def forward(self, x_in, out, pending=None, stream=None):
        """x_in / out / pending are hero.Tensor structs; runs the whole layer on the current stream."""
        self.h.hero_layer_forward(self.desc, x_in, out, self.workspace, pending=pending, stream=stream)

    def decode(self, k_cache, v_cache, lens, max_len, x_in, out, pending=None, stream=None):
        """One decode step against this layer's INT8 key / value cache (x_in / out have B rows)."""
        self.h.hero_layer_decode(self.desc, k_cache, v_cache, lens, max_len, x_in, out, self.workspace, pending=pending,
                                 stream=stream)
