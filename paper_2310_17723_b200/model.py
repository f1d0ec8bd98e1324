"""A stack of prepared layers with its chained device buffers: the object the benchmark and the smoke
check drive.  Construction does the offline work (seeded parameters, calibration, folding, upload); `forward`
is pure kernel launches through the C ABI."""
import numpy as np
import torch

from . import hero, prep, workloads
from .layer import Layer


def _ln_np(x, g, b, eps):
    x = np.asarray(x, np.float64)
    mu = x.mean(-1, keepdims=True)
    c = x - mu
    return c / np.sqrt((c * c).mean(-1, keepdims=True) + eps) * g + b


class Stack:
    def __init__(self, handle, shape, config_id, layer_cfgs, n_cal_seq=2, unit_ln=False, prepared=None):
        """shape: workloads.Shape; layer_cfgs: list of prep.LayerConfig (one per layer, chained).  `prepared`: optional
        list of already prepared layers (the dictionaries `prep.prepare_layer` returns), one per config, used instead
        of this constructor's own calibration and folding."""
        self.h, self.shape, self.cfgs = handle, shape, layer_cfgs
        self.M, self.H = shape.M, shape.H
        self.fp_torch = hero.TORCH_FP[shape.fp_dtype]
        post = shape.arch == "post_ln"
        x_cal = workloads.activations(shape, config_id, n_seq=n_cal_seq, tensor=7).astype(np.float64)
        self.layers, self.params = [], []
        cur = None
        ws = None
        for li, cfg in enumerate(layer_cfgs):
            p = workloads.layer_params(shape, config_id * 100 + li, unit_ln=unit_ln)
            if li == 0:
                self.ln0 = (p["ln0_g"], p["ln0_b"])
                cur = _ln_np(x_cal, p["ln0_g"].astype(np.float64), p["ln0_b"].astype(np.float64), cfg.eps) if post else x_cal
            if prepared is not None:
                C = prepared[li]["C"]
                layer = Layer(handle, prepared[li], workspace=ws)
            else:
                C, cur = prep.calibrate(cfg, p, cur, n_cal_seq, return_output=True)
                layer = Layer(handle, prep.prepare_layer(cfg, p, C), workspace=ws)
            ws = layer.workspace
            self.layers.append(layer)
            self.params.append((None, C))
        self._descs = {}
        # chained activation buffers: input of layer 0 .. output of the last layer
        self.bufs = self.make_edges()
        g0, b0 = self.ln0
        self.ln0_g = torch.from_numpy(np.asarray(g0, np.float32)).cuda()
        self.ln0_b = torch.from_numpy(np.asarray(b0, np.float32)).cuda()

    def make_edges(self):
        """A fresh set of chained activation buffers [(tensor, scale tensor or None, hero.Tensor)] for this stack."""
        layer_cfgs = self.cfgs
        bufs = []
        for li in range(len(layer_cfgs) + 1):
            kind = self._edge_kind(li)
            if kind == "fp":
                t = torch.empty(self.M, self.H, dtype=self.fp_torch, device="cuda")
                bufs.append((t, None, hero.tensor(t)))
            else:
                q8 = torch.float8_e4m3fn if getattr(layer_cfgs[min(li, len(layer_cfgs) - 1)], "payload", "i8") == "f8" else torch.int8
                t = torch.empty(self.M, self.H, dtype=q8, device="cuda")
                if kind == "twq":
                    s = torch.empty(self.M, dtype=torch.float32, device="cuda")
                else:
                    src = self.layers[li]._bufs["s_in"] if li < len(layer_cfgs) else self.layers[-1]._bufs["s_out"]
                    s = src
                bufs.append((t, s, hero.tensor(t, kind, s)))
        return bufs

    def _edge_kind(self, li):
        """Type of the tensor between layer li-1 and layer li: 'fp' or an INT8 granularity."""
        n = len(self.cfgs)
        if self.shape.arch == "pre_ln":
            return "fp"
        if li < n:
            cfg = self.cfgs[li]
            return "fp" if cfg.mode["qkv"] == "fp" else cfg.gran_in
        return self.cfgs[-1].gran_out

    def set_input(self, x_fp):
        """Entry LN^quant: turns the FP activation [M, H] into layer 0's input (the role of the embedding
        LayerNorm for a lone post-LN layer); for pre-LN stacks the FP tensor is the residual stream itself."""
        if self.shape.arch == "pre_ln":
            self.bufs[0][0].copy_(x_fp)
            return
        self.h.hero_layernorm_quant(hero.tensor(x_fp), self.ln0_g, self.ln0_b, self.cfgs[0].eps, self.bufs[0][2])

    def forward(self, stream=None):
        """Every layer on the chained buffers: one C call (hero_stack_forward) sequencing the layers' launches."""
        self.h.hero_stack_forward(self.desc(), self.workspace, stream=stream)

    def desc(self, entry_in=None, edges=None):
        """The hero_stack_desc of this stack; `entry_in` (a hero.Tensor over an FP activation buffer) adds the entry
        LN^quant in front, `edges` substitutes other chained buffers (e.g. a second set for an overlapped stream)."""
        key = (id(entry_in), id(edges))
        if key not in self._descs:
            e = [b[2] for b in (edges or self.bufs)]
            self._descs[key] = hero.stack_desc([l.desc for l in self.layers], e, entry_in,
                                               self.ln0_g if entry_in is not None else None,
                                               self.ln0_b if entry_in is not None else None, self.cfgs[0].eps)
        return self._descs[key]

    @property
    def workspace(self):
        return max((l.workspace for l in self.layers), key=lambda w: w.numel())

    @property
    def output(self):
        return self.bufs[-1]
