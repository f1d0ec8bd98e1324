"""ctypes binding of include/hero.h.  Marshals arguments; every step runs in libhero.so.

Tensors are torch CUDA tensors used purely as device buffers (data_ptr / shape / stride); the
stream is torch's current CUDA stream unless one is passed.
"""
import ctypes as C
import os
import sys

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libhero.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_DEVICE_TIMEOUT = range(7)
I8, U8, I32, F16, BF16, F32 = range(6)
GRAN_NONE, GRAN_TWQ, GRAN_FWQ, GRAN_SQ = range(4)
ACT_NONE, ACT_GELU_ERF, ACT_GELU_TANH = range(3)
MASK_NONE, MASK_CAUSAL = range(2)
POST_LN, PRE_LN = range(2)
MODE_INT8, MODE_FP = range(2)
PRESET_FP, PRESET_M1, PRESET_M2, PRESET_M3 = range(4)
MODULES = ("qkv", "attn", "attn_out", "fc1", "fc2")

F8 = 6                      # e4m3 payload of the FP8 variant
_DT = {torch.int8: I8, torch.uint8: U8, torch.int32: I32, torch.float16: F16, torch.bfloat16: BF16,
       torch.float32: F32, torch.float8_e4m3fn: F8}
GRAN = {"none": GRAN_NONE, "twq": GRAN_TWQ, "fwq": GRAN_FWQ, "sq": GRAN_SQ, "fp": GRAN_NONE}
ACT = {"none": ACT_NONE, "gelu_erf": ACT_GELU_ERF, "gelu_tanh": ACT_GELU_TANH}
MASK = {"none": MASK_NONE, "causal": MASK_CAUSAL}
FPDT = {"f16": F16, "bf16": BF16}
TORCH_FP = {"f16": torch.float16, "bf16": torch.bfloat16}


class HeroError(RuntimeError):
    def __init__(self, status, msg):
        super().__init__("hero status %d: %s" % (status, msg))
        self.status = status


class Tensor(C.Structure):
    _fields_ = [("data", C.c_void_p), ("dtype", C.c_int32), ("gran", C.c_int32), ("rows", C.c_int64),
                ("cols", C.c_int64), ("ld", C.c_int64), ("scale", C.c_void_p)]


class LnArgs(C.Structure):
    _fields_ = [("residual", Tensor), ("branch", Tensor), ("extra", Tensor), ("token_ids", C.c_void_p),
                ("type_ids", C.c_void_p), ("seq_len", C.c_int32), ("n_tokens", C.c_int64), ("gamma", C.c_void_p),
                ("beta", C.c_void_p), ("eps", C.c_float), ("out", Tensor), ("fp_out", Tensor),
                ("out_col_absmax", C.c_void_p)]


class LinearArgs(C.Structure):
    _fields_ = [("A", Tensor), ("W", C.c_void_p), ("N", C.c_int64), ("ldw", C.c_int64), ("w_scale", C.c_void_p),
                ("bias", C.c_void_p), ("act", C.c_int32), ("post_scale", C.c_void_p), ("out", Tensor),
                ("out_col_absmax", C.c_void_p)]


class AttnArgs(C.Structure):
    _fields_ = [("q", C.c_void_p), ("k", C.c_void_p), ("v", C.c_void_p), ("dtype", C.c_int32), ("ld", C.c_int64),
                ("B", C.c_int32), ("S", C.c_int32), ("nh", C.c_int32), ("dh", C.c_int32), ("s_q", C.c_float),
                ("s_k", C.c_float), ("s_v", C.c_float), ("s_p", C.c_float), ("mask", C.c_int32),
                ("key_len", C.c_void_p), ("out", Tensor), ("p_absmax", C.c_void_p), ("p_mode", C.c_int32),
                ("out_col_absmax", C.c_void_p)]


class AttnProbe(C.Structure):
    _fields_ = [("scores", C.c_void_p), ("p_codes", C.c_void_p), ("acc", C.c_void_p)]


class DecodeAttnArgs(C.Structure):
    _fields_ = [("q", C.c_void_p), ("ld_q", C.c_int64), ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
                ("ld_kv", C.c_int64), ("batch_stride", C.c_int64), ("k_new", C.c_void_p), ("v_new", C.c_void_p),
                ("ld_new", C.c_int64), ("len", C.c_void_p), ("max_len", C.c_int32), ("B", C.c_int32), ("nh", C.c_int32),
                ("dh", C.c_int32), ("s_q", C.c_float), ("s_k", C.c_float), ("s_v", C.c_float), ("s_p", C.c_float),
                ("p_mode", C.c_int32), ("out", Tensor)]


class LinearParams(C.Structure):
    _fields_ = [("W", C.c_void_p), ("w_scale", C.c_void_p), ("bias", C.c_void_p), ("post_scale", C.c_void_p)]


class LayerDesc(C.Structure):
    _fields_ = [("arch", C.c_int32), ("B", C.c_int32), ("S", C.c_int32), ("H", C.c_int32), ("nh", C.c_int32),
                ("F", C.c_int32), ("act", C.c_int32), ("eps", C.c_float), ("mask", C.c_int32),
                ("fp_dtype", C.c_int32), ("mode", C.c_int32 * 5), ("gran_in", C.c_int32), ("gran_mid", C.c_int32),
                ("gran_attn", C.c_int32), ("gran_out", C.c_int32), ("s_in", C.c_void_p), ("s_mid", C.c_void_p),
                ("s_attn", C.c_void_p), ("s_o", C.c_void_p), ("s_x2", C.c_void_p), ("s_out", C.c_void_p),
                ("s_q", C.c_float), ("s_k", C.c_float), ("s_v", C.c_float), ("s_p", C.c_float),
                ("qkv", LinearParams), ("o", LinearParams), ("fc1", LinearParams), ("fc2", LinearParams),
                ("ln1_g", C.c_void_p), ("ln1_b", C.c_void_p), ("ln2_g", C.c_void_p), ("ln2_b", C.c_void_p),
                ("p_mode", C.c_int32), ("payload", C.c_int32)]


class StackDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("layers", C.POINTER(LayerDesc)), ("edges", C.POINTER(Tensor)),
                ("pending", C.POINTER(Tensor)), ("entry_in", Tensor), ("entry_gamma", C.c_void_p), ("entry_beta", C.c_void_p),
                ("entry_eps", C.c_float)]


class KvCache(C.Structure):
    _fields_ = [("k_cache", C.c_void_p), ("v_cache", C.c_void_p), ("ld_kv", C.c_int64), ("batch_stride", C.c_int64),
                ("len", C.c_void_p), ("max_len", C.c_int32)]


class LayerLayout(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("qkv", "x_attn", "x_o", "x_mid", "x_mid_scale", "a", "x_2", "x_in", "x_in_scale",
                                          "h_in", "h_mid", "total")]


P_MODE = {"static": 0, "rowmax": 1}
HIST_BINS = 2048

EXPORTS = ("hero_create", "hero_destroy", "hero_last_error", "hero_check", "hero_launch_count",
           "hero_layernorm_quant", "hero_w8a8_linear", "hero_int8_attention", "hero_mode_preset",
           "hero_layer_workspace_bytes", "hero_layer_workspace_layout", "hero_layer_forward", "hero_layer_forward_host", "hero_layer_forward_host_async", "hero_profile_begin",
           "hero_profile_end", "hero_layer_forward_static", "hero_absmax_observe", "hero_quantize_weight", "hero_abs_histogram",
           "hero_int8_decode_attention", "hero_layer_decode", "hero_static_check", "hero_int8_attention_probe", "hero_stack_forward",
           "hero_stack_forward_host_async", "hero_quantize_weight_f8")

_lib = None


def lib():
    """The loaded CUDA library.  Missing library = hard error (there is no other implementation)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError("libhero.so is not built (%s); run `python -m paper_2310_17723_b200.build`. "
                               "There is no fallback path." % _LIB_PATH)
        try:                                     # a library older than its sources is loaded all the same, but said
            from . import build as _build
            if os.path.exists(_build.STAMP) and open(_build.STAMP).read().strip() != _build._digest():
                sys.stderr.write("hero: libhero.so was built from other sources than those in csrc/ now; "
                                 "run `python -m paper_2310_17723_b200.build`\n")
        except OSError:
            pass
        L = C.CDLL(_LIB_PATH)
        L.hero_last_error.restype = C.c_char_p
        L.hero_launch_count.restype = C.c_int64
        L.hero_launch_count.argtypes = [C.c_void_p]
        L.hero_create.argtypes = [C.POINTER(C.c_void_p)]
        L.hero_destroy.argtypes = [C.c_void_p]
        L.hero_check.argtypes = [C.c_void_p, C.c_void_p]
        L.hero_layernorm_quant.argtypes = [C.c_void_p, C.POINTER(LnArgs), C.c_void_p]
        L.hero_w8a8_linear.argtypes = [C.c_void_p, C.POINTER(LinearArgs), C.c_void_p]
        L.hero_int8_attention.argtypes = [C.c_void_p, C.POINTER(AttnArgs), C.c_void_p]
        L.hero_int8_attention_probe.argtypes = [C.c_void_p, C.POINTER(AttnArgs), C.POINTER(AttnProbe), C.c_void_p]
        L.hero_int8_decode_attention.argtypes = [C.c_void_p, C.POINTER(DecodeAttnArgs), C.c_void_p]
        L.hero_mode_preset.argtypes = [C.c_int32, C.POINTER(C.c_int32 * 5)]
        L.hero_layer_workspace_bytes.argtypes = [C.POINTER(LayerDesc), C.c_int64, C.POINTER(C.c_size_t)]
        L.hero_absmax_observe.argtypes = [C.c_void_p, C.POINTER(Tensor), C.c_void_p, C.c_void_p, C.c_void_p]
        L.hero_abs_histogram.argtypes = [C.c_void_p, C.POINTER(Tensor), C.c_float, C.c_void_p, C.c_void_p]
        L.hero_quantize_weight.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p]
        L.hero_quantize_weight_f8.argtypes = L.hero_quantize_weight.argtypes
        L.hero_layer_workspace_layout.argtypes = [C.POINTER(LayerDesc), C.c_int64, C.POINTER(LayerLayout)]
        L.hero_layer_forward.argtypes = [C.c_void_p, C.POINTER(LayerDesc), C.POINTER(Tensor), C.POINTER(Tensor),
                                         C.POINTER(Tensor), C.c_void_p, C.c_size_t, C.c_void_p]
        L.hero_layer_decode.argtypes = [C.c_void_p, C.POINTER(LayerDesc), C.POINTER(KvCache), C.POINTER(Tensor), C.POINTER(Tensor),
                                        C.POINTER(Tensor), C.c_void_p, C.c_size_t, C.c_void_p]
        L.hero_layer_forward_host_async.argtypes = [C.c_void_p, C.POINTER(LayerDesc)] + [C.POINTER(Tensor)] * 4 + \
            [C.c_void_p, C.c_size_t, C.c_void_p]
        L.hero_layer_forward_host.argtypes = [C.c_void_p, C.POINTER(LayerDesc)] + [C.POINTER(Tensor)] * 4 + \
            [C.c_void_p, C.c_size_t, C.c_void_p]
        L.hero_layer_forward_static.argtypes = [C.POINTER(LayerDesc), C.POINTER(Tensor), C.POINTER(Tensor),
                                                C.POINTER(Tensor), C.c_void_p]
        L.hero_static_check.argtypes = [C.c_void_p]
        L.hero_stack_forward.argtypes = [C.c_void_p, C.POINTER(StackDesc), C.c_void_p, C.c_size_t, C.c_void_p]
        L.hero_stack_forward_host_async.argtypes = [C.c_void_p, C.POINTER(StackDesc), C.POINTER(Tensor), C.POINTER(Tensor),
                                                    C.c_void_p, C.c_size_t, C.c_void_p]
        L.hero_profile_begin.argtypes = [C.c_void_p, C.c_int32]
        L.hero_profile_end.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        _lib = L
    return _lib


def _check(status):
    if status != OK:
        raise HeroError(status, lib().hero_last_error().decode())


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def tensor(t, gran="none", scale=None):
    """hero_tensor view of a 2-D torch CUDA tensor (row-major, unit inner stride); None -> absent."""
    if t is None:
        return Tensor(None, 0, 0, 0, 0, 0, None)
    assert t.is_cuda and t.dim() == 2 and t.stride(1) == 1, "need a 2-D row-major CUDA tensor"
    if scale is not None:
        assert scale.is_cuda and scale.dtype == torch.float32 and scale.is_contiguous()
    g = GRAN[gran] if isinstance(gran, str) else gran
    ld = t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])
    T = Tensor(t.data_ptr(), _DT[t.dtype], g, t.shape[0], t.shape[1], ld, None if scale is None else scale.data_ptr())
    T._keep = (t, scale)      # the struct holds raw pointers: keep the buffers alive as long as it lives
    return T


class Handle:
    """Owns a hero_handle on the current CUDA device."""

    def __init__(self):
        if not torch.cuda.is_available():
            raise RuntimeError("hero needs a CUDA device (sm_100a); none is visible")
        self._h = C.c_void_p()
        _check(lib().hero_create(C.byref(self._h)))

    def close(self):
        if self._h:
            lib().hero_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def check(self, stream=None):
        _check(lib().hero_check(self._h, _stream(stream)))

    @property
    def launches(self):
        return int(lib().hero_launch_count(self._h))

    # ---- the four calls of the boundary, same names as the C entry points ----
    def hero_layernorm_quant(self, residual, gamma, beta, eps, out, branch=None, extra=None, fp_out=None,
                             token_ids=None, type_ids=None, seq_len=0, n_tokens=0, out_col_absmax=None, stream=None):
        """residual / branch / extra / out / fp_out are hero.Tensor structs (see `tensor`); out_col_absmax: float32 [H]
        running per-column absolute maximum of the FP tensor the call stores (calibration observer)."""
        a = LnArgs(residual, branch or tensor(None), extra or tensor(None), _ptr(token_ids), _ptr(type_ids),
                   int(seq_len), int(n_tokens), _ptr(gamma), _ptr(beta), float(eps), out or tensor(None),
                   fp_out or tensor(None), _ptr(out_col_absmax))
        _check(lib().hero_layernorm_quant(self._h, C.byref(a), _stream(stream)))

    def hero_w8a8_linear(self, A, W, out, w_scale=None, bias=None, act="none", post_scale=None, out_col_absmax=None,
                         stream=None):
        """A, out: hero.Tensor; W: torch tensor [N, K] (K contiguous); out_col_absmax: float32 [N] running per-column
        absolute maximum of an FP16 / BF16 output (calibration observer fused into the epilogue)."""
        assert W.dim() == 2 and W.stride(1) == 1
        a = LinearArgs(A, W.data_ptr(), W.shape[0], W.stride(0), _ptr(w_scale), _ptr(bias),
                       ACT[act] if isinstance(act, str) else act, _ptr(post_scale), out, _ptr(out_col_absmax))
        _check(lib().hero_w8a8_linear(self._h, C.byref(a), _stream(stream)))

    def hero_int8_attention(self, q, k, v, B, S, nh, dh, out, s_q=1.0, s_k=1.0, s_v=1.0, s_p=1.0 / 255,
                            mask="none", key_len=None, p_absmax=None, p_mode="static", probe=None, out_col_absmax=None,
                            stream=None):
        """q, k, v: 2-D torch views [B*S, nh*dh] sharing one leading dimension; out: hero.Tensor; p_absmax: float32[1]
        running maximum of the softmax probabilities (F16 / BF16 core only).  probe = (scores int32 [B*nh, S, S] | None,
        p_codes uint8 [B*nh, S, S] | None, acc int32 [B*S, nh*dh] | None) calls hero_int8_attention_probe instead."""
        assert q.stride(0) == k.stride(0) == v.stride(0) and q.dtype == k.dtype == v.dtype
        a = AttnArgs(q.data_ptr(), k.data_ptr(), v.data_ptr(), _DT[q.dtype], q.stride(0), B, S, nh, dh, s_q, s_k,
                     s_v, s_p, MASK[mask] if isinstance(mask, str) else mask, _ptr(key_len), out, _ptr(p_absmax),
                     P_MODE[p_mode] if isinstance(p_mode, str) else p_mode, _ptr(out_col_absmax))
        if probe is not None:
            scores, codes, acc = probe
            pr = AttnProbe(_ptr(scores), _ptr(codes), _ptr(acc))
            _check(lib().hero_int8_attention_probe(self._h, C.byref(a), C.byref(pr), _stream(stream)))
            return
        _check(lib().hero_int8_attention(self._h, C.byref(a), _stream(stream)))

    def hero_int8_decode_attention(self, q, k_cache, v_cache, lens, max_len, nh, dh, out, s_q=1.0, s_k=1.0, s_v=1.0,
                                   s_p=1.0 / 255, k_new=None, v_new=None, p_mode="static", stream=None):
        """q: int8 [B, nh*dh] view; k_cache, v_cache: int8 [B, S_max, nh*dh] views (feature stride 1, equal strides);
        lens: int32 [B] device tensor; k_new / v_new: optional int8 [B, nh*dh] views of equal pitch (appended at
        lens[b] - 1); out: hero.Tensor [B, nh*dh]."""
        assert q.dim() == 2 and k_cache.dim() == 3 and k_cache.stride() == v_cache.stride() and k_cache.stride(2) == 1
        assert q.dtype == k_cache.dtype == v_cache.dtype == torch.int8 and lens.dtype == torch.int32 and lens.is_cuda
        ld_new = 0
        if k_new is not None:
            assert k_new.stride(0) == v_new.stride(0) and k_new.dtype == torch.int8
            ld_new = k_new.stride(0) if k_new.shape[0] > 1 else max(k_new.stride(0), k_new.shape[1])
        ld_q = q.stride(0) if q.shape[0] > 1 else max(q.stride(0), q.shape[1])
        a = DecodeAttnArgs(q.data_ptr(), ld_q, k_cache.data_ptr(), v_cache.data_ptr(), k_cache.stride(1), k_cache.stride(0),
                           _ptr(k_new), _ptr(v_new), ld_new, lens.data_ptr(), int(max_len), q.shape[0], nh, dh, s_q, s_k, s_v,
                           s_p, P_MODE[p_mode] if isinstance(p_mode, str) else p_mode, out)
        _check(lib().hero_int8_decode_attention(self._h, C.byref(a), _stream(stream)))

    def hero_absmax_observe(self, x, col_absmax=None, tensor_absmax=None, stream=None):
        """x: hero.Tensor (F16 / BF16); col_absmax float32[cols] / tensor_absmax float32[1]: running maxima, updated."""
        _check(lib().hero_absmax_observe(self._h, C.byref(x), _ptr(col_absmax), _ptr(tensor_absmax), _stream(stream)))

    def hero_abs_histogram(self, x, bound, hist, stream=None):
        """x: hero.Tensor (F16 / BF16); hist: int64 / uint64 [2048] device tensor, accumulated."""
        assert hist.numel() == HIST_BINS and hist.element_size() == 8
        _check(lib().hero_abs_histogram(self._h, C.byref(x), float(bound), C.c_void_p(hist.data_ptr()), _stream(stream)))

    def hero_quantize_weight(self, W, Wq, w_scale, in_scale=None, out_scale=None, bias=None, bias_out=None, stream=None):
        """W: float32 [N, K]; Wq: int8 [N, K], or float8_e4m3fn [N, K] for the FP8 variant (hero_quantize_weight_f8);
        w_scale: float32 [N]; optional folds in_scale [K], out_scale [N]."""
        assert W.dim() == 2 and W.stride(1) == 1 and Wq.stride(1) == 1 and W.dtype == torch.float32
        assert Wq.dtype in (torch.int8, torch.float8_e4m3fn)
        fn = lib().hero_quantize_weight if Wq.dtype == torch.int8 else lib().hero_quantize_weight_f8
        _check(fn(self._h, C.c_void_p(W.data_ptr()), W.stride(0), W.shape[0], W.shape[1],
                                          _ptr(in_scale), _ptr(out_scale), _ptr(bias), C.c_void_p(Wq.data_ptr()),
                                          Wq.stride(0), _ptr(w_scale), _ptr(bias_out), _stream(stream)))

    def hero_layer_workspace_bytes(self, desc, M):
        n = C.c_size_t()
        _check(lib().hero_layer_workspace_bytes(C.byref(desc), int(M), C.byref(n)))
        return int(n.value)

    def hero_layer_workspace_layout(self, desc, M):
        lay = LayerLayout()
        _check(lib().hero_layer_workspace_layout(C.byref(desc), int(M), C.byref(lay)))
        return lay

    def hero_layer_forward_host_async(self, desc, in_host, out_host, in_dev, out_dev, workspace, stream=None):
        """Host-buffer variant without the final synchronisation (out_host is valid after the stream is synchronised)."""
        _check(lib().hero_layer_forward_host_async(self._h, C.byref(desc), C.byref(in_host), C.byref(out_host),
                                                   C.byref(in_dev), C.byref(out_dev), C.c_void_p(workspace.data_ptr()),
                                                   workspace.numel(), _stream(stream)))

    def hero_layer_forward_host(self, desc, in_host, out_host, in_dev, out_dev, workspace, stream=None):
        """Host-buffer variant: copies in, runs the layer, copies out, synchronizes."""
        _check(lib().hero_layer_forward_host(self._h, C.byref(desc), C.byref(in_host), C.byref(out_host),
                                             C.byref(in_dev), C.byref(out_dev), C.c_void_p(workspace.data_ptr()),
                                             workspace.numel(), _stream(stream)))

    def hero_stack_forward(self, stack_desc, workspace, stream=None):
        """stack_desc: hero.StackDesc (see `stack_desc`); one C call runs the entry LN^quant (if any) and every layer."""
        _check(lib().hero_stack_forward(self._h, C.byref(stack_desc), C.c_void_p(workspace.data_ptr()), workspace.numel(),
                                        _stream(stream)))

    def hero_stack_forward_host_async(self, stack_desc, in_host, out_host, workspace, stream=None):
        """Host-buffer variant: H2D of in_host, the stack, D2H into out_host, all enqueued on the stream."""
        _check(lib().hero_stack_forward_host_async(self._h, C.byref(stack_desc), C.byref(in_host), C.byref(out_host),
                                                   C.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(stream)))

    def profile_begin(self, max_launches):
        self._prof_cap = int(max_launches)
        _check(lib().hero_profile_begin(self._h, self._prof_cap))

    def profile_end(self):
        """[(kernel family, milliseconds), ...] for every launch since profile_begin, in order."""
        ms = (C.c_float * self._prof_cap)()
        tag = (C.c_int32 * self._prof_cap)()
        n = C.c_int32()
        _check(lib().hero_profile_end(self._h, ms, tag, C.byref(n)))
        return [(int(tag[i]), float(ms[i])) for i in range(n.value)]

    def hero_layer_forward(self, desc, x_in, out, workspace, pending=None, stream=None):
        """x_in / out / pending: hero.Tensor; workspace: 1-D torch uint8 CUDA tensor."""
        pend = C.byref(pending) if pending is not None else None
        _check(lib().hero_layer_forward(self._h, C.byref(desc), C.byref(x_in), pend, C.byref(out),
                                        C.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(stream)))

    def hero_layer_decode(self, desc, k_cache, v_cache, lens, max_len, x_in, out, workspace, pending=None, stream=None):
        """One decode step: k_cache / v_cache int8 [B, S_max, H] views of equal strides (the new key / value are stored at
        lens[b] - 1), lens int32 [B]; x_in / out / pending: hero.Tensor with B rows."""
        assert k_cache.dim() == 3 and k_cache.stride() == v_cache.stride() and k_cache.stride(2) == 1
        assert k_cache.dtype == v_cache.dtype == torch.int8 and lens.dtype == torch.int32 and lens.is_cuda
        kv = KvCache(k_cache.data_ptr(), v_cache.data_ptr(), k_cache.stride(1), k_cache.stride(0), lens.data_ptr(), int(max_len))
        pend = C.byref(pending) if pending is not None else None
        _check(lib().hero_layer_decode(self._h, C.byref(desc), C.byref(kv), C.byref(x_in), pend, C.byref(out),
                                       C.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(stream)))


def stack_desc(layer_descs, edges, entry_in=None, entry_gamma=None, entry_beta=None, entry_eps=0.0):
    """hero_stack_desc over a list of LayerDesc and a list of len(layer_descs) + 1 hero.Tensor edges (device tensors)."""
    n = len(layer_descs)
    assert len(edges) == n + 1
    sd = StackDesc()
    layers = (LayerDesc * n)(*layer_descs)
    e = (Tensor * (n + 1))(*edges)
    sd.n_layers, sd.layers, sd.edges, sd.pending = n, layers, e, None
    sd.entry_in = entry_in if entry_in is not None else tensor(None)
    sd.entry_gamma, sd.entry_beta, sd.entry_eps = _ptr(entry_gamma), _ptr(entry_beta), float(entry_eps)
    sd._keep = (layers, e, list(layer_descs), list(edges), entry_in, entry_gamma, entry_beta)
    return sd


def host_tensor(t, gran="none", scale=None):
    """hero_tensor view of a 2-D (pinned) host torch tensor, for hero_layer_forward_host."""
    assert not t.is_cuda and t.dim() == 2 and t.stride(1) == 1
    g = GRAN[gran] if isinstance(gran, str) else gran
    T = Tensor(t.data_ptr(), _DT[t.dtype], g, t.shape[0], t.shape[1], t.stride(0), None if scale is None else scale.data_ptr())
    T._keep = (t, scale)
    return T


def hero_layer_forward_static(desc, x_in, out, pending=None, stream=None):
    """The layer forward without handle or workspace, for callers that may not allocate device memory: the
    scratch is a fixed 64 MiB array inside libhero.so (larger layers are refused).  Calls share that array, so
    do not let two of them overlap on the GPU."""
    pend = C.byref(pending) if pending is not None else None
    _check(lib().hero_layer_forward_static(C.byref(desc), C.byref(x_in), pend, C.byref(out), _stream(stream)))


def hero_static_check(stream=None):
    """Synchronizes the stream and raises if a kernel of hero_layer_forward_static left a code in its error word."""
    _check(lib().hero_static_check(_stream(stream)))


def mode_preset(preset):
    m = (C.c_int32 * 5)()
    _check(lib().hero_mode_preset(int(preset), C.byref(m)))
    return list(m)
