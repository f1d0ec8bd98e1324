"""GPU parity: hero_int8_decode_attention (one decode step over an INT8 key / value cache) against the oracle, and the
decode-shaped GeMM^quant + attention chain."""
import numpy as np
import pytest
import torch

from oracle import ops as O
from oracle import quant as Q
from paper_2310_17723_b200 import hero, workloads as W
from gpu_util import dev, f32, assert_int8_close, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def h():
    hd = hero.Handle()
    yield hd
    hd.check()
    hd.close()


def _case(B, S_max, nh, dh, seed, spread=40):
    g = W.rng(6, seed)
    H = nh * dh
    i8 = lambda *shape: np.clip(np.rint(g.standard_normal(shape) * spread), -127, 127).astype(np.int8)
    s = float(np.sqrt(1.5) / spread)          # logits d~ q.k with standard deviation about 1.5
    return i8(B, H), i8(B, S_max, H), i8(B, S_max, H), (s, s, 0.02)


def _run(h, q, kc, vc, lens, nh, dh, scales, s_p, spec, p_mode="static", new=None, max_len=None):
    B, H = q.shape
    tq, tk, tv = dev(q), dev(kc), dev(vc)
    tl = dev(np.asarray(lens, np.int32))
    if spec.kind == "fp":
        out = torch.full((B, H), float("nan"), dtype=torch.float16, device="cuda")
        od = hero.tensor(out)
    else:
        out = torch.full((B, H), -99, dtype=torch.int8, device="cuda")
        od = hero.tensor(out, spec.kind, f32(np.asarray(spec.scale).reshape(-1)))
    kn = vn = None
    if new is not None:
        kn, vn = dev(new[0]), dev(new[1])
    h.hero_int8_decode_attention(tq, tk, tv, tl, max_len or kc.shape[1], nh, dh, od, s_q=scales[0], s_k=scales[1], s_v=scales[2],
                                 s_p=s_p, k_new=kn, v_new=vn, p_mode=p_mode)
    h.check()
    res = out.float().cpu().numpy() if spec.kind == "fp" else out.cpu().numpy()
    return res, tk.cpu().numpy(), tv.cpu().numpy()


# B, S_max, lens, nh, dh: one key, a ragged quad, lengths that are not multiples of the split, empty sequences,
# 1 to 8 key splits (S_max 64 .. 20000), both head sizes
CASES = [
    (2, 64, [1, 5], 2, 64), (3, 300, [300, 0, 257], 3, 64), (2, 1000, [999, 513], 2, 128), (1, 4096, [4096], 4, 64),
    (4, 2048, [2048, 7, 1025, 2047], 8, 128), (1, 20000, [19999], 1, 128), (40, 128, list(range(89, 129)), 16, 64),
]


@pytest.mark.parametrize("p_mode", ["static", "rowmax"])
@pytest.mark.parametrize("B,S_max,lens,nh,dh", CASES)
def test_decode_attention_against_oracle(h, B, S_max, lens, nh, dh, p_mode):
    q, kc, vc, sc = _case(B, S_max, nh, dh, 17 + S_max + dh)
    s_p = 1.0 / 255
    fp = O.OutSpec("fp", dtype="f64")
    raw = O.attention_int8_decode(q, kc, vc, lens, nh, dh, *sc, s_p, fp, p_mode=p_mode).data
    got, k_after, v_after = _run(h, q, kc, vc, lens, nh, dh, sc, s_p, O.OutSpec("fp", dtype="f16"), p_mode)
    assert np.array_equal(k_after, kc) and np.array_equal(v_after, vc)          # the caches are read-only here
    assert rel_err(got, raw) < 2e-3
    for b, L in enumerate(lens):
        if L == 0:
            assert np.all(got[b] == 0)
    # INT8 output stage, feature-wise and static
    S_attn = Q.calib_scale(np.abs(raw).max(0))
    want = O.attention_int8_decode(q, kc, vc, lens, nh, dh, *sc, s_p, O.OutSpec("fwq", scale=S_attn), p_mode=p_mode)
    got8, _, _ = _run(h, q, kc, vc, lens, nh, dh, sc, s_p, O.OutSpec("fwq", scale=S_attn), p_mode)
    assert_int8_close(got8, want.data, frac=1e-4, what="X_attn (decode, FWQ)")
    S_t = float(Q.calib_scale(np.abs(raw).max()))
    want = O.attention_int8_decode(q, kc, vc, lens, nh, dh, *sc, s_p, O.OutSpec("sq", scale=S_t), p_mode=p_mode)
    got8, _, _ = _run(h, q, kc, vc, lens, nh, dh, sc, s_p, O.OutSpec("sq", scale=S_t), p_mode)
    assert_int8_close(got8, want.data, frac=1e-4, what="X_attn (decode, SQ)")


def test_decode_attention_static_scale_clipping_and_long_context_mass_loss(h):
    # a static s_p below 1 / 255 saturates the largest probabilities at 255; at 4096 keys most probabilities fall below
    # s_p / 2 and vanish (the paper-literal quantizer): device and oracle agree on both effects
    B, S_max, nh, dh = 2, 4096, 2, 64
    q, kc, vc, sc = _case(B, S_max, nh, dh, 5)
    lens = [4096, 64]
    for s_p in (0.25 / 255, 1.0 / 255):
        raw = O.attention_int8_decode(q, kc, vc, lens, nh, dh, *sc, s_p, O.OutSpec("fp", dtype="f64")).data
        got, _, _ = _run(h, q, kc, vc, lens, nh, dh, sc, s_p, O.OutSpec("fp", dtype="f16"))
        assert rel_err(got, raw) < 2e-3


def test_decode_attention_fused_append_and_strided_cache(h):
    # q, k_new, v_new are the three thirds of a [B, 3H] QKV row block; the caches are views into a wider allocation;
    # the step stores the new key / value at position len - 1 and attends to it
    B, S_max, nh, dh = 3, 515, 2, 128
    H = nh * dh
    q, kc, vc, sc = _case(B, S_max, nh, dh, 23)
    lens = [515, 1, 300]
    g = W.rng(6, 99)
    qkv = np.clip(np.rint(g.standard_normal((B, 3 * H)) * 40), -127, 127).astype(np.int8)
    kc_full, vc_full = kc.copy(), vc.copy()
    for b, L in enumerate(lens):                        # what the caches hold once the new token is in
        kc_full[b, L - 1], vc_full[b, L - 1] = qkv[b, H:2 * H], qkv[b, 2 * H:]
    want = O.attention_int8_decode(qkv[:, :H], kc_full, vc_full, lens, nh, dh, *sc, 1.0 / 255, O.OutSpec("fp", dtype="f64")).data
    t = dev(qkv)
    wide_k = torch.from_numpy(np.concatenate([kc, kc], axis=2)).cuda()      # [B, S_max, 2H]: ld_kv = 2H
    wide_v = torch.from_numpy(np.concatenate([vc, vc], axis=2)).cuda()
    tk, tv = wide_k[:, :, H:], wide_v[:, :, H:]
    out = torch.full((B, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    h.hero_int8_decode_attention(t[:, :H], tk, tv, dev(np.asarray(lens, np.int32)), S_max, nh, dh, hero.tensor(out), s_q=sc[0],
                                 s_k=sc[1], s_v=sc[2], s_p=1.0 / 255, k_new=t[:, H:2 * H], v_new=t[:, 2 * H:])
    h.check()
    assert rel_err(out.float().cpu().numpy(), want) < 1e-2
    assert np.array_equal(tk.cpu().numpy(), kc_full) and np.array_equal(tv.cpu().numpy(), vc_full)
    assert np.array_equal(wide_k[:, :, :H].cpu().numpy(), kc) and np.array_equal(wide_v[:, :, :H].cpu().numpy(), vc)


def test_decode_step_equals_causal_prefill_row_on_device(h):
    # the decode kernel at position t against the prefill kernel's row t (two independent device paths, one definition)
    B, S, nh, dh = 2, 384, 4, 64
    H = nh * dh
    g = W.rng(6, 7)
    qkv = np.clip(np.rint(g.standard_normal((B * S, 3 * H)) * 40), -127, 127).astype(np.int8)
    s = float(np.sqrt(1.5) / 40)
    t = dev(qkv)
    full = torch.empty(B * S, H, dtype=torch.float16, device="cuda")
    h.hero_int8_attention(t[:, :H], t[:, H:2 * H], t[:, 2 * H:], B, S, nh, dh, hero.tensor(full), s_q=s, s_k=s, s_v=0.02, s_p=1.0 / 255,
                          mask="causal")
    pos = [383, 100]
    rows = [b * S + pos[b] for b in range(B)]
    cache = t.view(B, S, 3 * H)
    out = torch.empty(B, H, dtype=torch.float16, device="cuda")
    h.hero_int8_decode_attention(t[rows][:, :H].contiguous(), cache[:, :, H:2 * H], cache[:, :, 2 * H:],
                                 dev(np.asarray([p + 1 for p in pos], np.int32)), S, nh, dh, hero.tensor(out), s_q=s, s_k=s, s_v=0.02,
                                 s_p=1.0 / 255)
    h.check()
    a, b_ = out.float().cpu().numpy(), full[rows].float().cpu().numpy()
    assert rel_err(a, b_) < 2e-3


def test_decode_attention_clamps_lengths_beyond_the_launch_bound(h):
    # len[b] > max_len (a caller's mistake) is treated as max_len: nothing outside the sized buffers is touched
    q, kc, vc, sc = _case(2, 96, 2, 64, 11)
    spec = O.OutSpec("fp", dtype="f16")
    want, _, _ = _run(h, q, kc, vc, [64, 10], 2, 64, sc, 1.0 / 255, spec, max_len=64)
    got, _, _ = _run(h, q, kc, vc, [90, 10], 2, 64, sc, 1.0 / 255, spec, max_len=64)
    assert np.array_equal(got, want)


def test_decode_attention_refusals(h):
    q, kc, vc, sc = _case(2, 64, 2, 64, 3)
    tq, tk, tv, tl = dev(q), dev(kc), dev(vc), dev(np.asarray([3, 4], np.int32))
    out = torch.empty(2, 128, dtype=torch.float16, device="cuda")
    with pytest.raises(hero.HeroError):                              # head size
        h.hero_int8_decode_attention(tq, tk, tv, tl, 64, 4, 32, hero.tensor(out))
    with pytest.raises(hero.HeroError):                              # longer than the launch can hold
        h.hero_int8_decode_attention(tq, tk, tv, tl, 200000, 2, 64, hero.tensor(out))
    with pytest.raises(hero.HeroError):                              # an INT8 output needs its scale
        h.hero_int8_decode_attention(tq, tk, tv, tl, 64, 2, 64, hero.tensor(torch.empty(2, 128, dtype=torch.int8, device="cuda")))
    with pytest.raises(hero.HeroError):                              # misaligned cache view
        h.hero_int8_decode_attention(tq, tk[:, :, 8:], tv[:, :, 8:], tl, 64, 1, 64, hero.tensor(out[:, :64]))
    with pytest.raises(hero.HeroError):                              # k_new without v_new
        a = hero.DecodeAttnArgs(tq.data_ptr(), 128, tk.data_ptr(), tv.data_ptr(), 128, 64 * 128, tq.data_ptr(), None, 128,
                                tl.data_ptr(), 64, 2, 2, 64, 1.0, 1.0, 1.0, 1.0 / 255, 0, hero.tensor(out))
        hero._check(hero.lib().hero_int8_decode_attention(h._h, hero.C.byref(a), hero._stream(None)))
    h.check()


# ------------------------------------------------------------------------------------------------------------------
# the whole layer, one decode step at a time, against the oracle's causal forward pass over the sequence so far
# ------------------------------------------------------------------------------------------------------------------
from oracle import layer as OL
from paper_2310_17723_b200.layer import Layer
from gpu_util import qt_to_device, oracle_layer_to_prepared, TORCH_FP


@pytest.mark.parametrize("arch,dh,p_mode", [("pre_ln", 64, "static"), ("pre_ln", 128, "rowmax"), ("post_ln", 64, "static")])
def test_layer_decode_steps_match_causal_forward_rows(h, arch, dh, p_mode):
    B, S, H, F = 3, 131, 256, 512                        # the last two tokens of each sequence are decoded one by one
    shape = W.tiny_shape(B=B, S=S, H=H, nh=H // dh, F=F, arch=arch, mask="causal", fp_dtype="bf16", eps=1e-5)
    spec = OL.LayerSpec(B=B, S=S, H=H, nh=H // dh, F=F, arch=arch, mask="causal", fp_dtype="bf16", eps=1e-5, p_mode=p_mode,
                        gran_out="fp")
    p = W.layer_params(shape, 61)
    x = W.activations(shape, 61)
    cal = O.layernorm(x, p["ln0_g"], p["ln0_b"], spec.eps) if arch == "post_ln" else x
    Lp = OL.prepare_layer(spec, p, OL.calibrate(spec, p, cal, B))
    if arch == "post_ln":
        x_in = OL.entry_ln(O.fp_tensor(x, "bf16"), p["ln0_g"], p["ln0_b"], spec.eps, Lp["ln_in_out"])
    else:
        x_in = O.fp_tensor(x, "bf16")
    T = OL.layer_forward(Lp, x_in)                       # causal forward pass over all S tokens (the oracle)
    layer = Layer(h, oracle_layer_to_prepared(Lp))
    qkv = T["qkv"].data.reshape(B, S, 3 * H)
    kc = torch.from_numpy(np.ascontiguousarray(qkv[:, :, H:2 * H])).cuda()
    vc = torch.from_numpy(np.ascontiguousarray(qkv[:, :, 2 * H:])).cuda()
    kc[:, S - 2:], vc[:, S - 2:] = 77, -77               # the two positions to be decoded hold garbage
    want_out = T["x_out"].real().reshape(B, S, H)
    for t in (S - 2, S - 1):
        rows = [b * S + t for b in range(B)]
        if arch == "post_ln":
            xin_t = O.QT("i8", x_in.data[rows], row_scale=x_in.row_scale[rows])
        else:
            xin_t = O.QT("fp", x_in.data[rows], dtype="bf16")
        _, in_desc, _ = qt_to_device(xin_t)
        out = torch.full((B, H), float("nan"), dtype=torch.bfloat16, device="cuda")
        lens = dev(np.full(B, t + 1, np.int32))
        n0 = h.launches
        layer.decode(kc, vc, lens, S, in_desc, hero.tensor(out))
        h.check()
        assert h.launches - n0 == (8 if arch == "pre_ln" else 7)
        got = out.float().cpu().numpy().astype(np.float64)
        assert rel_err(got, want_out[:, t]) < 1e-2, t
        # the step appended the token's key and value (the QKV GeMM^quant output of the few-row kernel)
        assert_int8_close(kc[:, t].cpu().numpy(), qkv[:, t, H:2 * H], frac=1e-3, what="appended keys")
        assert_int8_close(vc[:, t].cpu().numpy(), qkv[:, t, 2 * H:], frac=1e-3, what="appended values")
    assert np.array_equal(kc[:, :S - 2].cpu().numpy(), qkv[:, :S - 2, H:2 * H])


def test_layer_decode_refusals(h):
    shape = W.tiny_shape(B=2, S=64, H=256, nh=4, F=512, arch="pre_ln", mask="causal", fp_dtype="bf16", eps=1e-5)
    spec = OL.LayerSpec(B=2, S=64, H=256, nh=4, F=512, arch="pre_ln", mask="causal", fp_dtype="bf16", eps=1e-5,
                        mode=dict(OL.MODE_PRESETS["M1"]))
    p = W.layer_params(shape, 62)
    x = W.activations(shape, 62)
    Lp = OL.prepare_layer(spec, p, OL.calibrate(spec, p, x, 2))
    layer = Layer(h, oracle_layer_to_prepared(Lp))
    kc = torch.zeros(2, 64, 256, dtype=torch.int8, device="cuda")
    xin = torch.zeros(2, 256, dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(xin)
    lens = dev(np.asarray([5, 6], np.int32))
    with pytest.raises(hero.HeroError):                  # M1 leaves the attention core in FP: no decode form
        layer.decode(kc, kc.clone(), lens, 64, hero.tensor(xin), hero.tensor(out))
    with pytest.raises(hero.HeroError):                  # one row per sequence
        layer.decode(kc, kc.clone(), lens, 64, hero.tensor(torch.zeros(4, 256, dtype=torch.bfloat16, device="cuda")), hero.tensor(out))
    h.check()
