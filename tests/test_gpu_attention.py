"""GPU parity: hero_int8_attention against the oracle's INT8 attention core (Eq. 15-17)."""
import numpy as np
import pytest
import torch

from oracle import ops as O
from oracle import quant as Q
from paper_2310_17723_b200 import hero, workloads as W
from gpu_util import dev, f32, assert_int8_close, rel_err, int8_mismatch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def h():
    hd = hero.Handle()
    yield hd
    hd.check()
    hd.close()


def _qkv(B, S, nh, dh, seed, spread=40):
    """INT8 q, k, v as thirds of one [B*S, 3H] buffer (the QKV GEMM's output layout)."""
    g = W.rng(3, seed)
    H = nh * dh
    qkv = np.clip(np.rint(g.standard_normal((B * S, 3 * H)) * spread), -127, 127).astype(np.int8)
    return qkv, H


def _calib(raw):
    """Per-feature scale of X_attn from an absmax statistic (Eq. 4).  In use the statistic comes from calibration data, not
    from the tensor being quantized; taking it from the very tensor under test would put every element at an odd multiple
    of 1/254 of its column's maximum on an exact rounding tie (acc * 127 / max acc = k + 1/2), which no arithmetic can be
    expected to break the same way.  The statistic is therefore taken a few percent larger, as foreign data would give."""
    return Q.calib_scale(np.abs(raw).max(0) * 1.037)


def _scales(dh, spread=40):
    # logits d~ q.k with std ~ 1.5: s_q s_k spread^2 sqrt(dh) / sqrt(dh) = 1.5
    s = float(np.sqrt(1.5) / spread)
    return s, s, 0.02


def _run(h, qkv, B, S, nh, dh, s_q, s_k, s_v, s_p, out_spec, mask="none", key_len=None, p_mode="static"):
    H = nh * dh
    t = dev(qkv)
    if out_spec.kind == "fp":
        out = torch.full((B * S, H), float("nan"), dtype=torch.float16, device="cuda")
        od = hero.tensor(out)
    else:
        out = torch.full((B * S, H), -99, dtype=torch.int8, device="cuda")
        sc = f32(np.asarray(out_spec.scale).reshape(-1))
        od = hero.tensor(out, out_spec.kind, sc)
    kl = None if key_len is None else dev(np.asarray(key_len, np.int32))
    h.hero_int8_attention(t[:, :H], t[:, H:2 * H], t[:, 2 * H:], B, S, nh, dh, od, s_q=s_q, s_k=s_k, s_v=s_v, s_p=s_p,
                          mask=mask, key_len=kl, p_mode=p_mode)
    h.check()
    return out.float().cpu().numpy() if out_spec.kind == "fp" else out.cpu().numpy()


def _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, s_p, out_spec, mask="none", key_len=None, internals=False, p_mode="static"):
    H = nh * dh
    return O.attention_int8(qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:], B, S, nh, dh, s_q, s_k, s_v, s_p, out_spec,
                            mask=mask, key_len=key_len, return_internals=internals, p_mode=p_mode)


CASES = [  # B, S, nh, dh, mask
    (1, 128, 2, 64, "none"), (2, 128, 12, 64, "none"), (2, 384, 4, 64, "none"), (1, 512, 2, 64, "none"),
    (1, 256, 2, 128, "causal"), (2, 100, 3, 64, "none"), (1, 333, 2, 128, "causal"), (1, 1024, 1, 128, "causal"),
    (3, 40, 2, 64, "causal"),
]


@pytest.mark.parametrize("B,S,nh,dh,mask", CASES)
def test_int8_attention_fwq_output(h, B, S, nh, dh, mask):
    qkv, H = _qkv(B, S, nh, dh, 100 + S + dh)
    s_q, s_k, s_v = _scales(dh)
    s_p = 1.0 / 255
    raw = _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, s_p, O.OutSpec("fp", dtype="f64"), mask).data
    S_attn = _calib(raw)
    spec = O.OutSpec("fwq", scale=S_attn)
    want = _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, s_p, spec, mask)
    got = _run(h, qkv, B, S, nh, dh, s_q, s_k, s_v, s_p, spec, mask)
    # the INT8 bar (<= 1 LSB on <= 1e-4 of elements); measured 0 .. 6e-5, all of it ties of the fp32 output stage
    # (the P codes themselves agree with the oracle's everywhere: test_probe_scores_codes_and_accumulators)
    assert_int8_close(got, want.data, frac=1e-4, what="X_attn")


def test_accumulators_via_fp_output_and_sq_scale(h):
    # FP16 output = acc * s_p * s_v: checks the INT32 P_u8 V accumulators up to the rare P_u8 tie
    B, S, nh, dh = 2, 256, 2, 64
    qkv, H = _qkv(B, S, nh, dh, 7)
    s_q, s_k, s_v = _scales(dh)
    s_p = 1.0 / 255
    want = _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, s_p, O.OutSpec("fp", dtype="f16"))
    got = _run(h, qkv, B, S, nh, dh, s_q, s_k, s_v, s_p, O.OutSpec("fp", dtype="f16"))
    assert rel_err(got, want.data) < 2e-3
    s_attn = float(Q.calib_scale(np.abs(want.data).max()))
    spec = O.OutSpec("sq", scale=s_attn)
    want_q = _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, s_p, spec)
    got_q = _run(h, qkv, B, S, nh, dh, s_q, s_k, s_v, s_p, spec)
    assert_int8_close(got_q, want_q.data, frac=1e-4, what="X_attn (SQ)")


def test_key_length_mask_and_fully_masked_sequence(h):
    B, S, nh, dh = 3, 256, 2, 64
    qkv, H = _qkv(B, S, nh, dh, 8)
    s_q, s_k, s_v = _scales(dh)
    key_len = [256, 77, 0]
    spec = O.OutSpec("fwq", scale=np.full(H, 0.02))
    want = _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, 1.0 / 255, spec, "none", key_len)
    got = _run(h, qkv, B, S, nh, dh, s_q, s_k, s_v, 1.0 / 255, spec, "none", key_len)
    assert_int8_close(got, want.data, frac=1e-4, what="key_len")
    assert np.all(got[2 * S:] == 0)                       # a fully masked row outputs 0


def test_closed_forms_on_device(h):
    # uniform logits (q = 0): P = 1/S, P_u8 = RNE(255/S) -> acc = P_u8 * column sum of V, exactly
    B, S, nh, dh = 1, 384, 2, 64
    qkv, H = _qkv(B, S, nh, dh, 9)
    qkv[:, :H] = 0
    s_v = 0.03
    got = _run(h, qkv, B, S, nh, dh, 0.1, 0.1, s_v, 1.0 / 255, O.OutSpec("fp", dtype="f16"))
    colsum = qkv[:, 2 * H:].astype(np.int64).sum(0)
    want = Q.round_to_storage((1.0 / 255) * s_v * 1 * colsum, "f16")       # RNE(255/384) = 1
    assert np.allclose(got, np.broadcast_to(want, got.shape), rtol=1e-3, atol=1e-6)
    # causal row 0 attends to key 0 only: X_attn[0] = Qs(s_v V[0]; S_attn)
    qkv, H = _qkv(B, S, nh, dh, 10)
    spec = O.OutSpec("fwq", scale=np.full(H, 0.05))
    got = _run(h, qkv, B, S, nh, dh, 0.03, 0.03, s_v, 1.0 / 255, spec, "causal")
    assert np.array_equal(got[0], Q.quant_sym(s_v * qkv[0, 2 * H:].astype(float), 0.05))


def test_saturating_static_scale(h):
    # s_p smaller than max P / 255: large probabilities clip at 255, exactly as the oracle's Qu
    B, S, nh, dh = 1, 128, 2, 64
    qkv, H = _qkv(B, S, nh, dh, 11, spread=60)
    s_q, s_k, s_v = _scales(dh, spread=30)              # sharper softmax
    raw = _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, 0.25 / 255, O.OutSpec("fp", dtype="f64")).data
    spec = O.OutSpec("fwq", scale=_calib(raw))
    want, it = _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, 0.25 / 255, spec, internals=True)
    assert max(int(v.max()) for v in it["P_u8"].values()) == 255
    got = _run(h, qkv, B, S, nh, dh, s_q, s_k, s_v, 0.25 / 255, spec)
    # (a finer s_p brings every P code closer to a rounding tie of the fp32 exponential; measured: still no mismatch)
    assert_int8_close(got, want.data, frac=1e-4, what="clipped P")


def test_refusals(h):
    x = torch.zeros(128, 3 * 96, dtype=torch.int8, device="cuda")
    out = torch.zeros(128, 96, dtype=torch.int8, device="cuda")
    sc = torch.ones(96, device="cuda")
    with pytest.raises(hero.HeroError) as e:           # dh = 48 unsupported
        h.hero_int8_attention(x[:, :96], x[:, 96:192], x[:, 192:], 1, 128, 2, 48, hero.tensor(out, "fwq", sc))
    assert e.value.status == hero.ERR_UNSUPPORTED
    x = torch.zeros(128, 3 * 128, dtype=torch.int8, device="cuda")
    out = torch.zeros(128, 128, dtype=torch.int8, device="cuda")
    rs = torch.ones(128, device="cuda")
    with pytest.raises(hero.HeroError) as e:           # token-wise X_attn refused
        h.hero_int8_attention(x[:, :128], x[:, 128:256], x[:, 256:], 1, 128, 2, 64, hero.tensor(out, "twq", rs))
    assert e.value.status == hero.ERR_UNSUPPORTED


# ------------------------------------------------------------------ FP16 / BF16 attention (module left in FP mode, Table 1)
@pytest.mark.parametrize("fp", ["f16", "bf16"])
@pytest.mark.parametrize("B,S,nh,dh,mask", [(2, 128, 2, 64, "none"), (1, 384, 3, 64, "causal"), (2, 200, 2, 128, "none"),
                                            (1, 512, 2, 128, "causal")])
def test_fp_attention(h, fp, B, S, nh, dh, mask):
    from gpu_util import TORCH_FP
    g = W.rng(3, 500 + S + dh)
    H = nh * dh
    qkv = Q.round_to_storage(g.standard_normal((B * S, 3 * H)), fp)
    want = O.attention_fp(qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:], B, S, nh, dh, O.OutSpec("fp", dtype=fp), mask=mask)
    t = dev(qkv, TORCH_FP[fp])
    out = torch.full((B * S, H), float("nan"), dtype=TORCH_FP[fp], device="cuda")
    h.hero_int8_attention(t[:, :H], t[:, H:2 * H], t[:, 2 * H:], B, S, nh, dh, hero.tensor(out), mask=mask)
    h.check()
    # P is stored in FP16 / BF16 before the second GEMM (as any fused FP attention does): that rounding, not the
    # accumulation, sets the error
    assert rel_err(out.float().cpu().numpy(), want.data) < (2e-3 if fp == "f16" else 1e-2)
    # FP attention feeding an INT8 attention-output linear: quantized by S_attn in the epilogue
    raw = O.attention_fp(qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:], B, S, nh, dh, O.OutSpec("fp", dtype="f64"), mask=mask).data
    S_attn = Q.calib_scale(np.abs(raw).max(0))
    want_q = O.attention_fp(qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:], B, S, nh, dh, O.OutSpec("fwq", scale=S_attn), mask=mask)
    out_q = torch.full((B * S, H), -99, dtype=torch.int8, device="cuda")
    h.hero_int8_attention(t[:, :H], t[:, H:2 * H], t[:, 2 * H:], B, S, nh, dh, hero.tensor(out_q, "fwq", f32(S_attn)), mask=mask)
    h.check()
    frac, mx = int8_mismatch(out_q.cpu().numpy(), want_q.data)
    # P rounded to FP16 / BF16 perturbs X_attn by up to ~2^-11 / 2^-8 relative, i.e. a visible fraction of an INT8 step
    assert mx <= 1 and frac < (0.02 if fp == "f16" else 0.12), (frac, mx)


# ------------------------------------------------------------------ row-max-normalised P (the long-sequence-robust quantizer)
ROWMAX_CASES = [(1, 128, 2, 64, "none"), (2, 384, 4, 64, "none"), (1, 512, 2, 64, "none"), (1, 256, 2, 128, "causal"),
                (2, 100, 3, 64, "none"), (1, 333, 2, 128, "causal"), (3, 40, 2, 64, "causal"), (1, 512, 2, 128, "none"),
                (1, 1024, 1, 128, "causal"), (1, 640, 2, 64, "none"), (2, 777, 1, 64, "causal")]     # the last three: two-sweep kernel


@pytest.mark.parametrize("B,S,nh,dh,mask", ROWMAX_CASES)
def test_rowmax_p_quantizer_fwq_and_fp_output(h, B, S, nh, dh, mask):
    qkv, H = _qkv(B, S, nh, dh, 900 + S + dh)
    s_q, s_k, s_v = _scales(dh)
    raw = _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, 1.0, O.OutSpec("fp", dtype="f64"), mask, p_mode="rowmax").data
    spec = O.OutSpec("fwq", scale=_calib(raw))
    want = _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, 1.0, spec, mask, p_mode="rowmax")
    got = _run(h, qkv, B, S, nh, dh, s_q, s_k, s_v, 0.0, spec, mask, p_mode="rowmax")      # s_p is ignored
    assert_int8_close(got, want.data, frac=1e-4, what="X_attn (rowmax)")
    got = _run(h, qkv, B, S, nh, dh, s_q, s_k, s_v, 0.0, O.OutSpec("fp", dtype="f16"), mask, p_mode="rowmax")
    assert rel_err(got, raw) < 2e-3


def test_rowmax_p_quantizer_key_lengths_and_flat_rows(h):
    B, S, nh, dh = 3, 384, 2, 64
    qkv, H = _qkv(B, S, nh, dh, 950)
    s_q, s_k, s_v = _scales(dh)
    key_len = [384, 130, 0]                                        # full, ragged inside a block, nothing allowed
    raw = _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, 1.0, O.OutSpec("fp", dtype="f64"), "none", key_len, p_mode="rowmax").data
    spec = O.OutSpec("fwq", scale=_calib(raw))
    want = _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, 1.0, spec, "none", key_len, p_mode="rowmax")
    got = _run(h, qkv, B, S, nh, dh, s_q, s_k, s_v, 0.0, spec, "none", key_len, p_mode="rowmax")
    assert_int8_close(got, want.data, frac=1e-4, what="X_attn (rowmax, key_len)")
    assert not got[2 * S:].any()
    # q = 0: every allowed key gets P~ = 255 and the output is the mean of V, which the static quantizer cannot do at S = 512
    B, S, nh, dh = 1, 512, 1, 64
    qkv, H = _qkv(B, S, nh, dh, 951)
    qkv[:, :H] = 0
    got = _run(h, qkv, B, S, nh, dh, s_q, s_k, s_v, 0.0, O.OutSpec("fp", dtype="f16"), p_mode="rowmax")
    mean_v = s_v * qkv[:, 2 * H:].astype(np.float64).mean(0)
    assert rel_err(got, np.broadcast_to(mean_v, got.shape)) < 2e-3


# ------------------------------------------------------------------ the on-chip intermediates, written out for verification
PROBE_CASES = [  # B, S, nh, dh, mask, p_mode, key_len
    (2, 128, 2, 64, "none", "static", None), (2, 384, 3, 64, "none", "static", None), (1, 512, 2, 64, "none", "static", None),
    (1, 256, 2, 128, "causal", "static", None), (2, 100, 3, 64, "none", "static", None), (1, 333, 2, 128, "causal", "static", None),
    (3, 200, 2, 64, "none", "static", [200, 77, 0]),
    (1, 1024, 1, 128, "causal", "static", None), (1, 640, 2, 64, "none", "static", None),          # two-sweep kernel
    (2, 384, 2, 64, "none", "rowmax", None), (1, 777, 1, 64, "causal", "rowmax", None),
]


@pytest.mark.parametrize("B,S,nh,dh,mask,p_mode,key_len", PROBE_CASES)
def test_probe_scores_codes_and_accumulators(h, B, S, nh, dh, mask, p_mode, key_len):
    """Eq. 15-17 piece by piece: INT32 Q K^T bit-exact; P_u8 within one code on <= 1e-4 of the allowed entries;
    INT32 P_u8 V bit-exact for the codes the device itself formed; X_attn = the output stage applied to the device's
    accumulators at the INT8 bar (1 LSB on <= 1e-4)."""
    from gpu_util import report
    qkv, H = _qkv(B, S, nh, dh, 300 + S + dh)
    s_q, s_k, s_v = _scales(dh)
    s_p = 1.0 / 255
    raw, it = _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, s_p, O.OutSpec("fp", dtype="f64"), mask, key_len, internals=True, p_mode=p_mode)
    S_attn = _calib(raw.data)
    spec = O.OutSpec("fwq", scale=S_attn)
    t = dev(qkv)
    out = torch.full((B * S, H), -99, dtype=torch.int8, device="cuda")
    scores = torch.full((B * nh, S, S), -(2 ** 31), dtype=torch.int32, device="cuda")
    codes = torch.zeros((B * nh, S, S), dtype=torch.uint8, device="cuda")
    acc = torch.zeros((B * S, H), dtype=torch.int32, device="cuda")
    kl = None if key_len is None else dev(np.asarray(key_len, np.int32))
    h.hero_int8_attention(t[:, :H], t[:, H:2 * H], t[:, 2 * H:], B, S, nh, dh, hero.tensor(out, "fwq", f32(S_attn)), s_q=s_q, s_k=s_k,
                          s_v=s_v, s_p=s_p, mask=mask, key_len=kl, p_mode=p_mode, probe=(scores, codes, acc))
    h.check()
    scores, codes, acc, out = scores.cpu().numpy(), codes.cpu().numpy(), acc.cpu().numpy(), out.cpu().numpy()
    n_allowed = n_code_diff = 0
    max_code_diff = 0
    for b in range(B):
        allowed = O.attention_mask(S, mask, None if key_len is None else key_len[b])
        rows = slice(b * S, (b + 1) * S)
        for hd in range(nh):
            cols = slice(hd * dh, (hd + 1) * dh)
            q_, k_, v_ = qkv[rows, cols], qkv[rows, H + hd * dh:H + (hd + 1) * dh], qkv[rows, 2 * H + hd * dh:2 * H + (hd + 1) * dh]
            want_scores = O.int_matmul(q_, k_.T)
            got_scores = scores[b * nh + hd]
            assert np.array_equal(got_scores[allowed], want_scores[allowed]), "Q K^T accumulators differ (b=%d h=%d)" % (b, hd)
            got_codes = codes[b * nh + hd]
            assert not got_codes[~allowed].any(), "a masked key carries a non-zero code"
            d = np.abs(got_codes.astype(np.int32) - it["P_u8"][(b, hd)].astype(np.int32))[allowed]
            n_allowed += d.size
            n_code_diff += int((d != 0).sum())
            max_code_diff = max(max_code_diff, int(d.max()) if d.size else 0)
            # the device's accumulators are exactly P_u8 V for the device's own codes
            assert np.array_equal(acc[rows, cols], O.int_matmul(got_codes, v_)), "P V accumulators differ (b=%d h=%d)" % (b, hd)
    assert max_code_diff <= 1, "a P code is off by %d" % max_code_diff
    frac = n_code_diff / max(n_allowed, 1)
    assert frac <= 1e-4, "P_u8: %.3g of the allowed entries differ" % frac
    report("P_u8 %s S=%d dh=%d %s" % (p_mode, S, dh, mask), "mismatch %.3g of %d codes (bar 1e-4), max %d" % (frac, n_allowed, max_code_diff))
    # output stage (Eq. 17) on the device's own accumulators
    if p_mode == "static":
        real = float(s_p) * float(s_v) * acc.astype(np.float64)
    else:
        # the row sum of the un-quantized exponentials is the oracle's (the device's differs from it by fp32 rounding only)
        real = np.zeros_like(raw.data)
        for b in range(B):
            allowed = O.attention_mask(S, mask, None if key_len is None else key_len[b])
            rows = slice(b * S, (b + 1) * S)
            for hd in range(nh):
                cols = slice(hd * dh, (hd + 1) * dh)
                A = (s_q * s_k / np.sqrt(dh)) * O.int_matmul(qkv[rows, cols], qkv[rows, H + hd * dh:H + (hd + 1) * dh].T).astype(np.float64)
                neg = np.where(allowed, A, -np.inf)
                m = np.max(neg, axis=-1, keepdims=True)
                e = np.where(allowed, np.exp(neg - np.where(np.isfinite(m), m, 0.0)), 0.0)
                l = e.sum(-1, keepdims=True)
                real[rows, cols] = np.where(l > 0, s_v * acc[rows, cols] / (255.0 * np.where(l > 0, l, 1.0)), 0.0)
    want = O.emit(real, spec)
    assert_int8_close(out, want.data, frac=1e-4, what="X_attn from device accumulators (%s S=%d)" % (p_mode, S))
    # and end to end against the oracle's own chain, reported with its measured fraction
    want_e2e = _oracle(qkv, B, S, nh, dh, s_q, s_k, s_v, s_p, spec, mask, key_len, p_mode=p_mode)
    assert_int8_close(out, want_e2e.data, frac=1e-4, what="X_attn end to end (%s S=%d)" % (p_mode, S))


def test_probe_refuses_other_operand_types(h):
    x = torch.zeros(128, 3 * 128, dtype=torch.float16, device="cuda")
    out = torch.zeros(128, 128, dtype=torch.float16, device="cuda")
    acc = torch.zeros(128, 128, dtype=torch.int32, device="cuda")
    with pytest.raises(hero.HeroError) as e:
        h.hero_int8_attention(x[:, :128], x[:, 128:256], x[:, 256:], 1, 128, 2, 64, hero.tensor(out), probe=(None, None, acc))
    assert e.value.status == hero.ERR_UNSUPPORTED
