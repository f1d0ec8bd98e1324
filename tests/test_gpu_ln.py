"""GPU parity: hero_layernorm_quant against the oracle's LN^quant (Eq. 7, 19, 31), element by element."""
import numpy as np
import pytest
import torch

from oracle import ops as O
from oracle import quant as Q
from paper_2310_17723_b200 import hero, workloads as W
from gpu_util import dev, f32, qt_to_device, assert_int8_close, assert_scales_close, rel_err, TORCH_FP

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def h():
    hd = hero.Handle()
    yield hd
    hd.check()
    hd.close()


def _run(h, inputs, gamma, beta, eps, out_spec, M, H, fp_out=None, normalize=True):
    """inputs: list of oracle QT (1-3).  Returns dict with device results as numpy."""
    devs = [qt_to_device(t) for t in inputs]
    res = {}
    out_t = out_scale = None
    out_desc = None
    if normalize:
        if out_spec.kind == "fp":
            out_t = torch.empty(M, H, dtype=TORCH_FP[out_spec.dtype], device="cuda")
            out_desc = hero.tensor(out_t)
        else:
            out_t = torch.empty(M, H, dtype=torch.int8, device="cuda")
            if out_spec.kind == "twq":
                out_scale = torch.zeros(M, dtype=torch.float32, device="cuda")
            elif out_spec.kind == "fwq":
                out_scale = f32(out_spec.scale)
            else:
                out_scale = f32(np.array([out_spec.scale]))
            out_desc = hero.tensor(out_t, out_spec.kind, out_scale)
    fp_t = fp_desc = None
    if fp_out:
        fp_t = torch.empty(M, H, dtype=TORCH_FP[fp_out], device="cuda")
        fp_desc = hero.tensor(fp_t)
    g, b = f32(gamma), f32(beta)
    h.hero_layernorm_quant(devs[0][1], g, b, eps, out_desc, branch=devs[1][1] if len(devs) > 1 else None,
                           extra=devs[2][1] if len(devs) > 2 else None, fp_out=fp_desc)
    h.check()
    if out_t is not None:
        res["out"] = out_t.float().cpu().numpy() if out_spec.kind == "fp" else out_t.cpu().numpy()
    if out_spec is not None and out_spec.kind == "twq" and normalize:
        res["scale"] = out_scale.cpu().numpy()
    if fp_t is not None:
        res["fp_out"] = fp_t.float().cpu().numpy()
    return res


def _compare(res, want, want_r, out_spec):
    if want is not None:
        if out_spec.kind == "fp":
            assert rel_err(res["out"], want.data) < 2e-3
        else:
            assert_int8_close(res["out"], want.data, what="LN out")
            if out_spec.kind == "twq":
                assert_scales_close(res["scale"], want.row_scale, 1e-6, "LN row scales")
    if want_r is not None:
        # fp16/bf16 store of an fp32 sum vs the oracle's fp64 sum: equal except rare 1-ulp ties
        d = np.abs(res["fp_out"] - want_r.data)
        assert np.mean(d != 0) < 1e-3 and rel_err(res["fp_out"], want_r.data) < 8e-3


@pytest.mark.parametrize("M,H", [(128, 768), (37, 1024), (1, 768), (2100, 768), (300, 4096), (65, 8192), (129, 80), (7, 16384), (40, 2048), (33, 5120)])
def test_plain_fp16_to_twq(h, M, H):
    x, gamma, beta = W.ln_case(M, H)
    spec = O.OutSpec("twq")
    want, _ = O.ln_quant([O.fp_tensor(x, "f16")], gamma, beta, 1e-12, spec)
    res = _run(h, [O.fp_tensor(x, "f16")], gamma, beta, 1e-12, spec, M, H)
    _compare(res, want, None, spec)


@pytest.mark.parametrize("out_kind", ["twq", "fwq", "sq", "fp"])
@pytest.mark.parametrize("H", [768, 4096])
def test_residual_int8_twq_plus_int8_fwq(h, out_kind, H):
    # Eq. 19: LN^quant(S_in X_in,int8 , X_o,int8 S_o)
    M = 200
    g = W.rng(2, 77 + H)
    x, gamma, beta = W.ln_case(M, H)
    xin = O.emit(x, O.OutSpec("twq"))
    s_o = (np.abs(g.standard_normal(H)) * 0.01 + 0.002).astype(np.float32)
    xo = O.QT("i8", g.integers(-127, 128, (M, H), dtype=np.int8), col_scale=s_o.astype(np.float64))
    y = O.layernorm(xin.real() + xo.real(), gamma, beta, 1e-12)
    spec = {"twq": O.OutSpec("twq"), "fwq": O.OutSpec("fwq", scale=Q.calib_scale(np.abs(y).max(0))),
            "sq": O.OutSpec("sq", scale=float(Q.calib_scale(np.abs(y).max()))), "fp": O.OutSpec("fp", dtype="f16")}[out_kind]
    want, _ = O.ln_quant([xin, xo], gamma, beta, 1e-12, spec)
    res = _run(h, [xin, xo], gamma, beta, 1e-12, spec, M, H)
    _compare(res, want, None, spec)


@pytest.mark.parametrize("out_kind", ["twq", "fwq", "fp"])
@pytest.mark.parametrize("M,H", [(1, 1024), (33, 1024), (4737, 1024), (1, 768), (33, 768), (4737, 768)])
def test_two_rows_per_warp_odd_row_counts_and_untouched_tail(h, M, H, out_kind):
    # rows of 1024 / 768 are processed two per warp: an odd row count leaves the last warp with one row, several passes of
    # the grid (4737 rows) make that happen in the last pass only; nothing beyond row M - 1 may be written
    g = W.rng(2, 500 + M + H)
    x, gamma, beta = W.ln_case(M, H)
    xin = O.emit(x, O.OutSpec("twq"))
    s_o = (np.abs(g.standard_normal(H)) * 0.01 + 0.002).astype(np.float32)
    xo = O.QT("i8", g.integers(-127, 128, (M, H), dtype=np.int8), col_scale=s_o.astype(np.float64))
    y = O.layernorm(xin.real() + xo.real(), gamma, beta, 1e-12)
    spec = {"twq": O.OutSpec("twq"), "fwq": O.OutSpec("fwq", scale=Q.calib_scale(np.abs(y).max(0))),
            "fp": O.OutSpec("fp", dtype="f16")}[out_kind]
    want, _ = O.ln_quant([xin, xo], gamma, beta, 1e-12, spec)
    din, do = qt_to_device(xin), qt_to_device(xo)
    pad = 3
    if out_kind == "fp":
        full = torch.full((M + pad, H), 7.0, dtype=torch.float16, device="cuda")
        desc = hero.tensor(full[:M])
        sc = None
    else:
        full = torch.full((M + pad, H), 77, dtype=torch.int8, device="cuda")
        sc = torch.full((M + pad,), -5.0, dtype=torch.float32, device="cuda") if out_kind == "twq" else f32(spec.scale)
        desc = hero.tensor(full[:M], out_kind, sc[:M] if out_kind == "twq" else sc)
    h.hero_layernorm_quant(din[1], f32(gamma), f32(beta), 1e-12, desc, branch=do[1])
    h.check()
    if out_kind == "fp":
        assert rel_err(full[:M].float().cpu().numpy(), want.data) < 2e-3
        assert bool((full[M:] == 7.0).all())
    else:
        assert_int8_close(full[:M].cpu().numpy(), want.data, what="LN out")
        assert bool((full[M:] == 77).all())
        if out_kind == "twq":
            assert_scales_close(sc[:M].cpu().numpy(), want.row_scale, 1e-6, "LN row scales")
            assert bool((sc[M:] == -5.0).all())


@pytest.mark.parametrize("res_kind,br_kind", [("i8_twq", "f16"), ("f16", "f16"), ("bf16", "i8_fwq"), ("i8_fwq", "i8_fwq"),
                                              ("i8_sq", "bf16")])
@pytest.mark.parametrize("H", [1024, 768])        # two chunks of 16 elements per lane / three chunks of 8
def test_mixed_input_types(h, res_kind, br_kind, H):
    M = 96
    g = W.rng(2, 99)
    x, gamma, beta = W.ln_case(M, H)

    def make(kind, data):
        if kind in ("f16", "bf16"):
            return O.fp_tensor(data, kind)
        if kind == "i8_twq":
            return O.emit(data, O.OutSpec("twq"))
        if kind == "i8_fwq":
            return O.emit(data, O.OutSpec("fwq", scale=Q.calib_scale(np.abs(data).max(0))))
        return O.emit(data, O.OutSpec("sq", scale=float(Q.calib_scale(np.abs(data).max()))))

    a = make(res_kind, x)
    b = make(br_kind, g.standard_normal((M, H)) * 0.5)
    spec = O.OutSpec("twq")
    want, _ = O.ln_quant([a, b], gamma, beta, 1e-5, spec)
    res = _run(h, [a, b], gamma, beta, 1e-5, spec, M, H)
    _compare(res, want, None, spec)


@pytest.mark.parametrize("fp", ["f16", "bf16"])
@pytest.mark.parametrize("M,H", [(150, 4096), (150, 768), (151, 1024), (2401, 768)])     # (odd counts: two rows per warp)
def test_pre_ln_dual_output_and_bare_add(h, fp, M, H):
    g = W.rng(2, 123)
    hres = O.fp_tensor(g.standard_normal((M, H)), fp)
    br = O.QT("i8", g.integers(-127, 128, (M, H), dtype=np.int8),
              col_scale=(np.abs(g.standard_normal(H)) * 0.01 + 0.002).astype(np.float32).astype(np.float64))
    gamma, beta = np.ones(H, np.float32), np.zeros(H, np.float32)
    spec = O.OutSpec("twq")
    _, want_r = O.ln_quant([hres, br], gamma, beta, 1e-5, spec, fp_out_dtype=fp)
    res = _run(h, [hres, br], gamma, beta, 1e-5, spec, M, H, fp_out=fp)
    # (1) the stored residual stream equals the oracle's up to rare 1-ulp ties of the fp32 sum;
    _compare(res, None, want_r, spec)
    # (2) the device normalises ITS stored sum (one bf16 ulp on the row's largest element would move the whole
    # row's scale), so the quantized output is checked against the oracle applied to that same stored tensor
    want, _ = O.ln_quant([O.fp_tensor(res["fp_out"], fp)], gamma, beta, 1e-5, spec)
    _compare(res, want, None, spec)
    _, want_r2 = O.ln_quant([hres, br], None, None, 0.0, None, fp_out_dtype=fp, normalize=False)
    res2 = _run(h, [hres, br], gamma, beta, 0.0, spec, M, H, fp_out=fp, normalize=False)
    _compare(res2, None, want_r2, spec)


def test_embedding_gather_flavour(h):
    # Eq. 7: LN^quant(S_xt X_t,int8 , X_p , X_s) with the token row gathered by id
    V, P, T, H, S, B = 500, 64, 2, 768, 64, 3
    g = W.rng(0, 41)
    tok, pos, typ = W.embedding_tables(V, P, T, H)
    tok_q, tok_s = Q.quant_twq(tok)
    ids = g.integers(0, V, B * S).astype(np.int32)
    tids = g.integers(0, T, B * S).astype(np.int32)
    gamma = (1 + 0.1 * g.standard_normal(H)).astype(np.float32)
    beta = (0.1 * g.standard_normal(H)).astype(np.float32)
    want = O.embedding_ln_quant(ids, tids, tok_q, tok_s, pos, typ, S, gamma, beta, 1e-12, O.OutSpec("twq"))
    t_tok, t_pos, t_typ = dev(tok_q), dev(pos, torch.float16), dev(typ, torch.float16)
    s_tok = f32(tok_s)
    out = torch.empty(B * S, H, dtype=torch.int8, device="cuda")
    sc = torch.zeros(B * S, dtype=torch.float32, device="cuda")
    h.hero_layernorm_quant(hero.tensor(t_tok, "twq", s_tok), f32(gamma), f32(beta), 1e-12, hero.tensor(out, "twq", sc),
                           branch=hero.tensor(t_pos), extra=hero.tensor(t_typ), token_ids=dev(ids), type_ids=dev(tids),
                           seq_len=S, n_tokens=B * S)
    h.check()
    assert_int8_close(out.cpu().numpy(), want.data, what="embedding LN")
    assert_scales_close(sc.cpu().numpy(), want.row_scale, 1e-6, "embedding LN row scales")


def test_embedding_gather_clamps_out_of_range_ids_and_reports_them(h):
    # a bad id from upstream must not become an out-of-bounds read: the row is taken from the nearest valid table row
    # and the next hero_check() says so
    V, P, T, H, S, B = 50, 32, 2, 768, 32, 2
    g = W.rng(0, 43)
    tok, pos, typ = W.embedding_tables(V, P, T, H)
    tok_q, tok_s = Q.quant_twq(tok)
    ids = g.integers(0, V, B * S).astype(np.int32)
    tids = g.integers(0, T, B * S).astype(np.int32)
    bad_ids, bad_tids = ids.copy(), tids.copy()
    bad_ids[3], bad_ids[40], bad_tids[17] = V + 100000, -5, T + 7
    ids[3], ids[40], tids[17] = V - 1, 0, T - 1                       # what the clamp makes of them
    gamma = (1 + 0.1 * g.standard_normal(H)).astype(np.float32)
    beta = (0.1 * g.standard_normal(H)).astype(np.float32)
    want = O.embedding_ln_quant(ids, tids, tok_q, tok_s, pos, typ, S, gamma, beta, 1e-12, O.OutSpec("twq"))
    t_tok, t_pos, t_typ = dev(tok_q), dev(pos, torch.float16), dev(typ, torch.float16)
    out = torch.empty(B * S, H, dtype=torch.int8, device="cuda")
    sc = torch.zeros(B * S, dtype=torch.float32, device="cuda")
    h.hero_layernorm_quant(hero.tensor(t_tok, "twq", f32(tok_s)), f32(gamma), f32(beta), 1e-12, hero.tensor(out, "twq", sc),
                           branch=hero.tensor(t_pos), extra=hero.tensor(t_typ), token_ids=dev(bad_ids), type_ids=dev(bad_tids),
                           seq_len=S, n_tokens=B * S)
    with pytest.raises(hero.HeroError) as e:
        h.check()
    assert e.value.status == hero.ERR_INVALID_ARG and "embedding id" in str(e.value)
    h.check()                                                          # the word was cleared
    assert_int8_close(out.cpu().numpy(), want.data, what="embedding LN, clamped ids")
    assert_scales_close(sc.cpu().numpy(), want.row_scale, 1e-6, "embedding LN row scales")
    # a position table shorter than the sequence is refused on the host
    with pytest.raises(hero.HeroError) as e:
        h.hero_layernorm_quant(hero.tensor(t_tok, "twq", f32(tok_s)), f32(gamma), f32(beta), 1e-12, hero.tensor(out, "twq", sc),
                               branch=hero.tensor(t_pos), extra=hero.tensor(t_typ), token_ids=dev(ids), type_ids=dev(tids),
                               seq_len=P + 1, n_tokens=B * S)
    assert e.value.status == hero.ERR_INVALID_ARG


def test_constant_rows_and_empty_input(h):
    H = 768
    x = np.full((4, H), 2.5, np.float32)
    gamma, beta = np.ones(H, np.float32), np.zeros(H, np.float32)
    res = _run(h, [O.fp_tensor(x, "f16")], gamma, beta, 1e-12, O.OutSpec("twq"), 4, H)
    assert np.all(res["out"] == 0) and np.all(res["scale"] == 1.0)       # LN of a constant row is beta = 0 -> zero row -> S = 1
    empty = torch.empty(0, H, dtype=torch.float16, device="cuda")
    out = torch.empty(0, H, dtype=torch.int8, device="cuda")
    sc = torch.empty(0, dtype=torch.float32, device="cuda")
    h.hero_layernorm_quant(hero.tensor(empty), f32(gamma), f32(beta), 1e-12, hero.tensor(out, "twq", sc))


def test_argument_errors(h):
    H = 768
    x = torch.zeros(4, H, dtype=torch.float16, device="cuda")
    out = torch.empty(4, H, dtype=torch.int8, device="cuda")
    sc = torch.empty(4, dtype=torch.float32, device="cuda")
    g = torch.ones(H, device="cuda")
    with pytest.raises(hero.HeroError) as e:
        h.hero_layernorm_quant(hero.tensor(x[:, :100]), g, g, 1e-5, hero.tensor(out[:, :100], "twq", sc))
    assert e.value.status in (hero.ERR_UNSUPPORTED, hero.ERR_ALIGNMENT)
    with pytest.raises(hero.HeroError) as e:
        h.hero_layernorm_quant(hero.tensor(x), g, g, 1e-5, hero.tensor(out, "none", None))
    assert e.value.status == hero.ERR_INVALID_ARG
    # an 8-bit output of either payload without its scale pointer is an argument error, caught before any launch
    n0 = h.launches
    for dt in (torch.int8, torch.float8_e4m3fn):
        o8 = torch.empty(4, H, dtype=dt, device="cuda")
        for gran in ("twq", "fwq", "sq"):
            with pytest.raises(hero.HeroError) as e:
                h.hero_layernorm_quant(hero.tensor(x), g, g, 1e-5, hero.tensor(o8, gran, None))
            assert e.value.status == hero.ERR_INVALID_ARG, (dt, gran)
    a8 = torch.zeros(4, H, dtype=torch.float8_e4m3fn, device="cuda")
    w8 = torch.zeros(64, H, dtype=torch.float8_e4m3fn, device="cuda")
    o16 = torch.empty(4, 64, dtype=torch.float16, device="cuda")
    with pytest.raises(hero.HeroError) as e:                          # e4m3 input declared token-wise, no scale given
        h.hero_w8a8_linear(hero.tensor(a8, "twq", None), w8, hero.tensor(o16), w_scale=torch.ones(64, device="cuda"))
    assert e.value.status == hero.ERR_INVALID_ARG
    assert h.launches == n0
