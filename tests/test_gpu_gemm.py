"""GPU parity: hero_w8a8_linear against the oracle's GeMM^quant (Eq. 14, 18, 22, 28-30)."""
import numpy as np
import pytest
import torch

from oracle import ops as O
from oracle import quant as Q
from paper_2310_17723_b200 import hero, workloads as W
from gpu_util import dev, f32, assert_int8_close, rel_err, TORCH_FP

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def h():
    hd = hero.Handle()
    yield hd
    hd.check()
    hd.close()


def _linear(h, A, Wt, out_dtype, rs=None, cs=None, bias=None, act="none", post=None, N=None):
    M = A.shape[0]
    N = Wt.shape[0]
    tA = dev(A) if A.dtype == np.int8 else A
    tW = dev(Wt) if isinstance(Wt, np.ndarray) else Wt
    out = torch.full((M, N), -77, dtype=out_dtype, device="cuda") if out_dtype in (torch.int8, torch.int32) else \
        torch.full((M, N), float("nan"), dtype=out_dtype, device="cuda")
    a_desc = hero.tensor(tA, "twq", f32(rs)) if rs is not None else hero.tensor(tA)
    h.hero_w8a8_linear(a_desc, tW, hero.tensor(out), w_scale=None if cs is None else f32(cs),
                       bias=None if bias is None else f32(bias), act=act, post_scale=None if post is None else f32(post))
    h.check()
    return out


# shapes span one tile, several tiles, ragged M / N / K tails and every column-tile width
# (the last three are large enough to take the CTA-pair kernel: 256 x 256 tiles, ragged in M and N)
SHAPES = [(128, 128, 256), (1, 64, 16), (17, 80, 48), (127, 256, 272), (129, 1024, 512), (300, 768, 2304),
          (1000, 4096, 1024), (16, 4096, 4096), (2500, 512, 4096), (600, 128, 7984), (12288, 1024, 1024)]


@pytest.mark.parametrize("M,K,N", SHAPES)
def test_int32_accumulators_bit_exact(h, M, K, N):
    g = W.rng(2, 1000 + M + K + N)
    A = g.integers(-127, 128, (M, K), dtype=np.int8)
    Wt = g.integers(-127, 128, (N, K), dtype=np.int8)
    got = _linear(h, A, Wt, torch.int32).cpu().numpy()
    want = O.int_matmul(A, Wt.T.copy())
    assert np.array_equal(got, want)


def test_many_distinct_buffers_then_the_first_again(h):
    # more distinct operand / output buffers than the handle keeps tensor maps for: every call must describe ITS buffers
    # (a stale or colliding descriptor would read or write another tensor), and coming back to the first buffers, whose
    # maps have been displaced meanwhile, must give the first result again
    g = W.rng(2, 4242)
    M, K, N = 160, 192, 320
    As = [dev(g.integers(-127, 128, (M, K), dtype=np.int8)) for _ in range(150)]
    Wt = g.integers(-127, 128, (N, K), dtype=np.int8)
    tW = dev(Wt)
    outs = [torch.full((M, N), -77, dtype=torch.int32, device="cuda") for _ in range(len(As))]
    for a, o in zip(As, outs):
        h.hero_w8a8_linear(hero.tensor(a), tW, hero.tensor(o))
    again = torch.full((M, N), -77, dtype=torch.int32, device="cuda")
    h.hero_w8a8_linear(hero.tensor(As[0]), tW, hero.tensor(again))
    h.check()
    Wf = tW.double().T
    for i in (0, 1, 63, 127, 128, 149):
        want = (As[i].double() @ Wf).to(torch.int32)                 # exact: |sum| < 2^53
        assert torch.equal(outs[i], want), i
    assert torch.equal(again, outs[0])


def test_int32_extreme_values_bit_exact(h):
    M, K, N = 130, 16384, 64
    A = np.full((M, K), 127, np.int8)
    Wt = np.full((N, K), -127, np.int8)
    Wt[1::2] = 127
    got = _linear(h, A, Wt, torch.int32).cpu().numpy()
    assert np.array_equal(got, O.int_matmul(A, Wt.T.copy()))


# (1300, 512, N): the CTA-pair kernel's staged 8-bit output (short K) with a ragged last row-tile and a last column-tile
# whose second 128-column half is partly (N = 2000), barely (1936) or not at all (1888) inside the matrix
@pytest.mark.parametrize("M,K,N", [(128, 1024, 4096), (333, 4096, 1024), (16, 1024, 4096), (1024, 1024, 4096), (1500, 256, 4096),
                                   (1300, 512, 2000), (1300, 512, 1936), (1300, 512, 1888), (2304, 4096, 1024)])
def test_requant_epilogue_round_only(h, M, K, N):
    # Eq. 22: dequantize by row and column scale, add the folded bias, Round -> INT8
    A, Wt, rs, cs, bias = W.gemm_case(M, K, N)
    x = O.QT("i8", A, row_scale=rs.astype(np.float64))
    want = O.gemm_quant(x, Wt.T.copy(), cs, bias, "none", O.OutSpec("round"))
    got = _linear(h, A, Wt, torch.int8, rs=rs, cs=cs, bias=bias).cpu().numpy()
    assert_int8_close(got, want.data, what="requant epilogue")
    assert np.abs(want.data.astype(int)).max() > 60      # the case exercises a wide code range


@pytest.mark.parametrize("act", ["gelu_erf", "gelu_tanh"])
@pytest.mark.parametrize("M", [260, 1100])
def test_fc1_gelu_quant_epilogue(h, act, M):
    # Eq. 28-29: X_1 stays FP32 on chip, GELU, then FWQ with 1 / S_a
    K, N = 768, 3072
    g = W.rng(2, 555)
    A = g.integers(-127, 128, (M, K), dtype=np.int8)
    Wt = g.integers(-127, 128, (N, K), dtype=np.int8)
    rs = (g.uniform(0.5, 1.5, M) * 0.02).astype(np.float32)
    cs = (g.uniform(0.5, 1.5, N) * 1.5e-4 / np.sqrt(K / 768)).astype(np.float32)
    bias = (g.standard_normal(N) * 0.1).astype(np.float32)
    x = O.QT("i8", A, row_scale=rs.astype(np.float64))
    v = O.gemm_quant(x, Wt.T.copy(), cs, bias, act, O.OutSpec("fp", dtype="f64")).data
    S_a = Q.calib_scale(np.abs(v).max(0))
    want = O.gemm_quant(x, Wt.T.copy(), cs, bias, act, O.OutSpec("fwq", scale=S_a))
    inv = (1.0 / S_a).astype(np.float32)
    got = _linear(h, A, Wt, torch.int8, rs=rs, cs=cs, bias=bias, act=act, post=inv).cpu().numpy()
    assert_int8_close(got, want.data, what="GELU^quant")


@pytest.mark.parametrize("M,K,N", [(1100, 768, 3072), (200, 512, 256)])
def test_fc1_gelu_quant_saturates_both_ways(h, M, K, N):
    # output factors far too large for the data (a mis-calibrated 1 / S_a): GELU(v) / S_a leaves [-127, 127] on both
    # sides, the lower one only because the factor exceeds 127 / 0.17; the codes must saturate exactly as the oracle's
    g = W.rng(2, 777 + M)
    A = g.integers(-127, 128, (M, K), dtype=np.int8)
    Wt = g.integers(-127, 128, (N, K), dtype=np.int8)
    rs = (g.uniform(0.5, 1.5, M) * 0.02).astype(np.float32)
    cs = (g.uniform(0.5, 1.5, N) * 1.5e-4 / np.sqrt(K / 768)).astype(np.float32)
    bias = (g.standard_normal(N) * 0.1).astype(np.float32)
    S_a = np.full(N, 1.0 / 40.0)
    S_a[::3] = 1.0 / 2000.0                                 # every third column: -0.17 * 2000 < -127
    x = O.QT("i8", A, row_scale=rs.astype(np.float64))
    want = O.gemm_quant(x, Wt.T.copy(), cs, bias, "gelu_erf", O.OutSpec("fwq", scale=S_a)).data
    assert (want == -127).any() and (want == 127).any()
    got = _linear(h, A, Wt, torch.int8, rs=rs, cs=cs, bias=bias, act="gelu_erf", post=(1.0 / S_a).astype(np.float32)).cpu().numpy()
    assert_int8_close(got, want, what="GELU^quant, saturating")


@pytest.mark.parametrize("fp", ["f16", "bf16"])
def test_int8_gemm_fp_output(h, fp):
    # an INT8 module whose consumer is in FP mode: dequantize + bias only, stored in FP16 / BF16
    M, K, N = 200, 1024, 1024
    A, Wt, rs, cs, bias = W.gemm_case(M, K, N)
    x = O.QT("i8", A, row_scale=rs.astype(np.float64))
    want = O.gemm_quant(x, Wt.T.copy(), cs, bias, "none", O.OutSpec("fp", dtype=fp))
    got = _linear(h, A, Wt, TORCH_FP[fp], rs=rs, cs=cs, bias=bias).float().cpu().numpy()
    assert rel_err(got, want.data) < (1e-2 if fp == "bf16" else 2e-3)
    assert np.mean(got != want.data) < 2e-3            # equal up to rare 1-ulp rounding ties


@pytest.mark.parametrize("fp", ["f16", "bf16"])
@pytest.mark.parametrize("M,K,N", [(128, 64, 256), (200, 1024, 768), (77, 136, 48), (1030, 256, 4096)])
def test_fp_mode_gemm(h, fp, M, K, N):
    # a module left in FP16/BF16 (Table 1): X W + b with fp32 accumulation
    g = W.rng(2, 777 + M)
    A = Q.round_to_storage(g.standard_normal((M, K)), fp)
    Wm = Q.round_to_storage(g.standard_normal((K, N)) * 0.05, fp)
    bias = (g.standard_normal(N) * 0.1).astype(np.float32)
    want = O.gemm_fp(O.fp_tensor(A, fp), Wm, bias, "gelu_erf", O.OutSpec("fp", dtype=fp))
    tA = dev(A, TORCH_FP[fp])
    tW = dev(Wm.T.copy(), TORCH_FP[fp])
    got = _linear(h, tA, tW, TORCH_FP[fp], bias=bias, act="gelu_erf").float().cpu().numpy()
    assert rel_err(got, want.data) < (1e-2 if fp == "bf16" else 2e-3)
    # FP GEMM that feeds an INT8 consumer: quantized in the epilogue with 1 / S
    y = O.gemm_fp(O.fp_tensor(A, fp), Wm, bias, "none", O.OutSpec("fp", dtype="f64")).data
    S = Q.calib_scale(np.abs(y).max(0))
    want_q = O.gemm_fp(O.fp_tensor(A, fp), Wm, bias, "none", O.OutSpec("fwq", scale=S))
    got_q = _linear(h, tA, tW, torch.int8, bias=bias, post=(1.0 / S).astype(np.float32)).cpu().numpy()
    assert_int8_close(got_q, want_q.data, frac=1e-4, what="FP GEMM -> INT8")


def test_strided_views_and_untouched_padding(h):
    # A and out are column slices of wider buffers (ld > cols); bytes outside the view stay untouched
    M, K, N = 150, 256, 128
    g = W.rng(2, 888)
    Abig = torch.from_numpy(g.integers(-127, 128, (M, K + 64), dtype=np.int8)).cuda()
    Wt = g.integers(-127, 128, (N, K), dtype=np.int8)
    outbig = torch.full((M, N + 32), 99, dtype=torch.int32, device="cuda")
    h.hero_w8a8_linear(hero.tensor(Abig[:, :K]), dev(Wt), hero.tensor(outbig[:, :N]))
    h.check()
    want = O.int_matmul(Abig[:, :K].cpu().numpy(), Wt.T.copy())
    assert np.array_equal(outbig[:, :N].cpu().numpy(), want)
    assert torch.all(outbig[:, N:] == 99)


def test_refusals(h):
    A = torch.zeros(8, 64, dtype=torch.int8, device="cuda")
    Wt = torch.zeros(32, 64, dtype=torch.int8, device="cuda")
    cs = torch.ones(32, device="cuda")
    out = torch.zeros(8, 32, dtype=torch.int8, device="cuda")
    sc = torch.zeros(8, device="cuda")
    with pytest.raises(hero.HeroError) as e:      # token-wise output from a GEMM epilogue: refused (Sec. 2.1)
        h.hero_w8a8_linear(hero.tensor(A), Wt, hero.tensor(out, "twq", sc), w_scale=cs)
    assert e.value.status == hero.ERR_UNSUPPORTED
    with pytest.raises(hero.HeroError) as e:      # K not a multiple of 16 bytes
        h.hero_w8a8_linear(hero.tensor(A[:, :40]), Wt[:, :40], hero.tensor(out), w_scale=cs)
    assert e.value.status in (hero.ERR_UNSUPPORTED, hero.ERR_ALIGNMENT)
    empty = torch.zeros(0, 64, dtype=torch.int8, device="cuda")
    h.hero_w8a8_linear(hero.tensor(empty), Wt, hero.tensor(torch.zeros(0, 32, dtype=torch.int8, device="cuda")), w_scale=cs)


# ------------------------------------------------------------------------------------------------------------------
# few rows (M <= 128): the weight-streaming kernel with the K dimension split over a thread-block cluster
# ------------------------------------------------------------------------------------------------------------------
# (the library takes this kernel for M <= 16, and for M <= 128 when K is long and N leaves SMs idle: every case below does)
# every row-tile width (16 / 32 / 64 / 128), 1 to 8 K splits (K = 80 .. 16384 bytes), uneven splits (33, 65, 73 K steps),
# ragged feature tiles (N = 16, 144, 2064), ragged K (80, 9232)
FEW_ROWS = [(1, 128, 16), (1, 16384, 4096), (5, 1024, 144), (16, 4096, 4096), (17, 4224, 768), (16, 80, 2064),
            (33, 8320, 768), (64, 9232, 1024), (100, 16384, 256), (128, 8192, 3072)]


@pytest.mark.parametrize("M,K,N", FEW_ROWS)
def test_few_rows_int32_accumulators_bit_exact(h, M, K, N):
    g = W.rng(2, 3000 + M + K + N)
    A = g.integers(-127, 128, (M, K), dtype=np.int8)
    Wt = g.integers(-127, 128, (N, K), dtype=np.int8)
    got = _linear(h, A, Wt, torch.int32).cpu().numpy()
    assert np.array_equal(got, O.int_matmul(A, Wt.T.copy()))


@pytest.mark.parametrize("M,K,N", [(1, 4096, 4096), (8, 1024, 3072), (16, 16384, 4096), (48, 8192, 1024), (128, 16384, 1024)])
def test_few_rows_requant_epilogue(h, M, K, N):
    A, Wt, rs, cs, bias = W.gemm_case(M, K, N)
    x = O.QT("i8", A, row_scale=rs.astype(np.float64))
    want = O.gemm_quant(x, Wt.T.copy(), cs, bias, "none", O.OutSpec("round"))
    got = _linear(h, A, Wt, torch.int8, rs=rs, cs=cs, bias=bias).cpu().numpy()
    assert_int8_close(got, want.data, what="few rows, requant epilogue")
    want_fp = O.gemm_quant(x, Wt.T.copy(), cs, bias, "none", O.OutSpec("fp", dtype="bf16"))
    got_fp = _linear(h, A, Wt, torch.bfloat16, rs=rs, cs=cs, bias=bias).float().cpu().numpy()
    assert rel_err(got_fp, want_fp.data) < 1e-2 and np.mean(got_fp != want_fp.data) < 2e-3


@pytest.mark.parametrize("act", ["gelu_erf", "gelu_tanh"])
@pytest.mark.parametrize("M", [3, 16, 40, 128])
def test_few_rows_fc1_gelu_quant(h, act, M):
    K, N = (1024 if M <= 16 else 8192), 4096
    g = W.rng(2, 556 + M)
    A = g.integers(-127, 128, (M, K), dtype=np.int8)
    Wt = g.integers(-127, 128, (N, K), dtype=np.int8)
    rs = (g.uniform(0.5, 1.5, M) * 0.02).astype(np.float32)
    cs = (g.uniform(0.5, 1.5, N) * 1.5e-4 / np.sqrt(K / 768)).astype(np.float32)
    bias = (g.standard_normal(N) * 0.1).astype(np.float32)
    x = O.QT("i8", A, row_scale=rs.astype(np.float64))
    v = O.gemm_quant(x, Wt.T.copy(), cs, bias, act, O.OutSpec("fp", dtype="f64")).data
    S_a = Q.calib_scale(np.abs(v).max(0))
    want = O.gemm_quant(x, Wt.T.copy(), cs, bias, act, O.OutSpec("fwq", scale=S_a))
    got = _linear(h, A, Wt, torch.int8, rs=rs, cs=cs, bias=bias, act=act, post=(1.0 / S_a).astype(np.float32)).cpu().numpy()
    assert_int8_close(got, want.data, frac=1e-4, what="few rows, GELU^quant")


@pytest.mark.parametrize("fp", ["f16", "bf16"])
@pytest.mark.parametrize("M,K,N", [(2, 2048, 512), (20, 2048, 48), (128, 4096, 1024)])
def test_few_rows_fp_mode_gemm(h, fp, M, K, N):
    g = W.rng(2, 778 + M)
    A = Q.round_to_storage(g.standard_normal((M, K)), fp)
    Wm = Q.round_to_storage(g.standard_normal((K, N)) * 0.05, fp)
    bias = (g.standard_normal(N) * 0.1).astype(np.float32)
    want = O.gemm_fp(O.fp_tensor(A, fp), Wm, bias, "gelu_erf", O.OutSpec("fp", dtype=fp))
    tA, tW = dev(A, TORCH_FP[fp]), dev(Wm.T.copy(), TORCH_FP[fp])
    got = _linear(h, tA, tW, TORCH_FP[fp], bias=bias, act="gelu_erf").float().cpu().numpy()
    assert rel_err(got, want.data) < (1e-2 if fp == "bf16" else 2e-3)


def test_few_rows_strided_input_and_output(h):
    M, K, N = 9, 1024, 384
    g = W.rng(2, 901)
    big_a = torch.from_numpy(g.integers(-127, 128, (M, 2 * K), dtype=np.int8)).cuda()
    big_o = torch.full((M, 2 * N), -77, dtype=torch.int32, device="cuda")
    Wt = g.integers(-127, 128, (N, K), dtype=np.int8)
    h.hero_w8a8_linear(hero.tensor(big_a[:, K:]), dev(Wt), hero.tensor(big_o[:, :N]))
    h.check()
    assert np.array_equal(big_o[:, :N].cpu().numpy(), O.int_matmul(big_a[:, K:].cpu().numpy(), Wt.T.copy()))
    assert bool((big_o[:, N:] == -77).all())
