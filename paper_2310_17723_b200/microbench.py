"""Single-kernel micro-benchmarks of the library (also the small cases its ncu captures are taken on).

    python -m paper_2310_17723_b200.microbench ln   --M 65536 --H 1024 --kind i8       # LN^quant GB/s
    python -m paper_2310_17723_b200.microbench gemm --M 8192 --K 4096 --N 4096        # GeMM^quant TOP/s
    python -m paper_2310_17723_b200.microbench attn --B 8 --S 384 --nh 16 --dh 64     # INT8 attention
    python -m paper_2310_17723_b200.microbench absmax --M 65536 --H 4096             # calibration observer GB/s
    python -m paper_2310_17723_b200.microbench wquant --N 4096 --K 4096              # fold + Eq. 2 weight quantization GB/s
    python -m paper_2310_17723_b200.microbench decode --B 8 --S 2048 --nh 32 --dh 128 --graph   # decode attention GB/s
    python -m paper_2310_17723_b200.microbench layer-decode --workload c4 --B 8 --S 2048 --graph   # one decode step of a layer
    python -m paper_2310_17723_b200.microbench layer --workload c3 [--f8 | --fp]   # one whole layer, us per forward
    ... --sweep runs the standalone-kernel sweep of the benchmark configurations instead of one shape.

Inputs are synthetic and larger than L2 (several rotating buffers), times are CUDA events around `--iters` launches.
"""
import argparse
import json
import os

import torch

from . import hero, workloads as W


def _peaks():
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d["hbm_gbs"], 2.0 * d["bf16_tflops"], "measured"
    return 6650.0, 2.0 * 1590.0, "fallback"


GRAPH = False       # --graph: replay the launches from a CUDA graph (kernels of a few microseconds are otherwise timed at
                    # the rate the host can issue them)


def _time(fn, n_buf, iters):
    for i in range(n_buf):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if GRAPH:
        side = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for i in range(n_buf):
                    fn(i)
            reps = max(1, (iters + n_buf - 1) // n_buf)
            g.replay()
            e0.record()
            for _ in range(reps):
                g.replay()
            e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / (reps * n_buf) * 1e-3
    e0.record()
    for k in range(iters):
        fn(k % n_buf)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters * 1e-3


QUIET = False       # set by callers that only want the returned figures (bench.py prints one JSON line and nothing else)


def _say(text):
    if not QUIET:
        print(text, flush=True)


def bench_ln(h, M, H, kind, iters, out_gran="twq"):
    """kind 'f16': FP16 -> INT8 TWQ (entry flavour); 'i8': INT8 TWQ + INT8 FWQ -> INT8 TWQ (Eq. 19); out_gran 'fwq': the
    output is quantized with a calibrated per-feature scale instead (Eq. 4)."""
    n = max(2, min(32, int(400e6 // (M * H * 3)) + 1))
    g, b = torch.ones(H, device="cuda"), torch.zeros(H, device="cuda")
    sc = torch.empty(M, device="cuda")
    outs = [torch.empty(M, H, device="cuda", dtype=torch.int8) for _ in range(n)]
    if kind == "f16":
        xs = [torch.randn(M, H, device="cuda", dtype=torch.float16) for _ in range(n)]
        ins = [(hero.tensor(x), None) for x in xs]
    else:
        rs, cs = torch.rand(M, device="cuda") * 0.01 + 0.01, torch.rand(H, device="cuda") * 0.01 + 0.01
        xs = [torch.randint(-127, 128, (M, H), device="cuda", dtype=torch.int8) for _ in range(n)]
        ys = [torch.randint(-127, 128, (M, H), device="cuda", dtype=torch.int8) for _ in range(n)]
        ins = [(hero.tensor(x, "twq", rs), hero.tensor(y, "fwq", cs)) for x, y in zip(xs, ys)]
    if out_gran == "fwq":
        sc = torch.rand(H, device="cuda") * 0.01 + 0.02
    t = _time(lambda i: h.hero_layernorm_quant(ins[i][0], g, b, 1e-5, hero.tensor(outs[i], out_gran, sc), branch=ins[i][1]), n, iters)
    hbm, _, src = _peaks()
    gbs = M * H * 3 / t / 1e9
    _say("LN^quant %s%s M=%d H=%d: %.1f us, %.0f GB/s (algorithmic 3 B/element), %.2f of %s copy bandwidth"
         % (kind, "" if out_gran == "twq" else " -> " + out_gran, M, H, t * 1e6, gbs, gbs / hbm, src))
    return {"us": t * 1e6, "gbs": gbs}


def bench_gemm(h, M, K, N, act, fp, iters, f8=False):
    dt = torch.bfloat16 if fp else (torch.float8_e4m3fn if f8 else torch.int8)
    n = max(2, min(64, int(300e6 // (M * K + N * K + M * N)) + 1))
    if fp:
        As = [torch.randn(M, K, device="cuda", dtype=dt) for _ in range(n)]
        Ws = [torch.randn(N, K, device="cuda", dtype=dt) for _ in range(n)]
    elif f8:
        As = [(torch.randn(M, K, device="cuda") * 100).to(dt) for _ in range(n)]
        Ws = [(torch.randn(N, K, device="cuda") * 100).to(dt) for _ in range(n)]
    else:
        As = [torch.randint(-127, 128, (M, K), device="cuda", dtype=dt) for _ in range(n)]
        Ws = [torch.randint(-127, 128, (N, K), device="cuda", dtype=dt) for _ in range(n)]
    outs = [torch.empty(M, N, device="cuda", dtype=dt) for _ in range(n)]
    rs, cs = torch.rand(M, device="cuda") * 1e-3, torch.rand(N, device="cuda") * 1e-3
    bias = torch.randn(N, device="cuda")

    def run(i):
        a = hero.tensor(As[i]) if fp else hero.tensor(As[i], "twq", rs)
        h.hero_w8a8_linear(a, Ws[i], hero.tensor(outs[i]), w_scale=None if fp else cs, bias=bias, act=act)
    t = _time(run, n, iters)
    _, i8peak, src = _peaks()
    peak = i8peak / 2 if fp else i8peak
    tops = 2.0 * M * N * K / t / 1e12
    es = 2 if fp else 1
    gbs = (M * K * es + N * K * es + M * N * es + 4 * M + 8 * N) / t / 1e9
    hbm = _peaks()[0]
    _say("GeMM^quant %s M=%d K=%d N=%d act=%s: %.1f us, %.0f TOP/s, %.2f of 2 x %s BF16 peak%s; %.0f GB/s, %.2f of copy bandwidth"
         % ("bf16" if fp else ("e4m3" if f8 else "i8"), M, K, N, act, t * 1e6, tops, tops / peak, src, " / 2" if fp else "",
            gbs, gbs / hbm))
    return {"us": t * 1e6, "tops": tops, "gbs": gbs}


def bench_attn(h, B, S, nh, dh, mask, iters, p_mode="static", fp=False):
    H = nh * dh
    if fp:                                     # the FP16 core of a module left in FP mode (Table 1): FP16 in, FP16 out
        qkv = torch.randn(B * S, 3 * H, device="cuda", dtype=torch.float16)
        out = torch.empty(B * S, H, device="cuda", dtype=torch.float16)
        t = _time(lambda i: h.hero_int8_attention(qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:], B, S, nh, dh, hero.tensor(out),
                                                  mask=mask), 1, iters)
    else:
        qkv = (torch.randn(B * S, 3 * H, device="cuda") * 40).clamp(-127, 127).to(torch.int8)
        out = torch.empty(B * S, H, device="cuda", dtype=torch.int8)
        sc = torch.full((H,), 0.02, device="cuda")
        s = (1.5 ** 0.5) / 40
        t = _time(lambda i: h.hero_int8_attention(qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:], B, S, nh, dh,
                                                  hero.tensor(out, "fwq", sc), s_q=s, s_k=s, s_v=0.02, s_p=1 / 255, mask=mask,
                                                  p_mode=p_mode), 1, iters)
    scores = B * nh * S * S * (0.5 if mask == "causal" else 1.0)
    _say("%s attention B=%d S=%d nh=%d dh=%d %s P=%s: %.1f us, %.2f T scores/s, %.0f TOP/s tensor work"
         % ("FP16" if fp else "INT8", B, S, nh, dh, mask, "fp16" if fp else p_mode, t * 1e6, scores / t / 1e12,
            4 * scores * dh / t / 1e12))
    return {"us": t * 1e6, "tscores": scores / t / 1e12}


def bench_absmax(h, M, H, iters):
    """Per-feature and per-tensor absmax of an FP16 tensor: one read of 2 bytes per element."""
    n = max(2, min(16, int(400e6 // (M * H * 2)) + 1))
    xs = [torch.randn(M, H, device="cuda", dtype=torch.float16) for _ in range(n)]
    cf, ct = torch.zeros(H, device="cuda"), torch.zeros(1, device="cuda")
    t = _time(lambda i: h.hero_absmax_observe(hero.tensor(xs[i]), cf, ct), n, iters)
    hbm, _, src = _peaks()
    gbs = M * H * 2 / t / 1e9
    print("absmax observer f16 M=%d H=%d: %.1f us, %.0f GB/s (algorithmic 2 B/element), %.2f of %s copy bandwidth"
          % (M, H, t * 1e6, gbs, gbs / hbm, src), flush=True)


def bench_wquant(h, N, K, iters):
    """W~ = Diag(in) W Diag(1/out), Eq. 2: 4 bytes read (the second sweep hits L2) + 1 written per weight."""
    n = max(2, min(8, int(400e6 // (N * K * 5)) + 1))
    Ws = [torch.randn(N, K, device="cuda") * 0.02 for _ in range(n)]
    Wq = [torch.empty(N, K, device="cuda", dtype=torch.int8) for _ in range(n)]
    si, so = torch.rand(K, device="cuda") * 0.05 + 0.01, torch.rand(N, device="cuda") * 0.05 + 0.01
    ws, b, bo = torch.empty(N, device="cuda"), torch.randn(N, device="cuda"), torch.empty(N, device="cuda")
    t = _time(lambda i: h.hero_quantize_weight(Ws[i], Wq[i], ws, in_scale=si, out_scale=so, bias=b, bias_out=bo), n, iters)
    hbm, _, src = _peaks()
    gbs = N * K * 5 / t / 1e9
    print("weight fold + quantize N=%d K=%d: %.1f us, %.0f GB/s (algorithmic 5 B/weight), %.2f of %s copy bandwidth"
          % (N, K, t * 1e6, gbs, gbs / hbm, src), flush=True)


def bench_decode(h, B, S, nh, dh, iters, p_mode="static"):
    """One decode step of the INT8 attention core: every sequence holds S cache entries.  Algorithmic bytes: every key
    and value once (2 B S H); several caches are rotated so that the reads come from HBM.  The kernel does not fetch value
    rows whose probabilities quantize to zero, so the timed query is all zeros: a flat softmax, under which the row-max
    quantizer gives every key the code 255 and every value row is read (the worst case; the static quantizer of Eq. 16
    rounds 1 / S to zero for S > 510 and then reads the keys only)."""
    H = nh * dh
    n = max(2, min(32, int(400e6 // (2 * B * S * H)) + 1))
    q = torch.zeros(B, H, device="cuda", dtype=torch.int8)
    ks = [torch.randint(-127, 128, (B, S, H), device="cuda", dtype=torch.int8) for _ in range(n)]
    vs = [torch.randint(-127, 128, (B, S, H), device="cuda", dtype=torch.int8) for _ in range(n)]
    lens = torch.full((B,), S, device="cuda", dtype=torch.int32)
    out = torch.empty(B, H, device="cuda", dtype=torch.int8)
    osc = torch.full((H,), 0.01, device="cuda")
    s = 0.03
    t = _time(lambda i: h.hero_int8_decode_attention(q, ks[i], vs[i], lens, S, nh, dh, hero.tensor(out, "fwq", osc), s_q=s, s_k=s,
                                                     s_v=0.02, s_p=1.0 / 255, p_mode=p_mode), n, iters)
    hbm, _, src = _peaks()
    keys_only = p_mode == "static" and S > 510            # P = 1 / S rounds to zero: no value row is fetched
    gbs = (1.0 if keys_only else 2.0) * B * S * H / t / 1e9
    print("decode attention B=%d S=%d nh=%d dh=%d %s: %.1f us, %.0f GB/s (%s), %.2f of %s copy bandwidth"
          % (B, S, nh, dh, p_mode, t * 1e6, gbs, "keys once; all P_u8 = 0" if keys_only else "keys and values once", gbs / hbm, src),
          flush=True)


def bench_layer_decode(h, workload, B, S, iters, p_mode="rowmax"):
    """One decode step of a layer of the named configuration's width: B sequences with S cache entries each.  What bounds
    it is reading the layer's INT8 weights and the key / value caches once: bytes = 12 H^2 (F = 4H) + 2 B S H.  Several
    caches are rotated; the row-max quantizer is timed because it reads every value row (see bench_decode)."""
    from . import prep
    from .layer import Layer
    full = {"c3": W.C3, "c4": W.C4}[workload]
    shape = W.tiny_shape(B=B, S=128, H=full.H, nh=full.nh, F=full.F, arch=full.arch, mask="causal", fp_dtype=full.fp_dtype,
                         eps=full.eps)
    cfg = prep.LayerConfig(B=B, S=128, H=shape.H, nh=shape.nh, F=shape.F, arch=shape.arch, eps=shape.eps, mask="causal",
                           fp_dtype=shape.fp_dtype, mode=dict(prep.PRESETS["M3"]), p_mode=p_mode,
                           gran_out="fp" if shape.arch == "pre_ln" else "twq")
    p = W.layer_params(shape, 4)
    x_cal = W.activations(shape, 4, n_seq=1, tensor=7).astype("float64")
    if shape.arch == "post_ln":
        from .model import _ln_np
        x_cal = _ln_np(x_cal, p["ln0_g"].astype("float64"), p["ln0_b"].astype("float64"), cfg.eps)
    layer = Layer(h, prep.prepare_layer(cfg, p, prep.calibrate(cfg, p, x_cal, 1)))
    H = shape.H
    n = max(2, min(16, int(400e6 // (2 * B * S * H)) + 1))
    ks = [torch.randint(-127, 128, (B, S, H), device="cuda", dtype=torch.int8) for _ in range(n)]
    vs = [torch.randint(-127, 128, (B, S, H), device="cuda", dtype=torch.int8) for _ in range(n)]
    lens = torch.full((B,), S, device="cuda", dtype=torch.int32)
    if shape.arch == "pre_ln":
        x = torch.randn(B, H, device="cuda").to(hero.TORCH_FP[shape.fp_dtype])
        xin, out = hero.tensor(x), hero.tensor(torch.empty_like(x))
    else:
        xq = torch.randint(-127, 128, (B, H), device="cuda", dtype=torch.int8)
        xin = hero.tensor(xq, "twq", torch.full((B,), 0.02, device="cuda"))
        out = hero.tensor(torch.empty_like(xq), "twq", torch.empty(B, device="cuda"))
    t = _time(lambda i: layer.decode(ks[i], vs[i], lens, S, xin, out), n, iters)
    hbm, _, src = _peaks()
    byts = 4.0 * H * H + 2.0 * H * shape.F + 2.0 * B * S * H
    print("layer decode step %s B=%d S=%d %s: %.1f us, %.0f tokens/s, %.0f GB/s (weights + caches once), %.2f of %s copy bandwidth"
          % (workload, B, S, p_mode, t * 1e6, B / t, byts / t / 1e9, byts / t / 1e9 / hbm, src), flush=True)


def bench_layer(h, workload, payload, fp, iters):
    """One forward of a single layer of a benchmark configuration (INT8, e4m3 or all-FP modules), L2 flushed between
    forwards by a 256 MB write (its time is measured alone and subtracted)."""
    from . import prep
    from .model import Stack
    shape = {"c1": W.C1, "c3": W.C3, "c4": W.C4}[workload]
    mode = dict(prep.PRESETS["FP" if fp else "M3"])
    kw = dict(gran_in="fwq", gran_attn="sq") if workload == "c3" else {}
    cfg = prep.LayerConfig(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, arch=shape.arch, eps=shape.eps,
                           mask=shape.mask, fp_dtype=shape.fp_dtype, mode=mode, payload=payload, **kw)
    if fp:
        cfg.gran_out = "fp"
    st = Stack(h, shape, 3, [cfg], n_cal_seq=1)
    x = torch.randn(shape.M, shape.H, device="cuda").to(hero.TORCH_FP[shape.fp_dtype])
    st.set_input(x)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    t_flush = _time(lambda i: flush.fill_(i & 1), 1, iters)

    def step(i):
        flush.fill_(i & 1)
        st.forward()
    t = _time(step, 1, iters) - t_flush
    print("layer %s %s: %.1f us per forward, %.2f M tokens/s" % (workload, "fp" if fp else payload, t * 1e6, shape.M / t / 1e6), flush=True)
    # per-launch times of one forward (event pairs around every launch: the sum exceeds the un-instrumented time)
    h.profile_begin(64)
    st.forward()
    torch.cuda.synchronize()
    fam = {1: "ln", 2: "gemm", 3: "attention"}
    print("  launches: " + ", ".join("%s %.1f us" % (fam.get(k, "?"), ms * 1e3) for k, ms in h.profile_end()), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("kernel", choices=["ln", "gemm", "attn", "absmax", "wquant", "layer", "decode", "layer-decode"])
    ap.add_argument("--workload", default="c3", choices=["c1", "c3", "c4"])
    ap.add_argument("--M", type=int, default=65536)
    ap.add_argument("--H", type=int, default=1024)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--N", type=int, default=4096)
    ap.add_argument("--B", type=int, default=8)
    ap.add_argument("--S", type=int, default=384)
    ap.add_argument("--nh", type=int, default=16)
    ap.add_argument("--dh", type=int, default=64)
    ap.add_argument("--kind", default="i8", choices=["i8", "f16"])
    ap.add_argument("--act", default="none")
    ap.add_argument("--mask", default="none")
    ap.add_argument("--p-mode", default="static", choices=["static", "rowmax"])
    ap.add_argument("--fp", action="store_true")
    ap.add_argument("--f8", action="store_true", help="e4m3 operands and output (the FP8 variant)")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--out-gran", default="twq", choices=["twq", "fwq"], help="LN^quant output quantizer")
    ap.add_argument("--graph", action="store_true", help="time CUDA-graph replays of the launches")
    a = ap.parse_args()
    global GRAPH
    GRAPH = a.graph
    h = hero.Handle()
    if a.kernel == "ln":
        if a.sweep:
            for H in W.LN_SWEEP_H:
                for M in W.LN_SWEEP_M:
                    bench_ln(h, M, H, a.kind, a.iters)
        else:
            bench_ln(h, a.M, a.H, a.kind, a.iters, a.out_gran)
    elif a.kernel == "gemm":
        if a.sweep:
            for K, N in W.GEMM_SWEEP_KN:
                for M in W.GEMM_SWEEP_M:
                    bench_gemm(h, M, K, N, a.act, a.fp, a.iters, a.f8)
        else:
            bench_gemm(h, a.M, a.K, a.N, a.act, a.fp, a.iters, a.f8)
    elif a.kernel == "absmax":
        bench_absmax(h, a.M, a.H, a.iters)
    elif a.kernel == "wquant":
        bench_wquant(h, a.N, a.K, a.iters)
    elif a.kernel == "layer-decode":
        bench_layer_decode(h, a.workload, a.B, a.S, a.iters, a.p_mode)
    elif a.kernel == "decode":
        bench_decode(h, a.B, a.S, a.nh, a.dh, a.iters, a.p_mode)
    elif a.kernel == "layer":
        bench_layer(h, a.workload, "f8" if a.f8 else "i8", a.fp, a.iters)
    else:
        bench_attn(h, a.B, a.S, a.nh, a.dh, a.mask, a.iters, a.p_mode, a.fp)
    h.check()


if __name__ == "__main__":
    main()
