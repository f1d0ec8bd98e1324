#!/usr/bin/env python
"""Benchmark of the W8A8 layer forward (ZeroQuant-HERO hot path) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c1|c3|c4] [--impl reference]

A step is one pass of the whole hot path over one batch of synthetic input that is already resident in
HBM.  One JSON line is printed by rank 0.  `--impl reference` times the CPU oracle instead (a deliberately
plain fp64 program: context, not a target).
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "W8A8 layer tokens/sec"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------------------------
# workloads
# ------------------------------------------------------------------------------------------------
def workload_spec(name):
    """(shape, config id, [layer configs], description) for a benchmark workload."""
    from paper_2310_17723_b200 import prep, workloads as W
    m3 = dict(prep.PRESETS["M3"])

    def cfg(shape, **kw):
        return prep.LayerConfig(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, arch=shape.arch, eps=shape.eps,
                                mask=shape.mask, fp_dtype=shape.fp_dtype, mode=dict(m3), **kw)
    if name == "c1":
        s = W.C1
        return s, 1, [cfg(s)], "C1: BERT-base layer, B1 S128 H768, post-LN, M3, TWQ"
    if name == "c3":
        s = W.C3
        return s, 3, [cfg(s, gran_in="fwq", gran_attn="sq", gran_mid="twq", gran_out="twq")], \
            "C3: BERT-large layer, B32 S384 H1024 F4096, post-LN, M3, FWQ LN->QKV (folded), SQ X_attn, TWQ elsewhere"
    if name == "c4":
        s = W.C4
        return s, 4, [cfg(s)], "C4: GPT prefill layer, B8 S2048 H4096 nh32 F16384, pre-LN, causal, W8A8 everywhere"
    if name == "c5":
        s = W.C5
        g = W.rng(5, 99)
        n_layers = 24
        fp_layers = set(int(i) for i in g.choice(n_layers, size=2, replace=False))
        kinds = [str(k) for k in g.choice(["twq", "fwq", "sq_attn"], size=n_layers)]
        cfgs = []
        for li in range(n_layers):
            if li in fp_layers:
                c = prep.LayerConfig(B=s.B, S=s.S, H=s.H, nh=s.nh, F=s.F, arch=s.arch, eps=s.eps, mask=s.mask,
                                     fp_dtype=s.fp_dtype, mode=dict(prep.PRESETS["FP"]))
            elif kinds[li] == "fwq":
                c = cfg(s, gran_in="fwq")
            elif kinds[li] == "sq_attn":
                c = cfg(s, gran_attn="sq")
            else:
                c = cfg(s)
            cfgs.append(c)
        for li, c in enumerate(cfgs):                      # a layer emits what the next layer's QKV consumes
            if li + 1 < n_layers:
                nxt = cfgs[li + 1]
                c.gran_out = "fp" if nxt.mode["qkv"] == "fp" else nxt.gran_in
            else:
                c.gran_out = "fp"
        return s, 5, cfgs, "C5: 24 x BERT-large layer, B64 S512 H1024 F4096, post-LN, seeded TWQ/FWQ/SQ mix, layers %s in FP16, FP16 output" % sorted(fp_layers)
    raise SystemExit("unknown workload %r" % name)


def fp_variant(cfgs):
    """The same layers with every module left in FP16/BF16 (the library's own FP path, for the W8A8 speed-up)."""
    from paper_2310_17723_b200 import prep
    import copy
    out = []
    for c in cfgs:
        c2 = copy.deepcopy(c)
        c2.mode = dict(prep.PRESETS["FP"])
        c2.gran_out = "fp"
        out.append(c2)
    return out


def attn_ln_fp_variant(cfgs):
    """The same layers with attention and the LN outputs in FP16/BF16: the QKV and FC1 GEMMs then consume FP tensors and run
    in FP mode, the attention-output linear and FC2 stay INT8 (their inputs are quantized in the producers' epilogues)."""
    import copy
    out = []
    for c in cfgs:
        c2 = copy.deepcopy(c)
        c2.mode = dict(qkv="fp", attn="fp", attn_out="int8", fc1="fp", fc2="int8")
        out.append(c2)
    return out


def kernel_table(shape, cfg):
    """Per launch of one layer, in launch order: (name, family, algorithmic ops, algorithmic bytes)."""
    M, H, F, S, nh, dh = shape.M, shape.H, shape.F, shape.S, shape.nh, shape.dh
    causal = shape.mask == "causal"

    def gemm(name, K, N, module="qkv"):
        fam = "gemm" if cfg.mode[module] == "int8" else "gemm_fp"
        return (name, fam, 2.0 * M * N * K, float(M * K + N * K + M * N + 4 * M + 8 * N))
    attn_ops = 4.0 * shape.B * nh * S * S * dh * (0.5 if causal else 1.0)
    attn = ("attention", "attn", attn_ops, float(4 * M * H))
    rows = []
    if shape.arch == "pre_ln":
        rows.append(("ln1 (fp->i8 twq)", "ln", 0.0, float(M * H * 3 + 4 * M)))
    rows += [gemm("qkv gemm", H, 3 * H, "qkv"), attn, gemm("attn-out gemm", H, H, "attn_out")]
    if shape.arch == "pre_ln":
        rows.append(("add+ln2 (fp+i8->fp,i8)", "ln", 0.0, float(M * H * 6 + 4 * M)))
    else:
        rows.append(("ln1 (i8+i8->i8 twq)", "ln", 0.0, float(M * H * 3 + 8 * M)))
    rows += [gemm("fc1 gemm + gelu^quant", H, F, "fc1"), gemm("fc2 gemm", F, H, "fc2")]
    if shape.arch == "pre_ln":
        rows.append(("closing add (fp+i8->fp)", "ln", 0.0, float(M * H * 5)))
    else:
        rows.append(("ln2 (i8+i8->i8 twq)", "ln", 0.0, float(M * H * 3 + 8 * M)))
    return rows



# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the default workload's kernels, from one
# ncu pass over this script (see profiles/dram_traffic_c3_layer.md).  ncu flushes L2 before every captured launch, so
# reads equal the algorithmic input bytes and the outputs (all smaller than L2) are still cached when the kernel ends.
NCU_TRAFFIC_C3 = {"qkv gemm": 15.8e6, "attention": 38.1e6, "attn-out gemm": 13.7e6, "ln1 (i8+i8->i8 twq)": 25.2e6,
                  "fc1 gemm + gelu^quant": 18.6e6, "fc2 gemm": 54.8e6, "ln2 (i8+i8->i8 twq)": 25.3e6}
KERNEL_FUNCTION = {"qkv gemm": "gemm_pair_kernel<int8, no activation>", "attn-out gemm": "gemm_pair_kernel<int8, no activation>",
                   "fc2 gemm": "gemm_pair_kernel<int8, no activation>"}


def dominant_kernel(kern, workload, peaks, peak_kind, clocks):
    """The roofline object: rows of `kern` grouped by kernel function (the three GEMMs without activation are one
    function launched three times per step), the group with the largest time share, aggregated over its launches."""
    groups = {}
    for r in kern:
        key = KERNEL_FUNCTION.get(r["kernel"], r["kernel"])
        groups.setdefault(key, []).append(r)
    key, rows = max(groups.items(), key=lambda kv: sum(r["ms"] for r in kv[1]))
    ms = sum(r["ms"] for r in rows)
    launches = sum(r["launches_per_step"] for r in rows)
    achieved = sum(r["achieved"] * r["ms"] for r in rows) / ms            # total work / total time
    peak = rows[0]["peak"]
    traffic = None
    if workload == "c3" and all(r["kernel"] in NCU_TRAFFIC_C3 for r in rows):
        traffic = sum(NCU_TRAFFIC_C3[r["kernel"]] for r in rows) / launches
    src = {"tensor": "2 x bf16_tflops_sustained (INT8 runs at twice the BF16 rate; sustained: the kernel runs inside a long step)",
           "hbm": "hbm_gbs", "alu": "148 SMs x 16 ex2 per clock x sampled SM clock"}[rows[0]["bound"]]
    return {"bound": rows[0]["bound"], "achieved": achieved, "peak": peak, "unit": rows[0]["unit"], "frac": achieved / peak,
            "traffic": traffic, "kernel": key, "members": [r["kernel"] for r in rows], "launches_per_step": launches,
            "ms_per_step": round(ms, 5), "share": round(sum(r["share"] for r in rows), 4),
            "peak_source": "%s: %s" % (peak_kind if rows[0]["bound"] != "alu" else "derived", src)}

# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    Q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
        "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"

    def __init__(self, index):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# CPU oracle arm (also the cpu_baseline leg)
# ------------------------------------------------------------------------------------------------
def oracle_run(name, budget_s=12.0, repeats=1):
    """Times the oracle, as it stands, on whole sequences of the workload (all of its layers).
    Returns (tokens/s, cores, sample, seconds)."""
    import numpy as np
    from oracle import layer as OL, ops as O
    from paper_2310_17723_b200 import workloads as W
    shape, cid, cfgs, desc = workload_spec(name)
    x_cal = W.activations(shape, cid, n_seq=1, tensor=7).astype(np.float64)
    layers = []
    cur = None
    for li, cfg in enumerate(cfgs):                       # offline preparation of every layer (not timed)
        spec = OL.LayerSpec(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, arch=shape.arch, act=cfg.act,
                            eps=cfg.eps, mask=cfg.mask, fp_dtype=cfg.fp_dtype, mode=dict(cfg.mode), gran_in=cfg.gran_in,
                            gran_mid=cfg.gran_mid, gran_attn=cfg.gran_attn, gran_out=cfg.gran_out)
        p = W.layer_params(shape, cid * 100 + li)
        if li == 0:
            ln0 = (p["ln0_g"], p["ln0_b"])
            cur = O.layernorm(x_cal, p["ln0_g"], p["ln0_b"], spec.eps) if spec.arch == "post_ln" else x_cal
        C = OL.calibrate(spec, p, cur, 1)
        if len(cfgs) > 1:
            cur = OL.layer_fp64(spec, p, cur, B=1)["x_out"]
        layers.append((spec, OL.prepare_layer(spec, p, C)))

    def run(n_seq):
        x = W.activations(shape, cid, n_seq=n_seq)
        spec0, L0 = layers[0]
        if spec0.arch == "post_ln":
            cur_t = OL.entry_ln(O.fp_tensor(x, spec0.fp_dtype), ln0[0], ln0[1], spec0.eps, L0["ln_in_out"])
        else:
            cur_t = O.fp_tensor(x, spec0.fp_dtype)
        t0 = time.perf_counter()
        for spec, Lp in layers:
            cur_t = OL.layer_forward(Lp, cur_t, B=n_seq)["x_out"]
        return time.perf_counter() - t0

    t1 = run(1)
    n = int(max(1, min(shape.B, budget_s / max(t1, 1e-3))))
    best = min(run(n) for _ in range(repeats)) if n > 1 else t1
    cores = os.cpu_count() or 1
    try:
        from threadpoolctl import threadpool_info
        cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        pass
    sample = "%d of %d sequences (%d tokens) of %s through %d layer(s), one pass" % (n, shape.B, n * shape.S, shape.name, len(layers))
    return n * shape.S / best, cores, sample, best


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    shape, cid, cfgs, desc = workload_spec(args.workload)
    vals, ts = [], []
    for i in range(args.warmup + args.steps):
        v, cores, sample, t = oracle_run(args.workload, budget_s=max(2.0, 60.0 / max(1, args.warmup + args.steps)))
        if i >= args.warmup:
            vals.append(v)
            ts.append(t)
    value = sum(vals) / len(vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * sum(ts) / len(ts), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": desc, "l2": "n/a (CPU)"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# CUDA arm
# ------------------------------------------------------------------------------------------------
def run_ours(args):
    import numpy as np
    import torch
    from paper_2310_17723_b200 import build as B
    from paper_2310_17723_b200 import replicas
    rank, local, world = replicas.rank_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0 or world == 1:
        B.build()
    if dist:
        dist.barrier()
    from paper_2310_17723_b200 import hero, workloads as W
    from paper_2310_17723_b200.model import Stack

    shape, cid, cfgs, desc = workload_spec(args.workload)
    h = hero.Handle()
    stack = Stack(h, shape, cid, cfgs, n_cal_seq=1 if shape.M * shape.H > 2 ** 25 else 2)
    # every rank works on its own batch (replicas: the path shards by sequence, no exchange step)
    x_host = torch.from_numpy(W.activations(shape, cid, tensor=replicas.batch_tensor_index(rank))).to(stack.fp_torch)
    x_dev = x_host.cuda()
    stack.set_input(x_dev)
    h.check()
    flush = torch.empty(512 * 1024 * 1024, dtype=torch.int8, device="cuda")     # > 126 MB L2
    stream = torch.cuda.current_stream()

    def step():
        stack.forward()

    sampler = ClockSampler(local) if rank == 0 else None
    for _ in range(max(args.warmup, 3)):
        flush.zero_()
        step()
    torch.cuda.synchronize()
    n0 = h.launches
    step()
    launches_per_step = h.launches - n0
    torch.cuda.synchronize()
    eager_step = step
    replayed = [0]
    if args.graph:
        # the same launches through the C ABI, captured once; a replay issues them without host work in between
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                stack.forward()
        torch.cuda.synchronize()

        def step():
            graph.replay()
            replayed[0] += launches_per_step           # the handle counts launches as they are issued, i.e. at capture
        for _ in range(3):
            step()
        torch.cuda.synchronize()

    # ---- timed region: K steps, each bracketed by events on the launching stream, L2 flushed in between
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    wall0 = time.perf_counter()
    n0 = h.launches
    replayed[0] = 0
    for k in range(args.steps):
        flush.zero_()
        ev[k][0].record(stream)
        step()
        ev[k][1].record(stream)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    wall = time.perf_counter() - wall0
    gpu_launches = h.launches - n0 + replayed[0]
    h.check()
    total_ms = replicas.max_over_ranks(sum(a.elapsed_time(b) for a, b in ev), dist, "cuda")
    ms_per_step = total_ms / args.steps
    value = replicas.job_throughput(shape.M, args.steps, world, total_ms * 1e-3)

    # ---- per-kernel device times (a second, instrumented pass: event pairs around every launch)
    kern = []
    roof = None
    peaks, peak_kind = load_peaks()
    if rank == 0:
        h.profile_begin(launches_per_step * args.steps)
        for k in range(args.steps):
            flush.zero_()
            eager_step()
        recs = h.profile_end()
    clocks = sampler.stop() if sampler else None
    if rank == 0:
        table = []
        for cfg in cfgs:
            table += kernel_table(shape, cfg)
        assert len(table) == launches_per_step, (len(table), launches_per_step)
        int8_peak = 2.0 * peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
        merged = {}
        for i, (name, fam, ops, nbytes) in enumerate(table):
            ms = [recs[j][1] for j in range(i, len(recs), launches_per_step)]
            avg = sum(ms) / len(ms)
            key = (name, fam)
            if key in merged:                                  # same kernel in another layer of the stack
                merged[key] = (merged[key][0] + avg, merged[key][1] + ops, merged[key][2] + nbytes, merged[key][3] + 1)
            else:
                merged[key] = (avg, ops, nbytes, 1)
        for (name, fam), (avg, ops, nbytes, cnt) in merged.items():
            row = {"kernel": name if fam != "gemm_fp" else name + " (fp16)", "ms": round(avg, 5), "share": None, "launches_per_step": cnt}
            if fam == "gemm":
                row.update(bound="tensor", achieved=ops / (avg * 1e-3) / 1e12, peak=int8_peak, unit="TFLOP/s")
            elif fam == "gemm_fp":
                row.update(bound="tensor", achieved=ops / (avg * 1e-3) / 1e12, peak=int8_peak / 2, unit="TFLOP/s")
            elif fam == "ln":
                row.update(bound="hbm", achieved=nbytes / (avg * 1e-3) / 1e9, peak=peaks["hbm_gbs"], unit="GB/s")
            else:
                # bound by the special-function unit: one exponential per score and sweep that needs it
                # (ops = 4 dh per score, so scores = ops / (4 dh)); peak = 16 ex2 per clock and SM at the sampled clock
                scores = ops / (4.0 * shape.dh)
                mhz = (clocks or {}).get("sm_mhz") or peaks.get("sm_max_mhz", 1965.0)
                row.update(bound="alu", achieved=scores / (avg * 1e-3) / 1e12, peak=148 * 16 * mhz * 1e6 / 1e12,
                           unit="Texp/s", tensor_tops=ops / (avg * 1e-3) / 1e12)
            row["frac"] = row["achieved"] / row["peak"]
            kern.append(row)
        tot = sum(r["ms"] for r in kern)
        for r in kern:
            r["share"] = round(r["ms"] / tot, 4)
        roof = dominant_kernel(kern, args.workload, peaks, peak_kind, clocks)

    # ---- end to end through the C ABI with HOST buffers (pinned), copies inside the timed region
    e2e = None
    if len(cfgs) == 1 and shape.arch == "post_ln":
        t_in, s_in, d_in = stack.bufs[0]
        t_out, s_out, d_out = stack.bufs[1]
        hin = t_in.cpu().pin_memory()
        hout = torch.empty_like(t_out, device="cpu").pin_memory()
        gin, gout = cfgs[0].gran_in, cfgs[0].gran_out
        hsin = s_in.cpu().pin_memory() if s_in is not None else None
        hsout = torch.empty_like(s_out, device="cpu").pin_memory() if s_out is not None else None
        in_host = hero.host_tensor(hin, gin, hsin)
        out_host = hero.host_tensor(hout, gout, hsout)
        layer = stack.layers[0]

        # three steps in flight, each on its own stream with its own device staging tensors, workspace and pinned
        # output buffer: one step's copies overlap another step's kernels.  A slot is synchronised (its result is
        # then in host memory) before it is reused, so every step's input is copied in and its output read back.
        DEPTH = 3
        slots = []
        for _ in range(DEPTH):
            ti = torch.empty_like(t_in)
            si = torch.empty_like(s_in) if (s_in is not None and gin == "twq") else s_in
            to = torch.empty_like(t_out)
            so = torch.empty_like(s_out) if (s_out is not None and gout == "twq") else s_out
            ho = torch.empty_like(t_out, device="cpu").pin_memory()
            hso = torch.empty_like(s_out, device="cpu").pin_memory() if s_out is not None else None
            slots.append({"in": hero.tensor(ti, gin, si), "out": hero.tensor(to, gout, so), "host": hero.host_tensor(ho, gout, hso),
                          "ws": torch.empty_like(layer.workspace), "stream": torch.cuda.Stream(), "busy": False})
        e2e_k = [0]

        def e2e_step():
            sl = slots[e2e_k[0] % DEPTH]
            e2e_k[0] += 1
            if sl["busy"]:
                sl["stream"].synchronize()
            h.hero_layer_forward_host_async(layer.desc, in_host, sl["host"], sl["in"], sl["out"], sl["ws"], stream=sl["stream"])
            sl["busy"] = True
        h2d = hin.numel() + (hsin.numel() * 4 if gin == "twq" else 0)
        d2h = hout.numel() * hout.element_size() + (hsout.numel() * 4 if gout == "twq" else 0)
    else:
        t_in = stack.bufs[0][0]
        t_out = stack.bufs[-1][0]
        hin = x_host.pin_memory()
        hout = torch.empty_like(t_out, device="cpu").pin_memory()

        def e2e_step():
            t_in.copy_(hin, non_blocking=True)
            stack.forward()
            hout.copy_(t_out, non_blocking=True)
            torch.cuda.synchronize()
        h2d = hin.numel() * hin.element_size()
        d2h = hout.numel() * hout.element_size()
    for _ in range(3):
        e2e_step()
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        e2e_step()
    torch.cuda.synchronize()
    e2e_s = replicas.max_over_ranks(time.perf_counter() - t0, dist, "cuda")
    e2e = {"value": replicas.job_throughput(shape.M, args.steps, world, e2e_s), "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
           "steps_in_flight": 3 if (len(cfgs) == 1 and shape.arch == "post_ln") else 1}
    h.check()

    fp_path = None
    mixed_path = None
    if rank == 0 and world == 1 and not args.no_fp_path:
        # the same layer(s) in other module modes, through the same library and the same timing loop
        del stack
        torch.cuda.empty_cache()

        def time_variant(vcfgs):
            vstack = Stack(h, shape, cid, vcfgs, n_cal_seq=1)
            vstack.set_input(x_dev)
            for _ in range(3):
                flush.zero_()
                vstack.forward()
            torch.cuda.synchronize()
            fev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
            for k in range(args.steps):
                flush.zero_()
                fev[k][0].record(stream)
                vstack.forward()
                fev[k][1].record(stream)
            torch.cuda.synchronize()
            h.check()
            del vstack
            torch.cuda.empty_cache()
            return sum(a.elapsed_time(b) for a, b in fev) / args.steps

        fms = time_variant(fp_variant(cfgs))                 # every module in FP16 / BF16
        fp_path = {"value": shape.M / (fms * 1e-3), "unit": UNIT, "ms_per_step": fms, "dtype": shape.fp_dtype,
                   "w8a8_speedup": ms_per_step and fms / ms_per_step}
        if args.workload == "c4":
            # the config's comparison: attention and the LN outputs switched to BF16 (so QKV and FC1 run BF16 too),
            # attention-output linear and FC2 stay INT8
            mms = time_variant(attn_ln_fp_variant(cfgs))
            mixed_path = {"modes": "qkv, attention, fc1 in BF16; attention-output linear, fc2 INT8", "value": shape.M / (mms * 1e-3),
                          "unit": UNIT, "ms_per_step": mms, "w8a8_speedup": ms_per_step and mms / ms_per_step}
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        v, cores, sample, _t = oracle_run(args.workload)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
            "data": "synthetic",
            "config": {"workload": desc, "tokens_per_step_per_gpu": shape.M, "l2": "flushed between timed steps (512 MiB write)",
                       "launch": "CUDA graph replay of the step's launches" if args.graph else "one C-ABI call per layer, 7-8 kernel launches each",
                       "timing": "CUDA events per step on the launching stream, max over ranks",
                       "parallelism": "replicas x%d (sequence-sharded, no collective)" % world},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(gpu_launches), "roofline": roof, "kernels": kern,
            "kernels_note": "per-launch times come from a second pass with an event pair around every launch, which serialises the "
                            "launches (no programmatic overlap): their sum exceeds ms_per_step, so the fractions are lower bounds",
            "cpu_baseline": cpu, "fp16_path": fp_path, "wall_s_timed_region": wall}
    if mixed_path:
        line["attention_and_ln_bf16_path"] = mixed_path
    print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=["c1", "c3", "c4", "c5"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-fp-path", action="store_true")
    ap.add_argument("--graph", action="store_true", help="replay the step's launches from a CUDA graph (latency-bound workloads)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
