#!/usr/bin/env python
"""Benchmark of the W8A8 layer forward (ZeroQuant-HERO hot path) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5|c4|c3|c1] [--impl reference]

A step is one pass of the whole hot path (the entry LN^quant and every layer of the workload) over one batch of
synthetic input that is already resident in HBM.  The default workload is the largest single-GPU configuration, the
24-layer BERT-large-shaped stack.  One JSON line is printed by rank 0.  With --gpus N > 1 and no torchrun environment
the script starts its own N ranks (replicas: the path shards by sequence, nothing is exchanged).  `--impl reference`
times the CPU oracle instead (a deliberately plain fp64 program: context, not a target).
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


def kernel_table(shape, cfg, first=False):
    """Per launch of one layer, in launch order: (name, family, algorithmic ops, algorithmic bytes); `first`: the
    layer is preceded by the entry LN^quant of a post-LN workload."""
    M, H, F, S, nh, dh = shape.M, shape.H, shape.F, shape.S, shape.nh, shape.dh
    causal = shape.mask == "causal"
    i8 = lambda module: cfg.mode[module] == "int8"
    es = lambda is8: 1 if is8 else 2                          # bytes per element at a border

    def gemm(name, K, N, module, out8):
        fam = "gemm" if i8(module) else "gemm_fp"
        e = es(i8(module))
        return (name, fam, 2.0 * M * N * K, float(M * K * e + N * K * e + M * N * es(out8) + 4 * M + 8 * N))

    def ln(name, res8, br8, out8, fp_out=False):
        per = es(res8) + (es(br8) if br8 is not None else 0) + (es(out8) if out8 is not None else 0) + (2 if fp_out else 0)
        return ("%s (%s%s->%s%s)" % (name, "i8" if res8 else "fp", "" if br8 is None else ("+i8" if br8 else "+fp"),
                                      "" if out8 is None else ("i8" if out8 else "fp"), ",fp" if fp_out else ""),
                "ln", 0.0, float(M * H * per + 8 * M))
    attn_ops = 4.0 * shape.B * nh * S * S * dh * (0.5 if causal else 1.0)
    attn = ("attention" if i8("attn") else "attention (fp16)", "attn" if i8("attn") else "attn_fp", attn_ops,
            float(M * H * (3 * es(i8("attn")) + es(i8("attn_out")))))
    pre = shape.arch == "pre_ln"
    rows = []
    if first and not pre:
        rows.append(ln("entry ln", False, None, i8("qkv")))
    if pre:
        rows.append(ln("ln1", False, None, i8("qkv")))
    rows += [gemm("qkv gemm", H, 3 * H, "qkv", i8("attn")), attn, gemm("attn-out gemm", H, H, "attn_out", i8("attn_out"))]
    if pre:
        rows.append(ln("add+ln2", False, i8("attn_out"), i8("fc1"), fp_out=True))
    else:
        rows.append(ln("ln1", i8("qkv"), i8("attn_out"), i8("fc1")))
    rows += [gemm("fc1 gemm + gelu^quant", H, F, "fc1", i8("fc2")), gemm("fc2 gemm", F, H, "fc2", i8("fc2"))]
    if pre:
        rows.append(ln("closing add", False, i8("fc2"), None, fp_out=True))
    else:
        rows.append(ln("ln2", i8("fc1"), i8("fc2"), cfg.gran_out != "fp"))
    return rows


# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the kernel function that dominates a
# workload's step, each from one small ncu capture (one kernel, a few launches) recorded under profiles/; keyed by
# (workload, kernel function).  These are constants of a recorded capture, not values this run measures.
NCU_TRAFFIC = {
    ("c5", "gemm_pair_kernel<int8, no activation>"): {"bytes_per_launch": 90.2e6, "source": "profiles/launch_list_c5_stack.md: ncu launch "
                          "list of this workload at full size (one pass: time + dram__bytes_read.sum + dram__bytes_write.sum), "
                          "average over the 274 captured launches of the three members (69.9 MB read + 20.3 MB written; "
                          "algorithmic average 69.9 MB read + 55.9 MB written: most of an output is still in L2 when its kernel ends)"},
    ("c5", "attention"): {"bytes_per_launch": 144.7e6, "source": "profiles/launch_list_c5_stack.md: same capture, 92 launches of "
                          "attn_int8_pipe_kernel (128.0 MB read + 16.7 MB written; algorithmic 100.7 MB read + 33.6 MB written: "
                          "K and V of a head are read again by each of its four query tiles, not always from L2)"},
    ("c3", "gemm_pair_kernel<int8, no activation>"): {"bytes_per_launch": 28.1e6, "source": "profiles/dram_traffic_c3_layer.md: ncu capture "
                          "of the three launches (QKV 15.8 MB, attention output 13.7 MB, FC2 54.8 MB), recorded with an earlier build of "
                          "this kernel (same operand traffic)"},
}
KERNEL_FUNCTION = {"qkv gemm": "gemm_pair_kernel<int8, no activation>", "attn-out gemm": "gemm_pair_kernel<int8, no activation>",
                   "fc2 gemm": "gemm_pair_kernel<int8, no activation>"}
INT8_NOMINAL_TOPS = 4500.0          # dense INT8 rate of the part (datasheet figure without sparsity), for context


def peak_regime(clocks, peaks):
    """Which measured BF16 figure the timed region compares with: 'sustained' when the sampled clocks show the power
    cap biting (reason active, or the median SM clock well below the maximum), else 'burst'."""
    if not clocks or not clocks.get("sm_mhz"):
        return "burst", "no clock samples"
    mx = clocks.get("sm_max_mhz") or peaks.get("sm_max_mhz", 1965.0)
    capped = "sw_power_cap" in (clocks.get("reasons") or [])
    # the clock decides: a cap that shows up in some samples while the median clock stays at the maximum has not slowed
    # the timed region down, and comparing with the sustained figure would flatter the kernel
    if clocks["sm_mhz"] < 0.93 * mx:
        return "sustained", "median SM clock %.0f MHz below 0.93 x %.0f%s" % (clocks["sm_mhz"], mx,
                                                                             ", sw_power_cap active" if capped else "")
    return "burst", "median SM clock %.0f of %.0f MHz%s" % (clocks["sm_mhz"], mx,
                                                          " (sw_power_cap seen in some samples)" if capped else "")


def dominant_kernel(kern, workload, peaks, peak_kind, clocks):
    """The roofline object: rows of `kern` grouped by kernel function (the three GEMMs without activation are one
    function launched three times per layer), the group with the largest time share, aggregated over its launches."""
    groups = {}
    for r in kern:
        key = KERNEL_FUNCTION.get(r["kernel"], r["kernel"])
        groups.setdefault(key, []).append(r)
    key, rows = max(groups.items(), key=lambda kv: sum(r["ms"] for r in kv[1]))
    ms = sum(r["ms"] for r in rows)
    launches = sum(r["launches_per_step"] for r in rows)
    achieved = sum(r["achieved"] * r["ms"] for r in rows) / ms            # total work / total time
    bound = rows[0]["bound"]
    out = {"bound": bound, "achieved": achieved, "peak": rows[0]["peak"], "unit": rows[0]["unit"], "frac": achieved / rows[0]["peak"],
           "traffic": None, "kernel": key, "members": sorted(set(r["kernel"] for r in rows)), "launches_per_step": launches,
           "ms_per_step": round(ms, 5), "share": round(sum(r["share"] for r in rows), 4)}
    if bound == "tensor":
        regime, why = peak_regime(clocks, peaks)
        burst, sust = 2.0 * peaks["bf16_tflops"], 2.0 * peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
        out.update(regime=regime, regime_why=why, frac_of_burst=achieved / burst, frac_of_sustained=achieved / sust,
                   frac_of_nominal=achieved / INT8_NOMINAL_TOPS, peak_burst=burst, peak_sustained=sust, peak_nominal=INT8_NOMINAL_TOPS,
                   peak_source="%s: 2 x bf16_tflops%s (INT8 runs at twice the BF16 rate of the same tensor cores; no INT8 figure is "
                               "measured by the driver)" % (peak_kind, "_sustained" if regime == "sustained" else ""))
    elif bound == "hbm":
        out["peak_source"] = "%s: hbm_gbs" % peak_kind
    else:
        out["peak_source"] = "derived: 148 SMs x 16 ex2 per clock x sampled SM clock"
    t = NCU_TRAFFIC.get((workload, key))
    if t:
        out["traffic"] = t["bytes_per_launch"]
        out["traffic_source"] = t["source"]
    return out


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi queries (read-only) every 100 ms in a child process; `stop` summarises the samples that fell inside
    the window the caller marks with `begin()` .. `stop()`, i.e. while the GPU was working."""
    Q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
        "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"

    def __init__(self, index):
        self.rows, self.proc, self.t_begin = [], None, None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
            t0 = time.time()
            while not self.rows and time.time() - t0 < 5.0:      # the first sample takes a moment: wait for it
                time.sleep(0.02)
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def begin(self):
        self.t_begin = time.time()

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        t_end = time.time()
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], None, set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for t, r in self.rows:
            if self.t_begin is not None and not (self.t_begin <= t <= t_end + 0.05):
                continue
            f = [x.strip() for x in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
                power.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons), "samples": len(sm),
                "power_w_max": max(power) if power else None, "window": "warm-up through the per-kernel pass (GPU busy throughout)"}


# ------------------------------------------------------------------------------------------------
# CPU oracle arm (also the cpu_baseline leg)
# ------------------------------------------------------------------------------------------------
class OracleArm:
    """The oracle, as it stands, on whole sequences of a workload (entry LN^quant and all of its layers).  The offline
    preparation of the layers (calibration, folding, weight quantization) happens once, in the constructor, and is not
    timed."""

    def __init__(self, name):
        import numpy as np
        from oracle import layer as OL, ops as O
        from paper_2310_17723_b200 import workloads as W
        self.OL, self.O, self.W = OL, O, W
        self.shape, self.cid, cfgs, self.desc = workload_spec(name)
        shape, cid = self.shape, self.cid
        x_cal = W.activations(shape, cid, n_seq=1, tensor=7).astype(np.float64)
        self.layers = []
        cur = None
        for li, cfg in enumerate(cfgs):
            spec = OL.LayerSpec(B=shape.B, S=shape.S, H=shape.H, nh=shape.nh, F=shape.F, arch=shape.arch, act=cfg.act,
                                eps=cfg.eps, mask=cfg.mask, fp_dtype=cfg.fp_dtype, mode=dict(cfg.mode), gran_in=cfg.gran_in,
                                gran_mid=cfg.gran_mid, gran_attn=cfg.gran_attn, gran_out=cfg.gran_out)
            p = W.layer_params(shape, cid * 100 + li)
            if li == 0:
                self.ln0 = (p["ln0_g"], p["ln0_b"])
                cur = O.layernorm(x_cal, p["ln0_g"], p["ln0_b"], spec.eps) if spec.arch == "post_ln" else x_cal
            C = OL.calibrate(spec, p, cur, 1)
            if len(cfgs) > 1:
                cur = OL.layer_fp64(spec, p, cur, B=1)["x_out"]
            self.layers.append((spec, OL.prepare_layer(spec, p, C)))
        self.t1 = None                                        # seconds for one sequence (measured by the first run)

    def run(self, n_seq):
        """Seconds for one pass of n_seq sequences: a step = the entry LN^quant and every layer, as on the GPU."""
        OL, O, W = self.OL, self.O, self.W
        x = W.activations(self.shape, self.cid, n_seq=n_seq)
        spec0, L0 = self.layers[0]
        t0 = time.perf_counter()
        if spec0.arch == "post_ln":
            cur_t = OL.entry_ln(O.fp_tensor(x, spec0.fp_dtype), self.ln0[0], self.ln0[1], spec0.eps, L0["ln_in_out"])
        else:
            cur_t = O.fp_tensor(x, spec0.fp_dtype)
        for spec, Lp in self.layers:
            cur_t = OL.layer_forward(Lp, cur_t, B=n_seq)["x_out"]
        return time.perf_counter() - t0

    def step(self, budget_s):
        """One bounded sample: as many whole sequences as fit `budget_s` (at least one).
        Returns (tokens/s, cores, sample, seconds)."""
        if self.t1 is None:
            self.t1 = self.run(1)
            n, best = 1, self.t1
            if budget_s >= 2.0 * self.t1:
                n = int(max(1, min(self.shape.B, budget_s / max(self.t1, 1e-3))))
                best = self.run(n) if n > 1 else self.t1
        else:
            n = int(max(1, min(self.shape.B, budget_s / max(self.t1, 1e-3))))
            best = self.run(n)
        cores = os.cpu_count() or 1
        try:
            from threadpoolctl import threadpool_info
            cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
        except Exception:
            pass
        sample = "%d of %d sequences (%d tokens) of %s through %d layer(s), one pass" % (n, self.shape.B, n * self.shape.S,
                                                                                        self.shape.name, len(self.layers))
        return n * self.shape.S / best, cores, sample, best


def oracle_run(name, budget_s=12.0):
    """One bounded sample of the oracle on a workload: (tokens/s, cores, sample, seconds)."""
    return OracleArm(name).step(budget_s)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    arm = OracleArm(args.workload)                            # offline preparation, once
    desc = arm.desc
    vals, ts = [], []
    # every step is a bounded sample; the whole run (warm-up included) aims at about two minutes of oracle time, with one
    # whole sequence per step as the floor
    per_step = max(2.0, 120.0 / max(1, args.warmup + args.steps))
    for i in range(args.warmup + args.steps):
        v, cores, sample, t = arm.step(per_step)
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
def sweep_extra(h, peaks):
    """The metric's second and third parts on the standalone-kernel sweep: INT8 GeMM^quant TOP/s at M >= 8192 and
    LN^quant GB/s at 65536 rows, as fractions of the measured peaks (burst: each kernel is timed alone)."""
    import torch
    from paper_2310_17723_b200 import microbench as MB, workloads as W
    MB.QUIET = True
    i8_burst = 2.0 * peaks["bf16_tflops"]
    out = {"gemm_int8": [], "ln_quant": [], "peaks": {"int8_tops_burst": i8_burst, "int8_tops_nominal": INT8_NOMINAL_TOPS, "hbm_gbs": peaks["hbm_gbs"]},
           "note": "each kernel timed alone over rotating buffers larger than L2, CUDA events; GEMM epilogue = dequant + bias + "
                   "requant to INT8; LN^quant algorithmic bytes 3 per element, launches timed as CUDA-graph replays"}
    for K, N in W.GEMM_SWEEP_KN:
        for M in (8192, 32768):
            r = MB.bench_gemm(h, M, K, N, "none", False, 10)
            out["gemm_int8"].append({"M": M, "K": K, "N": N, "tops": round(r["tops"], 1), "frac_of_burst": round(r["tops"] / i8_burst, 3),
                                     "frac_of_nominal": round(r["tops"] / INT8_NOMINAL_TOPS, 3)})
            torch.cuda.empty_cache()
    # LN^quant launches of tens of microseconds are timed as CUDA-graph replays (as in profiles/ln_quant.md): between plain
    # launches the host's launch gaps are part of the figure and make it wander from run to run
    MB.GRAPH = True
    for H in W.LN_SWEEP_H:
        for kind in ("f16", "i8"):
            r = MB.bench_ln(h, 65536, H, kind, 40)
            out["ln_quant"].append({"M": 65536, "H": H, "inputs": "fp16" if kind == "f16" else "int8 twq + int8 fwq", "gbs": round(r["gbs"], 0),
                                    "frac_of_hbm": round(r["gbs"] / peaks["hbm_gbs"], 3)})
            torch.cuda.empty_cache()
    MB.GRAPH = False
    try:
        # a library INT8 GEMM of the same size as the driver's BF16 probe, for a MEASURED INT8 figure beside the derived
        # 2 x BF16 one (measurement only: nothing of the product path goes through it)
        a = torch.randint(-127, 128, (8192, 8192), device="cuda", dtype=torch.int8)
        b = torch.randint(-127, 128, (8192, 8192), device="cuda", dtype=torch.int8).t()
        for _ in range(3):
            torch._int_mm(a, b)
        best = 1e9
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); torch._int_mm(a, b); e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        out["peaks"]["int8_tops_library_gemm_8192"] = round(2.0 * 8192 ** 3 / (best * 1e-3) / 1e12, 1)
        del a, b
    except Exception as e:                                     # the figure is optional context
        out["peaks"]["int8_tops_library_gemm_8192"] = None
        out["peaks"]["int8_library_gemm_note"] = "torch._int_mm unavailable: %s" % str(e)[:80]
    torch.cuda.empty_cache()
    return out


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
    post = shape.arch == "post_ln"
    h = hero.Handle()
    stack = Stack(h, shape, cid, cfgs, n_cal_seq=1 if shape.M * shape.H > 2 ** 25 else 2)
    # every rank works on its own batch (replicas: the path shards by sequence, no exchange step)
    x_host = torch.from_numpy(W.activations(shape, cid, tensor=replicas.batch_tensor_index(rank))).to(stack.fp_torch)
    x_dev = x_host.cuda()
    flush = torch.empty(512 * 1024 * 1024, dtype=torch.int8, device="cuda")     # > 126 MB L2
    stream = torch.cuda.current_stream()
    # a step = the whole hot path on one batch: the entry LN^quant (post-LN workloads: it stands for the embedding
    # LayerNorm of Eq. 6-7 and turns the FP16 activations into layer 0's INT8 input) and every layer
    sd_full = stack.desc(entry_in=hero.tensor(x_dev)) if post else stack.desc()
    sd_layers = stack.desc()
    if not post:
        stack.set_input(x_dev)

    def step():
        h.hero_stack_forward(sd_full, stack.workspace)

    def step_layers_only():
        h.hero_stack_forward(sd_layers, stack.workspace)

    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.begin()
    for _ in range(max(args.warmup, 3)):
        flush.zero_()
        step()
    torch.cuda.synchronize()
    h.check()
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
                eager_step()
        torch.cuda.synchronize()

        def step():
            graph.replay()
            replayed[0] += launches_per_step           # the handle counts launches as they are issued, i.e. at capture
        for _ in range(3):
            step()
        torch.cuda.synchronize()

    def timed(fn, steps):
        """`steps` calls of fn, each bracketed by events on the launching stream, L2 flushed before each (outside the
        event pairs).  Returns the summed device milliseconds."""
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for k in range(steps):
            flush.zero_()
            ev[k][0].record(stream)
            fn()
            ev[k][1].record(stream)
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in ev)

    # ---- timed region: K steps
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    wall0 = time.perf_counter()
    n0 = h.launches
    replayed[0] = 0
    my_ms = timed(step, args.steps)
    if dist:
        dist.barrier()
    wall = time.perf_counter() - wall0
    gpu_launches = h.launches - n0 + replayed[0]
    h.check()
    total_ms = replicas.max_over_ranks(my_ms, dist, "cuda")
    ms_per_step = total_ms / args.steps
    value = replicas.job_throughput(shape.M, args.steps, world, total_ms * 1e-3)
    # the same steps without the entry LN^quant (the layers alone, their INT8 input already in place)
    layers_only_ms = timed(step_layers_only, args.steps) / args.steps if post else None
    full_again_ms = timed(step, args.steps) / args.steps if post else None      # the whole step once more, same phase
    # host time of the C-ABI call: a burst of calls short enough to stay inside the driver's launch queue, so the host
    # never waits for the device; wall clock until the last call has returned
    host_us = None
    if rank == 0:
        nburst = max(1, min(64, 512 // max(launches_per_step, 1)))
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(nburst):
            eager_step()
        host_us = (time.perf_counter() - t0) / nburst * 1e6
        torch.cuda.synchronize()

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
        for li, cfg in enumerate(cfgs):
            table += kernel_table(shape, cfg, first=(li == 0))
        assert len(table) == launches_per_step, (len(table), launches_per_step)
        regime, _why = peak_regime(clocks, peaks)
        int8_peak = 2.0 * (peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) if regime == "sustained" else peaks["bf16_tflops"])
        merged = {}
        for i, (name, fam, ops, nbytes) in enumerate(table):
            ms = [recs[j][1] for j in range(i, len(recs), launches_per_step)]
            avg = sum(ms) / len(ms)
            key = (name, fam)
            if key in merged:                                  # same kernel in another layer of the stack
                merged[key] = (merged[key][0] + avg, merged[key][1] + ops, merged[key][2] + nbytes, merged[key][3] + 1)
            else:
                merged[key] = (avg, ops, nbytes, 1)
        mhz = (clocks or {}).get("sm_mhz") or peaks.get("sm_max_mhz", 1965.0)
        for (name, fam), (avg, ops, nbytes, cnt) in merged.items():
            row = {"kernel": name if fam != "gemm_fp" else name + " (fp16)", "ms": round(avg, 5), "share": None, "launches_per_step": cnt}
            if fam == "gemm":
                row.update(bound="tensor", achieved=ops / (avg * 1e-3) / 1e12, peak=int8_peak, unit="TOP/s")
            elif fam == "gemm_fp":
                row.update(bound="tensor", achieved=ops / (avg * 1e-3) / 1e12, peak=int8_peak / 2, unit="TFLOP/s")
            elif fam == "ln":
                row.update(bound="hbm", achieved=nbytes / (avg * 1e-3) / 1e9, peak=peaks["hbm_gbs"], unit="GB/s")
            else:
                # bound by the special-function unit: one exponential per score and sweep that needs it
                # (ops = 4 dh per score, so scores = ops / (4 dh)); peak = 16 ex2 per clock and SM at the sampled clock
                scores = ops / (4.0 * shape.dh)
                row.update(bound="alu", achieved=scores / (avg * 1e-3) / 1e12, peak=148 * 16 * mhz * 1e6 / 1e12,
                           unit="Texp/s", tensor_tops=ops / (avg * 1e-3) / 1e12)
            row["frac"] = row["achieved"] / row["peak"]
            kern.append(row)
        tot = sum(r["ms"] for r in kern)
        for r in kern:
            r["share"] = round(r["ms"] / tot, 4)
        roof = dominant_kernel(kern, args.workload, peaks, peak_kind, clocks)

    # ---- end to end through the C ABI with HOST buffers (pinned), copies inside the timed region:
    # hero_stack_forward_host_async = H2D of the FP activations, entry LN^quant, every layer, D2H of the output
    # (payload and, for a token-wise output, its row scales).  Three steps in flight, each on its own stream with its
    # own chained device buffers, staging tensor, workspace and pinned output: one step's copies overlap another's
    # kernels.  A slot is synchronised (its result is then in host memory) before it is reused.
    DEPTH = 3 if shape.M * shape.H * 2 <= (1 << 28) else 2
    hin = x_host.pin_memory()
    t_out, s_out, _d = stack.bufs[-1]
    g_out = "fp" if t_out.dtype in (torch.float16, torch.bfloat16) else cfgs[-1].gran_out
    slots = []
    for _ in range(DEPTH):
        edges = stack.make_edges()
        stage = torch.empty_like(x_dev)
        if post:
            sd = stack.desc(entry_in=hero.tensor(stage), edges=edges)
        else:
            edges[0] = (stage, None, hero.tensor(stage))
            sd = stack.desc(edges=edges)
        ho = torch.empty_like(edges[-1][0], device="cpu").pin_memory()
        hso = torch.empty(shape.M, dtype=torch.float32).pin_memory() if g_out == "twq" else None
        slots.append({"sd": sd, "host": hero.host_tensor(ho, g_out, hso if g_out == "twq" else None), "keep": (edges, stage, ho, hso),
                      "ws": torch.empty_like(stack.workspace), "stream": torch.cuda.Stream(), "busy": False})
    in_host = hero.host_tensor(hin)
    e2e_k = [0]

    def e2e_step():
        sl = slots[e2e_k[0] % DEPTH]
        e2e_k[0] += 1
        if sl["busy"]:
            sl["stream"].synchronize()
        h.hero_stack_forward_host_async(sl["sd"], in_host, sl["host"], sl["ws"], stream=sl["stream"])
        sl["busy"] = True
    h2d = hin.numel() * hin.element_size()
    d2h = t_out.numel() * t_out.element_size() + (shape.M * 4 if g_out == "twq" else 0)
    for _ in range(3):
        e2e_step()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        e2e_step()
    torch.cuda.synchronize()
    e2e_s = replicas.max_over_ranks(time.perf_counter() - t0, dist, "cuda")
    e2e = {"value": replicas.job_throughput(shape.M, args.steps, world, e2e_s), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
           "d2h_bytes_per_step": int(d2h), "steps_in_flight": DEPTH, "api": "hero_stack_forward_host_async (pinned host buffers)",
           "ms_per_step": 1e3 * e2e_s / args.steps}
    h.check()
    del slots
    torch.cuda.empty_cache()

    fp_path = None
    mixed_path = None
    extra = None
    if rank == 0 and world == 1 and not args.no_fp_path:
        # the same layer(s) in other module modes, through the same library and the same timing loop
        del stack, sd_full, sd_layers
        torch.cuda.empty_cache()

        def time_variant(vcfgs):
            vstack = Stack(h, shape, cid, vcfgs, n_cal_seq=1)
            vsd = vstack.desc(entry_in=hero.tensor(x_dev)) if post else vstack.desc()
            if not post:
                vstack.set_input(x_dev)
            run = lambda: h.hero_stack_forward(vsd, vstack.workspace)
            for _ in range(3):
                flush.zero_()
                run()
            torch.cuda.synchronize()
            ms = timed(run, args.steps) / args.steps
            h.check()
            del vstack, vsd
            torch.cuda.empty_cache()
            return ms

        fms = time_variant(fp_variant(cfgs))                 # every module in FP16 / BF16
        fp_path = {"value": shape.M / (fms * 1e-3), "unit": UNIT, "ms_per_step": fms, "dtype": shape.fp_dtype,
                   "w8a8_speedup": ms_per_step and fms / ms_per_step}
        if args.workload == "c4":
            # the config's comparison: attention and the LN outputs switched to BF16 (so QKV and FC1 run BF16 too),
            # attention-output linear and FC2 stay INT8
            mms = time_variant(attn_ln_fp_variant(cfgs))
            mixed_path = {"modes": "qkv, attention, fc1 in BF16; attention-output linear, fc2 INT8", "value": shape.M / (mms * 1e-3),
                          "unit": UNIT, "ms_per_step": mms, "w8a8_speedup": ms_per_step and mms / ms_per_step}
    if rank == 0 and world == 1 and not args.no_extra:
        extra = sweep_extra(h, peaks)
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
                       "step": ("entry LN^quant + %d layer(s)" % len(cfgs)) if post else "%d pre-LN layer(s)" % len(cfgs),
                       "launch": "CUDA graph replay of the step's launches" if args.graph else
                                 "one C-ABI call per step (hero_stack_forward), %d kernel launches" % launches_per_step,
                       "timing": "CUDA events per step on the launching stream, max over ranks",
                       "parallelism": "replicas x%d (sequence-sharded, no collective)" % world},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(gpu_launches), "roofline": roof, "kernels": kern,
            "kernels_note": "per-launch times come from a second pass with an event pair around every launch, which serialises the "
                            "launches (no programmatic overlap): their sum exceeds ms_per_step, so the fractions are lower bounds",
            "cpu_baseline": cpu, "fp16_path": fp_path, "wall_s_timed_region": wall}
    if layers_only_ms is not None:
        line["without_entry_ln"] = {"ms_per_step": layers_only_ms, "value": shape.M / (layers_only_ms * 1e-3), "unit": UNIT,
                                    "whole_step_same_phase_ms": full_again_ms,
                                    "note": "the layers alone, their INT8 input already in place (one rank's device time); timed after the main "
                                            "region, i.e. later under the power cap: compare it with whole_step_same_phase_ms, the "
                                            "whole step timed right after it, not with ms_per_step"}
    if host_us is not None:
        line["host_us_per_step"] = {"value": host_us, "launches": launches_per_step,
                                    "note": "wall clock of the C-ABI call itself (argument checks, tensor-map lookup, launches), "
                                            "device not waited for"}
    if mixed_path:
        line["attention_and_ln_bf16_path"] = mixed_path
    if extra:
        line["extra"] = extra
    print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


def self_spawn(args):
    """`--gpus N` with N > 1 outside a torchrun environment: start N ranks of this script (one per GPU, rendezvous on
    127.0.0.1); rank 0 prints the JSON line.  Returns the launcher's exit code."""
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus), "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_rendezvous_only(args):
    """The multi-rank plumbing without the workload (also what the CPU test drives): process group, barrier, maximum
    over ranks, one JSON line from rank 0.  NCCL when a GPU per rank is visible, gloo otherwise."""
    import torch
    import torch.distributed as dist
    from paper_2310_17723_b200 import replicas
    rank, local, world = replicas.rank_info()
    use_cuda = torch.cuda.is_available() and torch.cuda.device_count() >= world
    if world > 1:
        if use_cuda:
            torch.cuda.set_device(local)
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group("gloo")
        dist.barrier()
    t = replicas.max_over_ranks(1.0 + rank, dist if world > 1 else None, "cuda" if use_cuda else "cpu")
    if rank == 0:
        print(json.dumps({"rendezvous": "ok", "n_gpus": world, "backend": "nccl" if use_cuda else "gloo", "max_over_ranks": t,
                          "value": replicas.job_throughput(100, 1, world, t)}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", choices=["c1", "c3", "c4", "c5"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-fp-path", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the standalone-kernel sweep figures")
    ap.add_argument("--graph", action="store_true", help="replay the step's launches from a CUDA graph (latency-bound workloads)")
    ap.add_argument("--rendezvous-only", action="store_true", help="only start the ranks, meet and print (no workload)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(self_spawn(args))
    if args.rendezvous_only:
        run_rendezvous_only(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
