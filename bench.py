#!/usr/bin/env python
"""Benchmark of the adaptive self-speculative decoding hot path on B200.

One step = one whole generation on one sequence: prefill of the prompt with the per-sublayer cosine
similarities, Algorithm 1 (ADMG), then rounds of draft steps under the skip mask and one (k+1)-row greedy
verify, until ``max_new`` tokens.  Default workload: the Llama-2-7B-shaped decoder with a 512-token random
prompt and 256 generated tokens.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 7b|13b|7b_long|tiny]

With N > 1 (launched by torch.distributed.run) every rank decodes its own sequence on its own GPU: the path
has no exchange step, so ranks are independent replicas and the value is the sum over ranks.
``--impl reference`` times the CPU oracle on a bounded sample of the same workload (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import synth  # noqa: E402

WORKLOADS = {
    # name: (shape, prompt_len, max_new, description)
    "tiny": (synth.TINY, 32, 64, "tiny decoder L=4 d=256, prompt 32, generate 64"),
    "7b": (synth.LLAMA_7B, 512, 256, "Llama-2-7B-shaped decoder, prompt 512, generate 256"),
    "13b": (synth.LLAMA_13B, 1024, 256, "Llama-2-13B-shaped decoder, prompt 1024, generate 256"),
    "7b_long": (synth.LLAMA_7B, 8192, 512, "Llama-2-7B-shaped decoder, prompt 8192, generate 512"),
}
METRIC = "speculative decode tokens/s"
UNIT = "tokens/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="7b", choices=sorted(WORKLOADS))
    ap.add_argument("--draft-len", type=int, default=4)
    ap.add_argument("--alpha", type=float, default=0.9997)
    ap.add_argument("--m", type=int, default=3)
    ap.add_argument("--n", type=int, default=2)
    ap.add_argument("--flags", type=int, default=5, help="ADMG rule subset: 1=CS thresholding, 2=rule 1, 4=rule 2")
    ap.add_argument("--draft-exit", type=float, default=0.1, help="draft exiting: stop a round's drafting below this top-2 "
                    "logit gap of the draft model (0 = every round drafts --draft-len tokens)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the extra blocks of the line (headline variants, sampling, "
                    "the 8192-token and 13B-shaped workloads)")
    ap.add_argument("--stage-timeline", action="store_true", help="also report the sublayer products of the kernel micro-benchmark "
                    "configuration (d_model 2048..8192) as stages of the pass kernel, from its device timeline")
    ap.add_argument("--no-13b", action="store_true", help="skip the 13B-shaped workload of the extra blocks (26 GB of weights)")
    ap.add_argument("--gemv-microbench", action="store_true", help="also time the stand-alone fused GEMV kernel")
    ap.add_argument("--ablation", action="store_true", help="also time the rule subsets of the paper's ablation (Table 5) and "
                    "the two extensions (MLP similarity threshold, running similarities) end to end")
    ap.add_argument("--alpha-mlp", type=float, default=0.9995, help="MLP similarity threshold of the ablation's extension rows")
    ap.add_argument("--refresh", type=int, default=8, help="rounds between mask updates of the ablation's running-similarity row")
    ap.add_argument("--gemv-shape", default="", help="time the stand-alone fused GEMV on one shape only: "
                    "n_in,n_rows,rows,epilogue with epilogue one of plain, swiglu, residual (e.g. 4096,22016,1,swiglu)")
    ap.add_argument("--gemm-microbench", action="store_true", help="also time the stand-alone tensor-core GEMM of the prompt path")
    # reduced cases for profiler captures only (never for a reported number)
    ap.add_argument("--prompt-len", type=int, default=0, help="override the workload's prompt length")
    ap.add_argument("--max-new", type=int, default=0, help="override the workload's generation length")
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count")
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def measured_traffic_ratio():
    """DRAM bytes per algorithmic byte of the one-row pass kernel, from the ncu capture summarised under profiles/
    (taken on a 4-layer case; the kernel's traffic is its weight stream, which grows in proportion to the layers).
    None when the kernel sources have changed since the counters were taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "pass_kernel_m1_dram_traffic.txt")
    if not os.path.exists(path):
        return None
    rec = dict(line.strip().split("=", 1) for line in open(path) if "=" in line and not line.startswith("#"))
    h = hashlib.sha256()
    for name in ("pass.cuh", "ring.cuh", "common.cuh"):
        with open(os.path.join(ROOT, "paper_2410_01028_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    if rec.get("sources_sha256") != h.hexdigest():
        return None
    return float(rec["dram_bytes"]) / float(rec["algorithmic_bytes"])


def tensor_peak():
    """Dense bf16 TFLOP/s of a cuBLAS GEMM on this machine: (burst, sustained, kind)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return float(d["bf16_tflops"]), float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "measured"
    return 1590.0, 1400.0, "fallback"


def prefill_flops(shape, S):
    """Floating-point operations of the prompt pass (Section 3.2): the sublayer products of all S rows, the LM head of
    the last row, and causal attention (Q K^T and P V over keys <= the row's position)."""
    d, f, L, kvd = shape.d_model, shape.d_ffn, shape.n_layers, shape.kv_dim
    per_row = 2.0 * L * (d * (d + 2 * kvd) + d * d + 3 * d * f)
    attn = 2.0 * 2.0 * L * d * (S * (S + 1) / 2.0)
    return S * per_row + attn + 2.0 * shape.vocab * d


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def workload(args):
    import dataclasses
    shape, S, new, desc = WORKLOADS[args.workload]
    reduced = []
    if args.layers:
        shape = dataclasses.replace(shape, n_layers=args.layers); reduced.append("%d layers" % args.layers)
    if args.prompt_len:
        S = args.prompt_len; reduced.append("prompt %d" % S)
    if args.max_new:
        new = args.max_new; reduced.append("generate %d" % new)
    if reduced:
        desc += " [REDUCED for profiling: " + ", ".join(reduced) + "]"
    return shape, S, new, desc


def admg_kwargs(a):
    return dict(draft_len=a.draft_len, alpha=a.alpha, m=a.m, n=a.n, flags=a.flags, draft_exit_margin=a.draft_exit)


# ---------------------------------------------------------------------------------------------- CPU oracle legs
def oracle_sample(args, model, shape, prompt, steps, warmup):
    """The oracle, as it stands, on a bounded sample of the workload: the first 64 prompt tokens, 12 new tokens."""
    import oracle
    n_prompt, max_new = min(64, len(prompt)), 12
    orc = oracle.Oracle(model, max_seq=n_prompt + max_new + 8)
    kw = admg_kwargs(args)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        toks, _, st = orc.generate(prompt[:n_prompt], max_new, mode=oracle.MODE_SPEC, **kw)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    per_step = sum(times) / len(times)
    # the oracle's time per pass (its own clocks around each pass), at this sample's context length
    pass_ms = {"draft": st["ms_draft"] / max(st["draft_passes"], 1), "verify": st["ms_verify"] / max(st["verify_passes"], 1),
               "verify_rows": 1 + st["drafted"] / max(st["verify_passes"], 1)}
    t0 = time.perf_counter()
    orc.decode_step(int(toks[-1]))
    pass_ms["full"] = (time.perf_counter() - t0) * 1e3
    return {"value": max_new / per_step, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "first %d prompt tokens, %d generated tokens, same ADMG and draft settings; %.1f s per step"
                      % (n_prompt, max_new, per_step),
            "pass_ms": pass_ms, "pass_ms_at": "%d to %d cached positions (the oracle's cost per row is dominated by the "
                                             "weights, not by the context)" % (n_prompt, n_prompt + max_new)}, per_step


def run_reference(args):
    _, rank, _ = rank_env()
    if rank != 0:
        return
    shape, S, new, desc = workload(args)
    model = synth.make_model(shape, seed=0)
    prompt = synth.make_prompt(shape.vocab, S, seed=1)
    steps, warmup = max(1, min(args.steps, 3)), min(args.warmup, 1)
    cb, per_step = oracle_sample(args, model, shape, prompt, steps, warmup)
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": desc, "sample": cb["sample"], **admg_kwargs(args)},
            "cpu_baseline": cb,
            "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------- GPU legs
def gemv_roofline(torch, asd, d, n_rows, M, epi, hbm_peak):
    """Times the stand-alone sublayer kernel (fused RMSNorm -> GEMV -> epilogue) on one shape, over a pool of distinct
    weight matrices larger than L2, with CUDA events on the launching stream."""
    per_launch = n_rows * d * 2
    pool = max(2, int(300e6 // per_launch) + 1)
    dev = torch.device("cuda")
    W = [torch.from_numpy(synth.make_matrix_bf16((n_rows, d), seed=7, stream=100 + i).view(np.int16)).to(dev)
         .view(torch.bfloat16) for i in range(min(pool, 2))]
    while len(W) < pool:
        W.append(W[len(W) % 2].clone())
    x = torch.from_numpy(synth.make_array_f32((M, d), seed=7, stream=99)).to(dev)
    gain = torch.from_numpy(synth.make_matrix_bf16((d,), seed=7, stream=98, mean=1.0).view(np.int16)).to(dev).view(torch.bfloat16)
    if epi == asd.EPI_SWIGLU:
        out = torch.empty((M, n_rows // 2), dtype=torch.bfloat16, device=dev)
    else:
        out = torch.zeros((M, n_rows), dtype=torch.float32, device=dev)
    cos = torch.zeros(16, dtype=torch.float32, device=dev)
    scratch = torch.zeros(asd.fused_gemv_scratch_bytes(), dtype=torch.uint8, device=dev)
    # the launches are captured in a CUDA graph (one pass over the pool per replay) so that the host's launch cost
    # does not bound the small shapes
    for i in range(pool):
        asd.fused_gemv(x, W[i % pool], epi, out, gain=gain, cos=cos, scratch=scratch)
    torch.cuda.synchronize()
    n_graph = max(pool, 20)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(n_graph):
            asd.fused_gemv(x, W[i % pool], epi, out, gain=gain, cos=cos, scratch=scratch)
    graph.replay()
    reps = 10
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (reps * n_graph)
    achieved = per_launch / (us * 1e-6) / 1e9
    names = {asd.EPI_PLAIN: "plain", asd.EPI_SWIGLU: "swiglu", asd.EPI_RESIDUAL: "residual+cosine"}
    return {"in": d, "out": n_rows, "rows": M, "epilogue": names[epi], "bytes_per_launch": per_launch, "us_per_launch": round(us, 2),
            "GBps": round(achieved, 1), "frac": round(achieved / hbm_peak, 3)}


def gemv_sweep(torch, asd, hbm_peak):
    """The stand-alone fused kernel over the sublayer shapes of d_model 2048..8192 (out = d with the residual + cosine
    epilogue, 3d plain, 2.6875d rows alternating gate / up with SwiGLU, and the W_d shape in = 2.6875d -> out = d), at
    1 and 5 rows, RMSNorm prologue on."""
    res = []
    for d in (2048, 4096, 5120, 8192):
        f2 = int(2.6875 * d)
        for M in (1, 5):
            for n_in, n_rows, epi in ((d, d, asd.EPI_RESIDUAL), (d, 3 * d, asd.EPI_PLAIN), (d, f2, asd.EPI_SWIGLU),
                                      (f2, d, asd.EPI_RESIDUAL)):
                res.append(gemv_roofline(torch, asd, n_in, n_rows, M, epi, hbm_peak))
    return res


def gemm_roofline(torch, asd, shape):
    """Times the stand-alone tcgen05 GEMM of the prompt path at the gate/up shape with 2048 rows (one chunk), over a
    pool of weight matrices larger than L2, with CUDA events on the launching stream."""
    d, n_rows, M = shape.d_model, 2 * shape.d_ffn, 2048
    dev = torch.device("cuda")
    pool = max(2, int(400e6 // (n_rows * d * 2)) + 1)
    W = [torch.from_numpy(synth.make_matrix_bf16((n_rows, d), seed=7, stream=100 + i).view(np.int16)).to(dev)
         .view(torch.bfloat16) for i in range(min(pool, 2))]
    while len(W) < pool:
        W.append(W[len(W) % 2].clone())
    A = torch.from_numpy(synth.make_matrix_bf16((M, d), seed=7, stream=97, std=1.0).view(np.int16)).to(dev).view(torch.bfloat16)
    C = torch.empty((M, n_rows), dtype=torch.float32, device=dev)
    status = torch.zeros(8, dtype=torch.int32, device=dev)
    n = 50
    for i in range(5):
        asd.gemm_bf16(A, W[i % pool], C, status)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(n):
        asd.gemm_bf16(A, W[i % pool], C, status)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / n
    burst, _, kind = tensor_peak()
    tf = 2.0 * M * n_rows * d / (us * 1e-6) / 1e12
    return {"bound": "tensor", "kernel": "gemm_tn_kernel<256> %dx%dx%d (fp32 out)" % (M, n_rows, d), "us_per_launch": us,
            "achieved": tf, "peak": burst, "unit": "TFLOP/s", "frac": tf / burst, "peak_kind": kind + " burst (kernel timed alone)",
            "status": int(status[0].item())}


def ablation(torch, asd, dec, dev_prompt, dev_out, new, args, ar_tokens):
    """One speculative generation per rule subset of the paper's ablation (Table 5: similarity threshold alone, with
    rule 2, rules 1 and 2 alone, all three) and per extension, with the hyper-parameters of the command line."""
    CS, R1, R2 = asd.USE_CS, asd.USE_RULE1, asd.USE_RULE2
    rows = [("CS", CS), ("CS + rule 2", CS | R2), ("rules 1 and 2", R1 | R2), ("CS + rules 1 and 2 (Algorithm 1)", CS | R1 | R2),
            ("CS + rule 2 + MLP threshold", CS | R2 | asd.USE_CS_MLP),
            ("CS + rule 2 + MLP threshold, running similarities", CS | R2 | asd.USE_CS_MLP | asd.RUNNING_C)]
    out = []
    for name, flags in rows:
        kw = dict(draft_len=args.draft_len, alpha=args.alpha, m=args.m, n=args.n, flags=flags, alpha_mlp=args.alpha_mlp,
                  refresh=args.refresh if flags & asd.RUNNING_C else 0, draft_exit_margin=args.draft_exit)
        dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_SPEC, **kw)  # warm-up
        _, st = dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_SPEC, **kw)
        same = bool((dev_out.cpu().numpy() == ar_tokens).all())
        ra, rm = dec.admg_update(args.alpha, args.m, args.n, flags, alpha_mlp=args.alpha_mlp)
        out.append({"rules": name, "flags": flags, "tokens_per_s": new / (st["ms_total"] * 1e-3),
                    "acceptance": st["accepted"] / max(st["drafted"], 1), "removed_attn": int(ra.sum()), "removed_mlp": int(rm.sum()),
                    "draft_ms": st["ms_draft"] / max(st["draft_passes"], 1), "spec_equals_ar": same})
    return out


def headline_variants(asd, dec, dev_prompt, dev_out, new, args, ar_tokens):
    """The same workload under three settings of the draft-model generator, so that the headline's dependence on the
    tuned threshold and on draft exiting (an extension the paper only points to) is visible: Table 2's
    hyper-parameters with all three rules; the threshold of the command line without draft exiting; and with it."""
    rows = [("Algorithm 1 with Table 2's hyper-parameters (alpha 0.985, m 3, n 2), no draft exiting",
             dict(draft_len=args.draft_len, alpha=0.985, m=3, n=2, flags=asd.ADMG_ALL, draft_exit_margin=0.0)),
            ("command-line setting without draft exiting", dict(admg_kwargs(args), draft_exit_margin=0.0)),
            ("command-line setting (the headline)", admg_kwargs(args))]
    out = []
    for name, kw in rows:
        dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_SPEC, **kw)
        _, st = dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_SPEC, **kw)
        ra, rm = dec.admg_update(kw["alpha"], kw["m"], kw["n"], kw["flags"])
        out.append({"setting": name, "tokens_per_s": new / (st["ms_total"] * 1e-3), "acceptance": st["accepted"] / max(st["drafted"], 1),
                    "removed_attn": int(ra.sum()), "removed_mlp": int(rm.sum()),
                    "draft_ms": st["ms_draft"] / max(st["draft_passes"], 1), "verify_ms": st["ms_verify"] / max(st["verify_passes"], 1),
                    "spec_equals_ar": bool((dev_out.cpu().numpy() == ar_tokens).all())})
    return out


def sampling_rows(asd, dec, dev_prompt, dev_out, new, args):
    """Sampling-based decoding at the paper's temperatures (Tables 3 and 4): plain sampled decoding and speculative
    decoding with distribution-preserving acceptance, same seed."""
    out = []
    for T in (0.2, 0.6):
        dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_AR, temperature=T, seed=1)
        _, st_a = dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_AR, temperature=T, seed=1)
        kw = dict(admg_kwargs(args), temperature=T, seed=1)
        dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_SPEC, **kw)
        _, st_s = dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_SPEC, **kw)
        out.append({"temperature": T, "sampled_ar_tokens_per_s": new / (st_a["ms_total"] * 1e-3),
                    "sampled_spec_tokens_per_s": new / (st_s["ms_total"] * 1e-3),
                    "acceptance": st_s["accepted"] / max(st_s["drafted"], 1)})
    return out


def other_workload(torch, asd, name, args, hbm_peak, peak_kind, model=None):
    """One more workload of the benchmark family in the same line (one warm-up and one timed generation each of plain
    greedy and speculative decoding): per-pass times, roofline fractions, tokens/s."""
    shape, S, new, desc = WORKLOADS[name]
    t0 = time.perf_counter()
    if model is None:
        model = synth.make_model(shape, seed=0)
    dec = asd.Decoder(shape, max_seq=S + new + 16, max_draft=8)
    dec.load_weights_host(model)
    dev_prompt = torch.from_numpy(synth.make_prompt(shape.vocab, S, seed=1)).cuda()
    dev_out = torch.zeros(new, dtype=torch.int32, device="cuda")
    kw = dict(admg_kwargs(args), draft_len=6 if name == "13b" else args.draft_len)
    dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_AR)
    _, st_ar = dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_AR)
    ar = dev_out.cpu().numpy().copy()
    dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_SPEC, **kw)
    _, st = dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_SPEC, **kw)
    same = bool((dev_out.cpu().numpy() == ar).all())

    def pp(kind, s):
        n = s[kind + "_passes"]
        if not n:
            return None
        gbs = s["bytes_" + kind] / s["ms_" + kind] / 1e6
        return {"ms": s["ms_" + kind] / n, "GBps": gbs, "frac_of_%s_peak" % peak_kind: gbs / hbm_peak, "frac_of_8TBps": gbs / 8000.0}

    _, tf_sustained, _ = tensor_peak()
    pf_tf = prefill_flops(shape, S) / (st["ms_prefill"] * 1e-3) / 1e12
    res = {"workload": desc, "draft_len": kw["draft_len"], "spec_tokens_per_s": new / (st["ms_total"] * 1e-3),
           "ar_tokens_per_s": new / (st_ar["ms_total"] * 1e-3), "acceptance": st["accepted"] / max(st["drafted"], 1),
           "spec_equals_ar": same, "passes": {"full": pp("full", st_ar), "draft": pp("draft", st), "verify": pp("verify", st)},
           "prefill_ms": st["ms_prefill"], "prefill_TFLOPs": pf_tf, "prefill_frac_of_sustained_tensor_peak": pf_tf / tf_sustained,
           "wall_s": None}
    dec.close()
    del dec
    torch.cuda.empty_cache()
    res["wall_s"] = time.perf_counter() - t0
    return res


def stage_timeline(torch, asd, d, hbm_peak):
    """The sublayer products of BASELINE config 2 (in = d -> out = d / 3d / 2 x 2.6875d, and in = 2.6875d -> out = d) as the
    stages of the pass kernel: a 2-layer decoder of width d, the device timeline of one decode pass (1 row) and one verify
    pass (5 rows), per stage the time from the end of the previous stage to the end of this one (everything a stage
    costs: waiting for its inputs, RMSNorm prologue, weight stream, epilogue) and the weight bytes per that time."""
    f = int(2.6875 * d)
    shape = synth.DecoderShape(n_layers=2, d_model=d, n_heads=d // 128, head_dim=128, d_ffn=f, vocab=32000)
    model = synth.make_model(shape, seed=3)
    dec = asd.Decoder(shape, max_seq=160, max_draft=8)
    dec.load_weights_host(model)
    prompt = synth.make_prompt(shape.vocab, 64, seed=1)
    t = dec.prefill(prompt)
    dec.set_debug(record_logits=False, trace=True)
    names = {1: ("qkv", "in d -> out 3d, rotary + K/V append", 2.0 * 3 * d * d), 3: ("o_proj", "in d -> out d, residual + cosine", 2.0 * d * d),
             4: ("gate_up", "in d -> out 2 x 2.6875d, SwiGLU", 2.0 * 2 * f * d), 5: ("down", "in 2.6875d -> out d, residual + cosine", 2.0 * d * f)}
    types = [0, 1, 2, 3, 4, 5, 1, 2, 3, 4, 5, 7, 6]
    out = []
    for rows in (1, 5):
        best = {}
        for rep in range(4):
            if rows == 1:
                t = dec.decode_step(t)
            else:
                a, o = dec.verify([t] + [1] * (rows - 1))
                t = int(o[-1])
            tr = dec.get_last_trace()
            for s in range(6, 11):                       # the second layer: its first stage follows a full stage, not the embedding
                if types[s] in names:
                    period = float(np.median(tr[s, 3] - tr[s - 1, 3])) / 1e3
                    stream = float(np.median(tr[s, 2] - tr[s, 7])) / 1e3
                    key = types[s]
                    if key not in best or period < best[key][0]:
                        best[key] = (period, stream)
        for key, (period, stream) in sorted(best.items()):
            nm, what, nbytes = names[key]
            out.append({"d": d, "rows": rows, "stage": nm, "shape": what, "MB": round(nbytes / 1e6, 1), "us": round(period, 2),
                        "GBps": round(nbytes / period / 1e3, 1), "frac": round(nbytes / period / 1e3 / hbm_peak, 3),
                        "stream_only_us": round(stream, 2)})
    dec.close()
    del dec
    torch.cuda.empty_cache()
    return out


def rank_env():
    """(world size, rank, local rank) from the environment torch.distributed.run sets up; (1, 0, 0) without it."""
    return int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0"))


def max_over_ranks(value, world, device):
    """A timing taken on every replica becomes the slowest replica's (replicas only: no data-path collective)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world, steps, new_tokens, ms):
    """Tokens per second of all replicas together: every replica generates `new_tokens` per step."""
    return world * steps * new_tokens / (ms * 1e-3)


def replica_prompt(vocab, n, rank):
    """Every replica decodes its own sequence."""
    return synth.make_prompt(vocab, n, seed=1 + rank)


def run_ours(args):
    import torch
    import paper_2410_01028_b200 as asd

    world, rank, local = rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    shape, S, new, desc = workload(args)
    hbm_peak, peak_kind = peaks()

    model = synth.make_model(shape, seed=0)
    dec = asd.Decoder(shape, max_seq=S + new + 16, max_draft=8, device="cuda:%d" % local)
    dec.load_weights_host(model)
    prompt = replica_prompt(shape.vocab, S, rank)
    dev_prompt = torch.from_numpy(prompt).cuda()
    dev_out = torch.zeros(new, dtype=torch.int32, device="cuda")
    kw = admg_kwargs(args)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # plain greedy decoding of the same workload by the same library (comparison value, outside the timed region)
    n_ar, st_ar = dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_AR)
    ar_tokens = dev_out.cpu().numpy().copy()

    for _ in range(args.warmup):
        dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_SPEC, **kw)
    sampler = ClockSampler(local)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    e0.record()
    launches = 0
    agg = None
    for _ in range(args.steps):
        n_out, st = dec.generate_device(dev_prompt, dev_out, new, mode=asd.MODE_SPEC, **kw)
        launches += st["kernel_launches"]
        agg = st if agg is None else {k: agg[k] + st[k] for k in st}
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
    lossless = bool((dev_out.cpu().numpy() == ar_tokens).all())
    value = whole_job_value(world, args.steps, new, ms)

    # end to end through the host-buffer entry point: prompt from pinned host memory, tokens back to the host
    pinned = torch.from_numpy(prompt).pin_memory()
    host_prompt = pinned.numpy()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        toks, _ = dec.generate(host_prompt, new, mode=asd.MODE_SPEC, **kw)
    torch.cuda.synchronize()
    e2e_s = max_over_ranks(time.perf_counter() - t0, world, "cuda")
    e2e = {"value": whole_job_value(world, args.steps, new, e2e_s * 1e3), "unit": UNIT, "h2d_bytes_per_step": int(prompt.nbytes),
           "d2h_bytes_per_step": int(toks.nbytes) + 4 * int(agg["rounds"] // args.steps) * (args.draft_len + 2)
                                 + (4 * int(agg["draft_passes"] // args.steps) if args.draft_exit > 0 else 0)}

    if rank != 0:
        return

    def per_pass(kind, st):
        n = st[kind + "_passes"]
        if not n:
            return None
        msp = st["ms_" + kind] / n
        gbs = st["bytes_" + kind] / st["ms_" + kind] / 1e6
        return {"ms": msp, "GBps": gbs, "frac_of_%s_peak" % peak_kind: gbs / hbm_peak, "frac_of_8TBps": gbs / 8000.0}

    passes = {"full": per_pass("full", st_ar), "draft": per_pass("draft", agg), "verify": per_pass("verify", agg)}
    # Dominant kernel: the persistent pass kernel at one row (every draft step and every plain decode step is one
    # launch of it). Its launches are timed inside the timed region by the library's CUDA events on the launching
    # stream; algorithmic bytes per launch = weights of the sublayers that ran + K/V read + LM head.
    dom = "draft" if agg["draft_passes"] else "full"
    dom_st = agg if agg["draft_passes"] else st_ar
    n_launch = dom_st[dom + "_passes"]
    us_per_launch = dom_st["ms_" + dom] / n_launch * 1e3
    bytes_per_launch = dom_st["bytes_" + dom] / n_launch
    achieved = bytes_per_launch / (us_per_launch * 1e-6) / 1e9
    ratio = measured_traffic_ratio()
    roofline = {"bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak,
                "traffic": None if ratio is None else ratio * bytes_per_launch,
                "traffic_how": None if ratio is None else "ncu dram__bytes_read.sum + dram__bytes_write.sum of a 4-layer pass, scaled by "
                               "algorithmic bytes (%.4f DRAM bytes per algorithmic byte)" % ratio,
                "peak_kind": peak_kind,
                "kernel": "pass_kernel<1> (%s pass: one persistent launch per pass)" % dom,
                "launches": int(n_launch), "bytes_per_launch": bytes_per_launch, "us_per_launch": us_per_launch,
                "how": "CUDA events around every launch inside the timed region, on the launching stream"}
    if args.gemv_microbench:
        roofline["fused_gemv_alone"] = gemv_sweep(torch, asd, hbm_peak)
    if args.stage_timeline:
        roofline["stage_timeline"] = [r for dd in (2048, 4096, 5120, 8192) for r in stage_timeline(torch, asd, dd, hbm_peak)]
    if args.gemv_shape:
        n_in, n_rows, rows, epi = args.gemv_shape.split(",")
        epi = {"plain": asd.EPI_PLAIN, "swiglu": asd.EPI_SWIGLU, "residual": asd.EPI_RESIDUAL}[epi]
        roofline["fused_gemv_alone"] = [gemv_roofline(torch, asd, int(n_in), int(n_rows), int(rows), epi, hbm_peak)]
    # the prompt pass is the tensor-core part of a step: dense products + causal attention, then one decode pass
    _, tf_sustained, tf_kind = tensor_peak()
    pf_ms = agg["ms_prefill"] / args.steps
    pf_tf = prefill_flops(shape, S) / (pf_ms * 1e-3) / 1e12
    prefill = {"ms": pf_ms, "bound": "tensor", "achieved": pf_tf, "peak": tf_sustained, "unit": "TFLOP/s",
               "frac": pf_tf / tf_sustained, "peak_kind": tf_kind + " sustained",
               "what": "whole prompt pass (GEMMs on tcgen05, flash attention, row kernels, the LM head stage of the pass kernel on the last row)"}
    if args.gemm_microbench:
        prefill["gemm_alone"] = gemm_roofline(torch, asd, shape)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 weights and activations, f32 accumulate", "data": "synthetic",
        "config": {"workload": desc, "l2": "inputs larger than L2 (weights %.1f GB per pass)" % (model.nbytes() / 1e9),
                   "parallelism": "replicas only" if world > 1 else "single GPU", **kw},
        "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
        "roofline": roofline, "passes": passes,
        "decode_tokens_per_s": (new - 1) / ((agg["ms_total"] - agg["ms_prefill"]) / args.steps * 1e-3),
        "prefill_ms": agg["ms_prefill"] / args.steps, "prefill": prefill,
        "ar_tokens_per_s": new / (st_ar["ms_total"] * 1e-3),
        "ar_decode_tokens_per_s": (new - 1) / ((st_ar["ms_total"] - st_ar["ms_prefill"]) * 1e-3),
        "acceptance": agg["accepted"] / max(agg["drafted"], 1), "rounds_per_step": agg["rounds"] / args.steps,
        "spec_equals_ar": lossless,
    }
    if args.ablation:
        line["ablation"] = ablation(torch, asd, dec, dev_prompt, dev_out, new, args, ar_tokens)
    if not args.no_cpu_baseline:
        cb, _ = oracle_sample(args, model, shape, synth.make_prompt(shape.vocab, S, seed=1), 1, 0)
        line["cpu_baseline"] = cb
    if not args.no_extras and world == 1 and not (args.layers or args.prompt_len or args.max_new):
        line["headline_variants"] = headline_variants(asd, dec, dev_prompt, dev_out, new, args, ar_tokens)
        line["sampling"] = sampling_rows(asd, dec, dev_prompt, dev_out, new, args)
        if args.workload == "7b":
            # the long-context workload shares the 7B-shaped weights; the 13B-shaped one generates its own
            dec.close()
            del dec
            torch.cuda.empty_cache()
            others = [other_workload(torch, asd, "7b_long", args, hbm_peak, peak_kind, model=model)]
            if not args.no_13b:
                del model
                others.append(other_workload(torch, asd, "13b", args, hbm_peak, peak_kind))
            line["other_workloads"] = others
    print(json.dumps(line))


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
