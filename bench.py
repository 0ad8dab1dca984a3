#!/usr/bin/env python
"""Benchmark of the LSP decode hot path on B200:  python bench.py --gpus N --steps K --warmup W

One *step* is one whole LSP decode (Algorithm 1: every denoiser pass, fused LM-head confidence reduction, scan,
commit and KV append) of one batch of the workload.  The default workload is the LLaDA-8B-shaped full decode
("cfg3": 32 layers, d 4096, 32x128 heads, FFN 12288, vocab 126464, bf16, batch 1, prompt 256 + 256 masked,
tau 0.9, delimiters 1..32); `--workload cfg4|cfg5|cfg2` selects the Dream-7B-shaped decode, the long batched
decode or the head-only configuration.  Weights and prompts are seeded synthetic values (random init).

Prints ONE JSON line:
  value          committed tokens/s over the K timed decodes, inputs resident in HBM (CUDA events, max over ranks)
  e2e            the same through lsp_generate_host: prompt copied from pinned host memory and the finished token
                 buffer copied back inside the timed region, every decode
  roofline       the dominant kernel class of the workload (layer GEMMs), algorithmic bytes / kernel time, measured
                 with per-launch CUDA events in a second pass over the same K decodes
  classes        the same figures for every kernel class (attention, LM head, append, ...)
  cpu_baseline   the CPU oracle timed on a bounded sample of the same workload (rank 0, N = 1 only)
  also           the other workloads: a shorter run of the Dream-7B-shaped decode (cfg4, tensor-bound passes), the
                 head-only configuration (cfg2) and the long batched decode next to scattered acceptance (cfg5)
  loop_variants  ms per pass of the same decode with the block lengths kept on the device and / or the in-place K/V
                 layout, beside the synchronous loop with the append copy (the contract, which `value` times)
  adaptive_tau   the same workload decoded in the adaptive-threshold mode (Eq. 2, block in [0.25 N, 0.50 N]): passes,
                 suffix length per pass (geometric decay), rows touched in total against the G/beta..G/alpha bounds

`--impl reference` times the CPU oracle alone (there is no other reference implementation of this path).
With N > 1 (torchrun) every rank runs an independent replica of the workload with its own prompts: the path has
no exchange step, so there is no collective on it; only the timing is reduced (max) across ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

CLASSES = ("misc", "gemm", "attn", "head", "scan", "commit")
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch from the ncu captures summarised under
# profiles/, keyed by kernel class: the captured launch's traffic and algorithmic bytes, and the hash of the kernel
# sources the capture was taken on.  The class's launches differ in shape, and traffic grows in proportion to the
# weight bytes streamed, so the reported figure is the class's mean algorithmic bytes per launch scaled by the
# captured ratio.  A class whose sources changed since the capture reports null.
CLASS_SOURCES = {
    "gemm": ("gemm_stream.cuh", "gemm_swap.cuh", "gemm_umma.cuh", "epilogues.cuh", "common.cuh"),
    "head": ("gemm_stream.cuh", "gemm_swap.cuh", "gemm_umma.cuh", "epilogues.cuh", "common.cuh"),
    "attn": ("attention_umma.cuh", "common.cuh"),
    "commit": ("misc_kernels.cuh", "common.cuh"),
}
NCU_TRAFFIC = {
    # k_gemm_stream<128,1,1,EpiStore>, M 64, N 12288, K 4096: profiles/k_gemm_stream_M64_N12288_K4096.md
    "gemm": {"captured_bytes": 105.06e6, "algorithmic_bytes": 102.8e6, "src": "34127c2c8b24"},
    # k_gemm_stream<256,1,1,EpiHead>, 64 rows: profiles/k_gemm_stream_head_M64_V126464.md
    "head": {"captured_bytes": 1062.8e6, "algorithmic_bytes": 1037.0e6, "src": "34127c2c8b24"},
    # k_attn_umma, 16 x (128 query rows over 2048 keys): profiles/k_attn_umma_B16_F1920.md
    "attn": {"captured_bytes": 569.2e6, "algorithmic_bytes": 570.4e6, "src": "196044e4044b"},
    # k_commit_append of a 16 x 1920-row prompt block: profiles/k_commit_append_prompt_B16_P1920.md
    "commit": {"captured_bytes": 1968.9e6, "algorithmic_bytes": 2013.3e6, "src": "10338810cc4a"},
}


def source_hash(name=None):
    h = hashlib.sha1()
    d = os.path.join(ROOT, "paper_2603_05454_b200", "csrc")
    files = CLASS_SOURCES.get(name) or sorted(os.listdir(d))
    for f in files:
        h.update(open(os.path.join(d, f), "rb").read())
    return h.hexdigest()[:12]


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return json.load(open(p)), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid = uuid
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", self.uuid, "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        rows = [l.strip().split(", ") for l in open(self.f.name) if l.strip()]
        os.unlink(self.f.name)
        sm, mx, pw, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.strip() == "Active":
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm_sorted = sorted(sm)
        return {"sm_mhz": sm_sorted[len(sm_sorted) // 2], "sm_max_mhz": max(mx), "power_w_max": max(pw),
                "samples": len(sm), "reasons": sorted(reasons)}


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 0) for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


# ------------------------------------------------------------------------------------------------------------
# CPU oracle legs (the only place this file executes oracle/)
# ------------------------------------------------------------------------------------------------------------
ORACLE_LAYERS = 1     # depth of the model slice the oracle sample runs
ORACLE_STEPS = 2      # denoiser steps of the decode the sample covers


def oracle_sample_setup(wl, gen_device):
    """Builds the oracle model for a slice (first ORACLE_LAYERS layers, full widths and vocabulary) of the workload's
    model and the prompt of sequence 0.  Input values come from the shared seeded generator."""
    import dataclasses
    import lsp_synth as S
    from oracle import dlm
    sh = dataclasses.replace(wl.shape, n_layers=min(ORACLE_LAYERS, wl.shape.n_layers))
    w = S.make_weights(sh, 0, device=gen_device)
    om = dlm.OracleDLM(sh, w)
    del w
    prompt = S.make_prompt(1, wl.prompt_len, sh, 0)[0].numpy()
    return sh, om, prompt


def oracle_sample_run(wl, om, prompt):
    """ORACLE_STEPS steps of the oracle's decode of one sequence.  Returns (seconds, tokens committed)."""
    import numpy as np
    from oracle.decode import decode, make_is_delim
    t0 = time.perf_counter()
    _, recs, _ = decode(om, prompt, wl.gen_len, make_is_delim(*wl.delim),
                        dict(tau=float(np.float32(wl.tau))), max_steps=ORACLE_STEPS)
    dt = time.perf_counter() - t0
    return dt, sum(r["L_commit"] for r in recs)


def oracle_sample_text(wl):
    return (f"oracle.decode, first {ORACLE_STEPS} denoiser steps of one sequence of {wl.name} "
            f"(prompt {wl.prompt_len} + {wl.gen_len} masked) on a {ORACLE_LAYERS}-layer slice of the model "
            f"(full widths and vocabulary); value = tokens it committed / (seconds x n_layers/{ORACLE_LAYERS}), "
            "i.e. scaled to the full depth (the head's share is scaled too, so a lower bound on the oracle's rate)")


def run_reference(args):
    """The reference arm: the CPU oracle as it stands, on the host cores."""
    import torch
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import lsp_synth as S
    wl = S.config(args.workload if args.workload != "cfg2" else "cfg3")
    gen_device = "cuda:0" if torch.cuda.is_available() else "cpu"
    sh, om, prompt = oracle_sample_setup(wl, gen_device)
    scale = wl.shape.n_layers / sh.n_layers
    for _ in range(args.warmup):
        oracle_sample_run(wl, om, prompt)
    t, tok = 0.0, 0
    for _ in range(args.steps):
        dt, n = oracle_sample_run(wl, om, prompt)
        t += dt
        tok += n
    value = tok / (t * scale)
    cores = blas_threads()
    line = {"impl": "reference", "metric": "committed_tokens_per_s", "value": value, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "batch": 1, "prompt_len": wl.prompt_len, "gen_len": wl.gen_len,
                       "tau": wl.tau, "step": "one bounded oracle sample"},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                             "sample": oracle_sample_text(wl)},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------------------------------------
# replicas: the only cross-rank step is the reduction of the timing
# ------------------------------------------------------------------------------------------------------------
def reduce_replicas(ms_local, tokens_local, world, device="cpu"):
    """Whole-job figures of `world` independent replicas: every rank decodes its own batch, the job takes as long as
    its slowest rank (MAX over ranks of each entry of ms_local) and commits the sum of the ranks' tokens."""
    import torch
    ms = torch.tensor(list(ms_local), dtype=torch.float64, device=device)
    tok = torch.tensor([float(tokens_local)], dtype=torch.float64, device=device)
    if world > 1:
        torch.distributed.all_reduce(ms, op=torch.distributed.ReduceOp.MAX)
        torch.distributed.all_reduce(tok, op=torch.distributed.ReduceOp.SUM)
    return [float(x) for x in ms], float(tok[0])


# ------------------------------------------------------------------------------------------------------------
# the CUDA path
# ------------------------------------------------------------------------------------------------------------
def class_report(cnt, tms, peaks):
    """Per-class achieved bandwidth / throughput from the library's work counters and per-launch event times."""
    hbm = peaks["hbm_gbs"]
    tc = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    out = {}
    work = {"gemm": (cnt["gemm_bytes"], cnt["gemm_flops"]), "attn": (cnt["attn_bytes"], cnt["attn_flops"]),
            "head": (cnt["head_bytes"], cnt["head_flops"]), "commit": (cnt["append_bytes"], 0.0)}
    for i, name in enumerate(CLASSES):
        ms = float(tms[i])
        n = cnt["launches_" + name]
        e = {"launches": int(n), "ms_total": round(ms, 3), "us_per_launch": round(1e3 * ms / n, 3) if n else None}
        if name in work and ms > 0:
            b, f = work[name]
            e["gbs"] = round(b / (ms * 1e-3) / 1e9, 1)
            e["hbm_frac"] = round(e["gbs"] / hbm, 4)
            if f:
                e["tflops"] = round(f / (ms * 1e-3) / 1e12, 1)
                e["tensor_frac_sustained"] = round(e["tflops"] / tc, 4)
            e["bytes_per_launch"] = round(b / n) if n else None
        t = NCU_TRAFFIC.get(name)
        e["traffic"] = None
        if t and n and name in work and t.get("src") == source_hash(name):
            e["traffic"] = round(work[name][0] / n * t["captured_bytes"] / t["algorithmic_bytes"])
        out[name] = e
    return out


def run_gemm_chain(dec, w, sh, M, dev, reps=3):
    """The layer GEMMs of one denoiser pass at M rows, launched back to back over the model's own weights (every layer's
    QKV, O, gate/up + SwiGLU and down projections: the full weight set, far larger than L2), one CUDA-event pair around
    all of them.  Unlike the per-launch event pairs of the in-decode class figures this keeps the launches overlapped
    the way the decode runs them (programmatic dependent launch), so it is the kernels' own rate."""
    import torch
    import lsp_synth as S
    d, f = sh.d_model, sh.d_ffn
    qd, kvd = sh.n_heads * sh.head_dim, sh.n_kv_heads * sh.head_dim
    bf = torch.bfloat16
    a_d = S.normal((M, d), 7, 1, 0.05, bf, dev)
    a_q = S.normal((M, qd), 7, 2, 0.05, bf, dev)
    x = torch.zeros(M, d, dtype=bf, device=dev)
    o_qkv = torch.empty(M, qd + 2 * kvd, dtype=bf, device=dev)
    h_f = torch.empty(M, f, dtype=bf, device=dev)
    dec.debug_set(3, 1)                                   # queue only; no synchronisation per call

    def chain():
        for lw in dec.layer_weights:
            dec.op_linear(0, a_d, lw["w_qkv"], None, o_qkv)
            dec.op_linear(1, a_q, lw["w_o"], None, x)
            dec.op_linear(2, a_d, lw["w_gate"], lw["w_up"], h_f)
            dec.op_linear(1, h_f, lw["w_down"], None, x)

    chain()
    torch.cuda.synchronize(dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(reps):
        x.zero_()
        chain()
    ev1.record()
    torch.cuda.synchronize(dev)
    dec.debug_set(3, 0)
    dec.op_linear(0, a_d[:1], dec.layer_weights[0]["w_qkv"], None, o_qkv[:1])      # synchronising call: surfaces a device-side status
    ms = ev0.elapsed_time(ev1) / reps
    wbytes = sh.n_layers * 2.0 * ((qd + 2 * kvd) * d + d * qd + 2 * f * d + d * f)
    abytes = sh.n_layers * 2.0 * M * (d + (qd + 2 * kvd) + qd + d + d + f + f + d)
    flops = sh.n_layers * 2.0 * M * ((qd + 2 * kvd) * d + d * qd + 2 * f * d + d * f)
    return {"rows": M, "ms": ms, "launches": 4 * sh.n_layers, "gbs": (wbytes + abytes) / (ms * 1e-3) / 1e9,
            "tflops": flops / (ms * 1e-3) / 1e12}


def run_adaptive_leg(dec, wl, bm, tokens, Pl, Gl, steps, barrier):
    """The same resident decoder in the adaptive-threshold mode (Eq. 2; block size kept within [alpha N, beta N],
    alpha = 0.25, beta = 0.50, snap window 16): the active suffix then shrinks geometrically, so a decode takes
    O(log G) denoiser passes and touches O(G) rows in total instead of O(G^2)."""
    import numpy as np
    import torch
    from paper_2603_05454_b200 import SchedCfg
    B, G = wl.batch, wl.gen_len
    alpha, beta = 0.25, 0.50
    dec.set_sched(SchedCfg(mode=1, tau=wl.tau, alpha=alpha, beta=beta, delim_bitmap=bm))
    for _ in range(2):
        dec.begin(tokens, Pl, Gl)
        dec.generate()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    passes = 0
    for _ in range(steps):
        dec.begin(tokens, Pl, Gl)
        passes += dec.generate()[0]
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1)
    dec.begin(tokens, Pl, Gl)
    n, recs = dec.generate(max_recs=B * (G + 1))
    n_before = [int(np.mean([r["n_before"] for r in recs[i:i + B]])) for i in range(0, len(recs), B)]
    masked_rows = sum(r["n_before"] for r in recs)
    ratios = [n_before[i + 1] / n_before[i] for i in range(len(n_before) - 1) if n_before[i] >= 32]
    out = {"alpha": alpha, "beta": beta, "snap_window": 16, "value": B * G * steps / (ms * 1e-3), "unit": "tokens/s",
           "ms_per_decode": ms / steps, "denoiser_passes_per_decode": passes / steps,
           "masked_suffix_per_pass_mean_over_batch": n_before,
           "suffix_ratio_per_pass_while_at_least_32": [round(x, 3) for x in ratios],
           "masked_rows_total_per_sequence": masked_rows / B,
           "bounds_G_over_beta_G_over_alpha": [G / beta, G / alpha], "quadratic_G2_over_2": G * G / 2}
    dec.set_sched(SchedCfg(tau=wl.tau, delim_bitmap=bm))
    return out


def run_decode_bench(wl, dev, rank, world, peaks, steps, warmup, sampler=None, with_e2e=True, adaptive=False,
                     variants=False):
    import numpy as np
    import torch
    import lsp_synth as S
    from paper_2603_05454_b200 import LSPDecoder, SchedCfg

    sh = wl.shape
    B, P, G = wl.batch, wl.prompt_len, wl.gen_len
    w = S.make_weights(sh, 0, device=dev)
    bm = S.delimiter_bitmap(sh.vocab, *wl.delim).to(dev)
    dec = LSPDecoder(sh, w, SchedCfg(tau=wl.tau, delim_bitmap=bm), B, P + G, device=dev)
    prompt = S.make_prompt(B, P, sh, 100 + rank)           # every replica decodes its own prompts
    host_in = torch.zeros(B, P + G, dtype=torch.int32).pin_memory()
    host_in[:, :P] = prompt
    host_out = torch.zeros(B, P + G, dtype=torch.int32).pin_memory()
    tokens = torch.zeros(B, P + G, dtype=torch.int32, device=dev)
    tokens.copy_(host_in)
    Pl, Gl = [P] * B, [G] * B

    def decode_resident():
        dec.begin(tokens, Pl, Gl)
        n, _ = dec.generate()
        return n

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(warmup):
        decode_resident()
    assert int((tokens == sh.mask_id).sum()) == 0, "decode left masked positions"
    dec.reset_counters()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    if sampler:
        sampler.start()
    ev0.record()
    passes = 0
    for _ in range(steps):
        passes += decode_resident()
    ev1.record()
    barrier()
    clocks = sampler.stop() if sampler else None
    ms = ev0.elapsed_time(ev1)
    cnt = dec.counters()
    res = {"ms": ms, "passes": passes, "launches": int(cnt["launches"]), "clocks": clocks, "tokens": B * G * steps}

    if with_e2e:
        for _ in range(min(warmup, 2)):
            dec.generate_host(tokens, host_in, host_out, Pl, Gl)
        barrier()
        ev0.record()
        for _ in range(steps):
            dec.generate_host(tokens, host_in, host_out, Pl, Gl)
        ev1.record()
        barrier()
        res["e2e_ms"] = ev0.elapsed_time(ev1)
        res["h2d"] = host_in.numel() * 4
        res["d2h"] = host_out.numel() * 4
        assert int((host_out == sh.mask_id).sum()) == 0 and bool((host_out[:, :P] == host_in[:, :P]).all())

    # Variants of the loop on the same resident decoder: block lengths kept on the device (the host
    # enqueues pass k+1 before it has read L_k) and the in-place K/V layout (the append degenerates to a length bump).
    # The synchronous loop with the staged layout and the append copy (timed above) stays the contract.
    if variants:
        res["variants"] = {"sync_staged": {"ms_per_pass": ms / passes, "tokens_per_s": B * G * steps / (ms * 1e-3),
                                           "kv_append_bytes_per_token": cnt["append_bytes"] / max(1.0, cnt["tokens"])}}
        for vname, (lag, inpl) in (("lagged_staged", (1, 0)), ("sync_inplace", (0, 1)), ("lagged_inplace", (1, 1))):
            dec.set_option(4, lag)
            dec.set_option(3, inpl)
            decode_resident()
            dec.reset_counters()
            barrier()
            ev0.record()
            p2 = 0
            for _ in range(steps):
                p2 += decode_resident()
            ev1.record()
            barrier()
            assert int((tokens == sh.mask_id).sum()) == 0, "decode left masked positions"
            c2 = dec.counters()
            v_ms = ev0.elapsed_time(ev1)
            res["variants"][vname] = {"ms_per_pass": v_ms / p2, "tokens_per_s": B * G * steps / (v_ms * 1e-3),
                                      "passes_per_decode": p2 / steps,
                                      "kv_append_bytes_per_token": c2["append_bytes"] / max(1.0, c2["tokens"])}
        dec.set_option(4, 0)
        dec.set_option(3, 0)

    # second pass over the same decodes with one CUDA-event pair around every launch (per-class kernel time)
    dec.set_option(2, 1)
    decode_resident()
    dec.reset_counters()
    for _ in range(steps):
        decode_resident()
    tms = dec.last_timing()
    cnt2 = dec.counters()
    dec.set_option(2, 0)
    res["classes"] = class_report(cnt2, tms, peaks)
    # per-step profile of one more decode (rows shrink as the prefix grows)
    dec.begin(tokens, Pl, Gl)
    n, recs = dec.generate(max_recs=B * (G + 1))
    rows_ms = {}
    for i in range(0, len(recs), B):
        rows = sum(r["rows"] for r in recs[i:i + B])
        rows_ms.setdefault(rows, []).append(recs[i]["ms"])
    ks = sorted(rows_ms)
    pick = [ks[0], ks[len(ks) // 2], ks[-1]] if ks else []
    res["step_ms_by_rows"] = {str(k): round(float(np.median(rows_ms[k])), 4) for k in pick}
    live = [r["L_commit"] for r in recs if r["n_before"] > 0]
    res["l_commit_mean"] = float(np.mean(live)) if live else None
    if adaptive:
        res["adaptive"] = run_adaptive_leg(dec, wl, bm, tokens, Pl, Gl, steps, barrier)
    # the layer GEMMs alone at the decode's median row count
    all_rows = sorted(sum(r["rows"] for r in recs[i:i + B]) for i in range(0, len(recs), B))
    all_rows = [x for x in all_rows if x > 0]
    if all_rows:
        res["gemm_chain"] = run_gemm_chain(dec, w, sh, all_rows[len(all_rows) // 2], dev)
        # ... and over the decode's whole row-count distribution: a dozen row counts at its quantiles, each weighted by
        # the passes it stands for (the decode's passes run from prompt + generation rows down to two)
        qs = sorted({all_rows[min(len(all_rows) - 1, int((i + 0.5) * len(all_rows) / 12))] for i in range(12)})
        edges = [0] + [(a + b) // 2 for a, b in zip(qs[:-1], qs[1:])] + [10 ** 9]
        tot_ms = tot_bytes = tot_flops = 0.0
        per = []
        for i, M in enumerate(qs):
            wgt = sum(1 for x in all_rows if edges[i] < x <= edges[i + 1])
            g = run_gemm_chain(dec, w, sh, M, dev, reps=2)
            tot_ms += wgt * g["ms"]
            tot_bytes += wgt * g["gbs"] * g["ms"] * 1e6
            tot_flops += wgt * g["tflops"] * g["ms"] * 1e9
            per.append({"rows": M, "passes": wgt, "ms": round(g["ms"], 4), "gbs": round(g["gbs"], 1), "tflops": round(g["tflops"], 1)})
        res["gemm_chain_all"] = {"gbs": tot_bytes / (tot_ms * 1e6), "tflops": tot_flops / (tot_ms * 1e9),
                                 "ms_per_pass": tot_ms / len(all_rows), "launches": 4 * sh.n_layers, "by_rows": per}
    dec.close()
    del dec, w
    torch.cuda.empty_cache()
    return res


def run_head_bench(dev, peaks, steps, warmup):
    """cfg2: the fused LM head + confidence reduction + scan alone on [8 x 1024, 4096] hidden states."""
    import numpy as np
    import torch
    import lsp_synth as S
    from paper_2603_05454_b200 import LSPDecoder, SchedCfg
    d, V, B, L = 4096, 126464, 8, 1024
    sh = S.ModelShape(1, d, 32, 32, 128, 64, V, dtype="bf16", head_scale=6.0)
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device=dev)
    w = dict(embed=z(8, d), w_head=S.normal((V, d), 0, S.TID_HEAD, 0.02 * 6.0, torch.bfloat16, dev),
             final_norm=torch.ones(d, dtype=torch.bfloat16, device=dev),
             layers=[dict(attn_norm=z(d), w_qkv=z(3 * d, d), w_o=z(d, d), ffn_norm=z(d), w_gate=z(64, d), w_up=z(64, d),
                          w_down=z(d, 64))])
    bm = S.delimiter_bitmap(V, 1, 32).to(dev)
    dec = LSPDecoder(sh, w, SchedCfg(tau=0.9, delim_bitmap=bm), B, L, device=dev)
    hidden = S.normal((B * L, d), 0, 77, 1.0, torch.bfloat16, dev)
    host_h = hidden.cpu().pin_memory()
    off = np.arange(B + 1, dtype=np.int32) * L
    for _ in range(warmup):
        dec.head_scan(hidden, off)
    dec.reset_counters()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    ev0.record()
    for _ in range(steps):
        dec.head_scan(hidden, off)
    ev1.record()
    torch.cuda.synchronize(dev)
    ms = ev0.elapsed_time(ev1)
    cnt = dec.counters()
    ev0.record()
    for _ in range(steps):
        hidden.copy_(host_h, non_blocking=True)
        dec.head_scan(hidden, off)
        dec.scores()
    ev1.record()
    torch.cuda.synchronize(dev)
    e2e_ms = ev0.elapsed_time(ev1)
    dec.set_option(2, 1)
    dec.head_scan(hidden, off)
    dec.reset_counters()
    for _ in range(steps):
        dec.head_scan(hidden, off)
    tms = dec.last_timing()
    cnt2 = dec.counters()
    dec.close()
    return dict(ms=ms, e2e_ms=e2e_ms, launches=int(cnt["launches"]), positions=B * L * steps,
                h2d=host_h.numel() * 2, d2h=B * L * 12, classes=class_report(cnt2, tms, peaks))


def run_topology_compare(wl, dev, peaks, warmup, class_passes=24):
    """cfg5: the LSP decode next to the scattered-acceptance baseline (top-k anywhere, k = 32 per step) on the same
    kernels: denoiser calls, token flips, step latency and KV-append bytes per committed token.  One timed decode per
    topology; the warm-up decodes use a 64-token generation (they warm the same kernels; a full LSP decode of this
    workload takes minutes with a random-init model)."""
    import numpy as np
    import torch
    import lsp_synth as S
    from paper_2603_05454_b200 import LSPDecoder, SchedCfg
    sh = wl.shape
    B, P, G = wl.batch, wl.prompt_len, wl.gen_len
    w = S.make_weights(sh, 0, device=dev)
    bm = S.delimiter_bitmap(sh.vocab, *wl.delim).to(dev)
    k = int(wl.extra.get("scattered_k", 32))
    scheds = {"lsp": SchedCfg(tau=wl.tau, delim_bitmap=bm),
              "scattered_top_k": SchedCfg(mode=2, fixed_k=k, topology=1)}
    prompt = S.make_prompt(B, P, sh, 100)
    tokens = torch.zeros(B, P + G, dtype=torch.int32, device=dev)
    out = {}
    dec = LSPDecoder(sh, w, scheds["lsp"], B, P + G, device=dev)
    for name, sc in scheds.items():
        dec.set_sched(sc)
        for _ in range(warmup):
            tokens[:, :P] = prompt.to(dev)
            dec.begin(tokens, [P] * B, [64] * B)
            dec.generate()
        tokens[:, :P] = prompt.to(dev)
        dec.reset_counters()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(dev)
        ev0.record()
        dec.begin(tokens, [P] * B, [G] * B)
        n, recs = dec.generate(max_recs=B * (G + 1))
        ev1.record()
        torch.cuda.synchronize(dev)
        ms = ev0.elapsed_time(ev1)
        assert int((tokens == sh.mask_id).sum()) == 0
        cnt = dec.counters()
        # flips between 25 % and 75 % completion of each sequence (the window the paper reports)
        fl = fb = 0
        for b in range(B):
            done = 0
            for r in recs[b::B]:
                if r["n_before"] == 0:
                    continue
                if 0.25 * G <= done < 0.75 * G:
                    fl += r["flips"]; fb += r["flip_base"]
                done += r["L_commit"]
        out[name] = {"denoiser_calls": n, "tokens_per_s": B * G / (ms * 1e-3), "ms_per_denoiser_step": ms / n,
                     "decode_ms": ms, "token_flips_25_75": fl, "flip_rate_25_75": (fl / fb) if fb else None,
                     "kv_append_bytes_per_committed_token": cnt["append_bytes"] / (B * G),
                     "gpu_launches": int(cnt["launches"]),
                     "rows_first_last": [sum(r["rows"] for r in recs[:B]), sum(r["rows"] for r in recs[-B:])]}
    # per-class kernel times (one CUDA-event pair per launch) over the first passes of one more LSP decode
    dec.set_sched(scheds["lsp"])
    tokens[:, :P] = prompt.to(dev)
    dec.begin(tokens, [P] * B, [G] * B)
    dec.set_option(2, 1)
    dec.reset_counters()
    n_cls = 0
    while n_cls < class_passes and dec.active()[1] > 0:
        dec.denoise_step()
        dec.commit()
        n_cls += 1
    tms = dec.last_timing()
    cnt = dec.counters()
    dec.set_option(2, 0)
    classes = class_report(cnt, tms, peaks)
    dec.close()
    del dec, w
    torch.cuda.empty_cache()
    return out, k, classes, n_cls


def head_line(dev, peaks, peak_kind, steps, warmup, sampler=None):
    """cfg2 as a bench line (also used as an entry under 'also')."""
    if sampler:
        sampler.start()
    r = run_head_bench(dev, peaks, steps, warmup)
    clocks = sampler.stop() if sampler else None
    head = r["classes"]["head"]
    return {"metric": "scored_positions_per_s", "value": r["positions"] / (r["ms"] * 1e-3), "unit": "positions/s",
            "n_gpus": 1, "steps": steps, "warmup": warmup, "ms_per_step": r["ms"] / steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "cfg2: fused LM head + confidence + LSP scan, hidden [8,1024,4096], vocab 126464",
                       "l2": "inputs_exceed_l2 (1.04 GB head weight)"},
            "roofline": {"bound": "tensor", "achieved": head.get("tflops"), "peak": peaks["bf16_tflops"],
                         "unit": "TFLOP/s", "frac": (head.get("tflops") or 0) / peaks["bf16_tflops"],
                         "traffic": head.get("traffic"), "peak_kind": "burst, of " + peak_kind,
                         "kernel": "k_gemm_stream<256,.,.,EpiHead> (LM head with the top-2 / log-sum-exp reduction in its epilogue)"},
            "e2e": {"value": r["positions"] / (r["e2e_ms"] * 1e-3), "unit": "positions/s",
                    "h2d_bytes_per_step": r["h2d"], "d2h_bytes_per_step": r["d2h"]},
            "gpu_launches": r["launches"], "classes": r["classes"], "clocks": clocks}


def topology_line(wl, dev, peaks, peak_kind, warmup, sampler=None):
    """cfg5 as a bench line (also used as an entry under 'also'): one timed decode per topology."""
    if sampler:
        sampler.start()
    cmp_, k, classes, n_cls = run_topology_compare(wl, dev, peaks, warmup)
    clocks = sampler.stop() if sampler else None
    lsp = cmp_["lsp"]
    g = classes["gemm"]
    tc = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    return {"metric": "committed_tokens_per_s", "value": lsp["tokens_per_s"], "unit": "tokens/s", "n_gpus": 1, "steps": 1,
            "warmup": warmup, "ms_per_step": lsp["decode_ms"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"cfg5: LLaDA-8B shape, batch {wl.batch}, prompt {wl.prompt_len} + {wl.gen_len} masked, "
                                   f"LSP (tau {wl.tau}) next to scattered top-{k} acceptance, random init",
                       "warmup_decodes": "64-token generations", "head_scale": wl.shape.head_scale,
                       "l2": "inputs_exceed_l2"},
            "roofline": {"bound": "tensor", "achieved": g.get("tflops"), "peak": tc, "unit": "TFLOP/s",
                         "frac": g.get("tensor_frac_sustained"), "traffic": g.get("traffic"),
                         "peak_kind": "sustained, of " + peak_kind,
                         "kernel": "k_gemm_stream (layer GEMMs; 17 k to 33 k rows per pass: tensor-bound)",
                         "timed": f"per-launch CUDA events over the first {n_cls} passes of one more LSP decode"},
            "classes": classes, "topologies": cmp_, "gpu_launches": lsp["gpu_launches"], "clocks": clocks}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="own", choices=["own", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=["cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--also", default="cfg4,cfg2,cfg5",
                    help="further workloads reported under 'also' at N=1, comma-separated ('none' to skip)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.warmup < 3:
        args.warmup = 3

    import torch
    import lsp_synth as S
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=dev)
    if world > 1 and args.workload in ("cfg2", "cfg5"):
        # single-GPU measurements (the head alone; the topology comparison): rank 0 runs them, the others leave
        torch.distributed.destroy_process_group()
        if rank != 0:
            return 0
        world = 1
    peaks, peak_kind = load_peaks()
    uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    sampler = ClockSampler(uuid)

    if args.workload == "cfg2":
        print(json.dumps(head_line(dev, peaks, peak_kind, args.steps, args.warmup, sampler)))
        return 0

    wl = S.config(args.workload)
    if args.workload == "cfg5":
        print(json.dumps(topology_line(wl, dev, peaks, peak_kind, args.warmup, sampler)))
        return 0
    r = run_decode_bench(wl, dev, rank, world, peaks, args.steps, args.warmup, sampler, adaptive=(world == 1),
                         variants=(world == 1))
    (ms_max, e2e_max), tokens_total = reduce_replicas([r["ms"], r.get("e2e_ms", 0.0)], r["tokens"], world, dev)
    value = tokens_total / (ms_max * 1e-3)
    gemm = r["classes"]["gemm"]
    line = {"metric": "committed_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_max / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{wl.name}: LSP decode, {wl.shape.n_layers} layers d={wl.shape.d_model} "
                                   f"heads {wl.shape.n_heads}/{wl.shape.n_kv_heads}x{wl.shape.head_dim} ffn "
                                   f"{wl.shape.d_ffn} vocab {wl.shape.vocab}, random init",
                       "batch": wl.batch, "prompt_len": wl.prompt_len, "gen_len": wl.gen_len, "tau": wl.tau,
                       "delimiters": list(wl.delim), "head_scale": wl.shape.head_scale, "snap_window": 16,
                       "step": "one full decode (all denoiser passes)", "parallelism": f"replicas x{world}",
                       "l2": "inputs_exceed_l2 (every pass streams the full weight set, far larger than the 126 MB L2)"},
            "denoiser_passes_per_decode": r["passes"] / args.steps,
            "ms_per_denoiser_step": ms_max / r["passes"],
            "ms_per_denoiser_step_by_rows": r["step_ms_by_rows"],
            "tokens_per_pass": r["l_commit_mean"],
            "roofline": {"bound": "hbm", "achieved": gemm.get("gbs"), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gemm.get("hbm_frac"), "traffic": gemm.get("traffic"),
                         "kernel": "k_gemm_stream (layer projections and FFN; all but the first pass have at most 257 rows: weight-streaming regime)",
                         "peak_kind": "of " + peak_kind,
                         "timed": "per-launch CUDA events, second pass over the same K decodes (each event pair adds "
                                  "about 5 us and breaks the overlap between consecutive launches: a lower bound)",
                         "back_to_back": None},
            "classes": r["classes"],
            "e2e": {"value": tokens_total / (e2e_max * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": r["h2d"],
                    "d2h_bytes_per_step": r["d2h"]},
            "gpu_launches": r["launches"], "clocks": r["clocks"]}
    if r.get("adaptive"):
        line["adaptive_tau"] = r["adaptive"]
    if r.get("variants"):
        line["loop_variants"] = r["variants"]
    if r.get("gemm_chain_all"):
        ga = r["gemm_chain_all"]
        line["roofline"]["over_row_distribution"] = {
            "what": "the same kernels back to back (one CUDA-event pair around all layers' GEMMs, no per-launch events) at "
                    "twelve row counts spread over the decode's passes, weighted by the passes each stands for",
            "achieved": round(ga["gbs"], 1), "unit": "GB/s", "frac": round(ga["gbs"] / peaks["hbm_gbs"], 4),
            "tflops": round(ga["tflops"], 1), "gemm_ms_per_pass": round(ga["ms_per_pass"], 4), "by_rows": ga["by_rows"]}
    if r.get("gemm_chain"):
        gc = r["gemm_chain"]
        line["roofline"]["back_to_back"] = {
            "what": "the same kernels: all layers' QKV, O, gate/up and down GEMMs at the decode's median row count, "
                    "launched back to back over the model's weights, one CUDA-event pair around all of them",
            "rows": gc["rows"], "launches": gc["launches"], "ms": round(gc["ms"], 4), "achieved": round(gc["gbs"], 1),
            "unit": "GB/s", "frac": round(gc["gbs"] / peaks["hbm_gbs"], 4), "tflops": round(gc["tflops"], 1)}

    also = [a for a in args.also.split(",") if a and a != "none" and a != args.workload] if (rank == 0 and world == 1) else []
    line["also"] = []
    for name in also:
        if name == "cfg2":
            line["also"].append(head_line(dev, peaks, peak_kind, args.steps, args.warmup))
            continue
        if name == "cfg5":
            line["also"].append(topology_line(S.config("cfg5"), dev, peaks, peak_kind, args.warmup))
            continue
        wl2 = S.config(name)
        k2 = max(1, min(2, args.steps))
        r2 = run_decode_bench(wl2, dev, 0, 1, peaks, k2, 3, None, with_e2e=False)
        g2 = r2["classes"]["gemm"]
        line["also"].append({"workload": wl2.name, "batch": wl2.batch, "prompt_len": wl2.prompt_len, "gen_len": wl2.gen_len,
                         "head_scale": wl2.shape.head_scale, "tau": wl2.tau, "steps": k2,
                         "value": r2["tokens"] / (r2["ms"] * 1e-3), "unit": "tokens/s",
                         "denoiser_passes_per_decode": r2["passes"] / k2,
                         "ms_per_denoiser_step": r2["ms"] / r2["passes"],
                         "ms_per_denoiser_step_by_rows": r2["step_ms_by_rows"],
                         "roofline": {"bound": "tensor", "achieved": g2.get("tflops"),
                                      "peak": peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]),
                                      "unit": "TFLOP/s", "frac": g2.get("tensor_frac_sustained"),
                                      "traffic": g2.get("traffic"), "peak_kind": "sustained, of " + peak_kind,
                                      "back_to_back": ({"rows": r2["gemm_chain"]["rows"], "ms": round(r2["gemm_chain"]["ms"], 4),
                                                        "achieved": round(r2["gemm_chain"]["tflops"], 1), "unit": "TFLOP/s",
                                                        "frac": round(r2["gemm_chain"]["tflops"] /
                                                                      peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]), 4)}
                                                       if r2.get("gemm_chain") else None)},
                         "classes": r2["classes"]})
    if not line["also"]:
        del line["also"]

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sh, om, prompt = oracle_sample_setup(wl, dev)
        dt, tok = oracle_sample_run(wl, om, prompt)
        scale = wl.shape.n_layers / sh.n_layers
        line["cpu_baseline"] = {"value": tok / (dt * scale), "unit": "tokens/s", "cores": blas_threads(),
                                "kind": "oracle", "sample": oracle_sample_text(wl), "seconds": round(dt, 3)}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
