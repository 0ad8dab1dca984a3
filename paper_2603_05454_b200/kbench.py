"""Kernel micro-benchmarks through the C ABI:  python -m paper_2603_05454_b200.kbench <what> [options]

  gemm   one linear layer  out = A W^T  (or the residual / SwiGLU epilogues) at a given M, N, K; the weights are
         read from a ring of copies larger than the L2 cache so that every launch streams them from HBM
  layer  the four GEMMs of one transformer layer (fused QKV, O, gate/up + SwiGLU, down) of a model shape given by
         --d --heads --kv-heads --ffn (default: a shape the tile heuristics were not fitted on: 5120, 40/8, 13824)
  head   the fused LM head + confidence reduction + scan on M hidden rows
  decode per-class kernel times of a full decode of a named workload (same figures bench.py reports)

Times are CUDA-event times around `reps` back-to-back launches after warm-up; GB/s counts every operand and the
result once, TFLOP/s counts 2 M N K (x2 for the dual-weight SwiGLU epilogue).
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

import lsp_synth as S
from . import LSPDecoder, SchedCfg

DEV = "cuda:0"


def _tiny_decoder(max_batch=1, max_len=8):
    sh = S.ModelShape(1, 64, 1, 1, 64, 64, 128, dtype="bf16")
    return LSPDecoder(sh, S.make_weights(sh, 0, device=DEV), SchedCfg(), max_batch, max_len, device=DEV)


def bench_gemm(M, N, K, op=0, reps=50, copies=0, warm=5, opts=()):
    dec = _tiny_decoder()
    for k, v in opts:
        (dec.set_option if k in (0, 1, 2) else dec.debug_set)(k, v)
    per = N * K * 2 * (2 if op == 2 else 1)
    if copies <= 0:
        copies = max(2, int(np.ceil(400e6 / per)))           # ring of weights > 3x the 126 MB L2
    A = S.normal((M, K), 0, 1, 1.0, torch.bfloat16, DEV)
    W = S.normal((copies * N, K), 0, 2, 0.02, torch.bfloat16, DEV)
    W2 = S.normal((copies * N, K), 0, 3, 0.02, torch.bfloat16, DEV) if op == 2 else None
    out = torch.zeros(M, N, dtype=torch.bfloat16, device=DEV)
    dec.debug_set(3, 1)
    dec.debug_set(5, copies)
    dec.debug_set(4, warm)
    dec.op_linear(op, A, W[:N], W2[:N] if W2 is not None else None, out)
    torch.cuda.synchronize()
    dec.debug_set(4, reps)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    dec.op_linear(op, A, W[:N], W2[:N] if W2 is not None else None, out)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / reps
    dec.debug_set(3, 0)
    dec.debug_set(4, 1)
    dec.op_linear(0, A[:1], W[:N], None, out[:1])          # synchronising call: surfaces a device-side status
    dec.close()
    nw = 2 if op == 2 else 1
    bytes_ = (nw * N * K + M * K + M * N) * 2
    flops = 2.0 * M * N * K * nw
    return dict(M=M, N=N, K=K, op=op, us=round(us, 2), gbs=round(bytes_ / us / 1e3, 1),
                tflops=round(flops / us / 1e6, 1), copies=copies)


def bench_head(M, V, d, reps=10, head_scale=6.0):
    sh = S.ModelShape(1, d, max(1, d // 128), max(1, d // 128), 128, 64, V, dtype="bf16", head_scale=head_scale)
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device=DEV)
    w = dict(embed=z(8, d), w_head=S.normal((V, d), 0, S.TID_HEAD, 0.02 * head_scale, torch.bfloat16, DEV),
             final_norm=torch.ones(d, dtype=torch.bfloat16, device=DEV),
             layers=[dict(attn_norm=z(d), w_qkv=z(3 * d, d), w_o=z(d, d), ffn_norm=z(d), w_gate=z(64, d), w_up=z(64, d),
                          w_down=z(d, 64))])
    dec = LSPDecoder(sh, w, SchedCfg(tau=0.9, delim_bitmap=S.delimiter_bitmap(V, 1, 32).to(DEV)), 1, max(2, M), device=DEV)
    hidden = S.normal((M, d), 0, 77, 1.0, torch.bfloat16, DEV)
    off = np.array([0, M], dtype=np.int32)
    for _ in range(3):
        dec.head_scan(hidden, off)
    dec.set_option(2, 1)
    dec.reset_counters()
    for _ in range(reps):
        dec.head_scan(hidden, off)
    t = dec.last_timing()
    c = dec.counters()
    dec.close()
    us = float(t[3]) * 1e3 / reps
    return dict(M=M, V=V, d=d, us=round(us, 2), us_merge_scan=round(float(t[4]) * 1e3 / reps, 2),
                gbs=round(c["head_bytes"] / reps / us / 1e3, 1), tflops=round(c["head_flops"] / reps / us / 1e6, 1))


def _fast_weights(sh):
    """Same shapes and scales as lsp_synth.make_weights, filled by torch's generator in a few launches (profiling
    aid: a run under a profiler pays for every launch, the seeded generator takes thousands)."""
    g = torch.Generator(device=DEV)
    g.manual_seed(0)
    rnd = lambda *s, std=sh.w_std: torch.empty(*s, dtype=torch.bfloat16, device=DEV).normal_(0.0, std, generator=g)
    d, hq, hkv, dh, f, v = sh.d_model, sh.n_heads, sh.n_kv_heads, sh.head_dim, sh.d_ffn, sh.vocab
    one = lambda: torch.ones(d, dtype=torch.bfloat16, device=DEV)
    return dict(embed=rnd(v, d), w_head=rnd(v, d, std=sh.w_std * sh.head_scale), final_norm=one(),
                layers=[dict(w_qkv=rnd((hq + 2 * hkv) * dh, d), w_o=rnd(d, hq * dh), w_gate=rnd(f, d), w_up=rnd(f, d),
                             w_down=rnd(d, f), attn_norm=one(), ffn_norm=one()) for _ in range(sh.n_layers)])


def bench_decode(name, decodes=1, layers=0, max_passes=0, fast_init=False, opts=(), batch=0, prompt=0, gen=0):
    """Per-class kernel times of a decode.  layers > 0 cuts the model to its first layers, max_passes > 0 stops each
    decode after that many denoiser passes (both are profiling aids: fewer launches, same kernels and row counts)."""
    wl = S.config(name)
    sh = wl.shape
    if layers > 0:
        sh.n_layers = layers
    B, P, G = batch or wl.batch, prompt or wl.prompt_len, gen or wl.gen_len
    w = _fast_weights(sh) if fast_init else S.make_weights(sh, 0, device=DEV)
    dec = LSPDecoder(sh, w, SchedCfg(tau=wl.tau, delim_bitmap=S.delimiter_bitmap(sh.vocab, *wl.delim).to(DEV)), B, P + G,
                     device=DEV)
    for k, v in opts:
        (dec.set_option if k in (0, 1, 2) else dec.debug_set)(k, v)
    tokens = torch.zeros(B, P + G, dtype=torch.int32, device=DEV)
    tokens[:, :P] = S.make_prompt(B, P, sh, 100).to(DEV)

    def run():
        dec.begin(tokens, [P] * B, [G] * B)
        if max_passes <= 0:
            return dec.generate()[0]
        n = 0
        while n < max_passes and dec.active()[1] > 0:
            dec.denoise_step()
            dec.commit()
            n += 1
        return n

    run()
    dec.reset_counters()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    n_plain = run()
    e1.record()
    torch.cuda.synchronize()
    plain_ms = e0.elapsed_time(e1)
    tp = dec.last_timing()          # plain run: device time of the passes and host time spent queueing them
    dec.set_option(2, 1)
    dec.reset_counters()
    n = 0
    for _ in range(decodes):
        n += run()
    t = dec.last_timing()
    c = dec.counters()
    dec.close()
    names = ("misc", "gemm", "attn", "head", "scan", "commit")
    return dict(workload=name, passes=n, ms_per_pass_plain=round(plain_ms / n_plain, 4),
                ms_per_pass={k: round(float(t[i]) / n, 4) for i, k in enumerate(names)},
                ms_per_pass_total=round(float(t[6]) / n, 4), ms_per_pass_plain_device=round(float(tp[6]) / n_plain, 4),
                host_queue_ms_per_pass_plain=round(float(tp[7]) / n_plain, 4), launches_per_pass=c["launches"] / n,
                gemm_gbs=round(c["gemm_bytes"] / (float(t[1]) * 1e6), 1),
                gemm_tflops=round(c["gemm_flops"] / (float(t[1]) * 1e9), 1),
                attn_gbs=round(c["attn_bytes"] / (float(t[2]) * 1e6), 1),
                head_gbs=round(c["head_bytes"] / (float(t[3]) * 1e6), 1),
                attn_tflops=round(c["attn_flops"] / (float(t[2]) * 1e9), 1),
                append_gbs=round(c["append_bytes"] / max(1e-9, float(t[5]) * 1e6), 1))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["gemm", "layer", "head", "decode"])
    ap.add_argument("--M", type=int, nargs="+", default=[128])
    ap.add_argument("--N", type=int, default=4096)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--V", type=int, default=126464)
    ap.add_argument("--heads", type=int, default=40)
    ap.add_argument("--kv-heads", type=int, default=8)
    ap.add_argument("--ffn", type=int, default=13824)
    ap.add_argument("--d", type=int, default=4096)
    ap.add_argument("--op", type=int, default=0)
    ap.add_argument("--reps", type=int, default=50)
    ap.add_argument("--copies", type=int, default=0)
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--layers", type=int, default=0)
    ap.add_argument("--max-passes", type=int, default=0)
    ap.add_argument("--fast-init", action="store_true")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--prompt", type=int, default=0)
    ap.add_argument("--gen", type=int, default=0)
    ap.add_argument("--opt", type=int, nargs=2, action="append", default=[], help="lsp_set_option key value")
    a = ap.parse_args()
    if a.what == "gemm":
        for m in a.M:
            print(json.dumps(bench_gemm(m, a.N, a.K, a.op, a.reps, a.copies, opts=a.opt)), flush=True)
    elif a.what == "layer":
        d = a.d if a.d != 4096 else 5120
        qd, kvd = a.heads * 128, a.kv_heads * 128
        for m in a.M:
            for name, (n, k, op) in (("qkv", (qd + 2 * kvd, d, 0)), ("o", (d, qd, 1)), ("gate_up", (a.ffn, d, 2)),
                                     ("down", (d, a.ffn, 1))):
                print(json.dumps(dict(gemm=name, **bench_gemm(m, n, k, op, a.reps, a.copies, opts=a.opt))), flush=True)
    elif a.what == "head":
        for m in a.M:
            print(json.dumps(bench_head(m, a.V, a.d, a.reps)), flush=True)
    else:
        print(json.dumps(bench_decode(a.workload, 1, a.layers, a.max_passes, a.fast_init, a.opt, a.batch, a.prompt, a.gen)), flush=True)


if __name__ == "__main__":
    main()
