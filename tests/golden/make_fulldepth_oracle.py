#!/usr/bin/env python
"""Writes tests/golden/fulldepth_<workload>.txt: the CPU oracle's first decode passes of the full-depth benchmark
workloads (all layers, full vocabulary), one sequence, for the policies the GPU parity test teacher-forces.

    python tests/golden/make_fulldepth_oracle.py [cfg3 cfg4] [--out DIR]

Calls only oracle/ and the shared seeded input generator (lsp_synth); nothing of the CUDA library is imported.  If a
CUDA device is present the generator produces the weights there (same bits as on the CPU, much faster) and hands them
over one layer at a time; all of the oracle's arithmetic runs on the host in float64.

Every stored block is one (policy, pass): the step's N, rows, L', L, flags, tau, then yhat, p_max and delta of every
masked position.  The block "exact" is pass 0 once more with NO activation rounding (the same bf16 weights, float64
throughout): the distance between it and the bf16-rounding oracle is what rounding to bf16 at the declared points does
to the scores at this depth, i.e. the yardstick for how far two correct bf16 pipelines may sit from each other.
The header carries a hash of the oracle's and the generator's sources; the test recomputes the records itself when
that hash no longer matches.
"""
import argparse
import hashlib
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

# policy name -> (kwargs of oracle.scan.lsp_scan besides tau, passes computed); tau comes from the workload
POLICIES = {
    "cfg3": {"bench": (dict(mode=0), 2), "fixed_k": (dict(mode=2, fixed_k=120), 3)},
    "cfg4": {"bench": (dict(mode=0), 2), "fixed_k": (dict(mode=2, fixed_k=230), 3)},
}
PROMPT_SEED = 100          # the benchmark's prompts (bench.py draws rank r's from seed 100 + r)
FLAG_TOL = 2e-2            # near-threshold band recorded in the flags
TIE_TOL = 0.5              # near-tie band (logit units) recorded in the flags


def source_hash():
    h = hashlib.sha1()
    for f in ("oracle/scores.py", "oracle/scan.py", "oracle/dlm.py", "oracle/decode.py", "lsp_synth.py",
              "tests/golden/make_fulldepth_oracle.py"):
        h.update(open(os.path.join(ROOT, f), "rb").read())
    return h.hexdigest()[:16]


class _Layers:
    """weights["layers"] for the oracle's one-layer-at-a-time mode: layer l is generated when asked for."""

    def __init__(self, shape, seed, device):
        self.shape, self.seed, self.device = shape, seed, device

    def __getitem__(self, l):
        import lsp_synth as S
        return {k: v.cpu() for k, v in S.make_layer(self.shape, self.seed, l, self.device).items()}


def compute(name, log=print):
    """Returns {policy: [record per pass]} for sequence 0 of workload `name`."""
    import torch
    import lsp_synth as S
    from oracle import dlm
    from oracle.decode import decode, make_is_delim
    wl = S.config(name)
    sh = wl.shape
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    w = {"embed": S.normal((sh.vocab, sh.d_model), 0, S.TID_EMBED, sh.w_std, torch.bfloat16, dev).cpu(),
         "w_head": S.normal((sh.vocab, sh.d_model), 0, S.TID_HEAD, sh.w_std * sh.head_scale, torch.bfloat16, dev).cpu(),
         "final_norm": torch.ones(sh.d_model, dtype=torch.bfloat16), "layers": _Layers(sh, 0, dev)}
    om = dlm.OracleDLM(sh, w, one_layer_at_a_time=True)
    # pass 0 does not depend on the policy: the second policy's identical call is answered from this memo
    memo, plain_forward = {}, om.forward

    def forward(ids, pos, ck, cv, head_rows):
        key = (np.asarray(ids).tobytes(), np.asarray(pos).tobytes(), ck[0].shape[0], np.asarray(head_rows).tobytes())
        if ck[0].shape[0] != 0:
            return plain_forward(ids, pos, ck, cv, head_rows)
        if key not in memo:
            memo[key] = plain_forward(ids, pos, ck, cv, head_rows)
        return memo[key]

    om.forward = forward
    prompt = S.make_prompt(wl.batch, wl.prompt_len, sh, PROMPT_SEED)[0].numpy()
    out = {}
    for pname, (pol, n_pass) in POLICIES[name].items():
        t0 = time.time()
        policy = dict(pol, tau=float(np.float32(wl.tau)), W=16, l_min=1, flag_tol=float(np.float32(FLAG_TOL)),
                      tie_tol=float(np.float32(TIE_TOL)))
        _, recs, _ = decode(om, prompt, wl.gen_len, make_is_delim(*wl.delim), policy, max_steps=n_pass)
        out[pname] = recs
        log(f"{name}/{pname}: {len(recs)} passes in {time.time() - t0:.0f} s; rows {[r['rows'] for r in recs]}, "
            f"L {[r['L_commit'] for r in recs]}")
    # pass 0 without any activation rounding (policy-independent)
    import dataclasses
    from oracle.scores import scores_from_logits
    t0 = time.time()
    om_x = dlm.OracleDLM(dataclasses.replace(sh, dtype="fp32"), w, one_layer_at_a_time=True)
    P, G = wl.prompt_len, wl.gen_len
    ids = np.concatenate([prompt, np.full(G, sh.mask_id)])
    ck, cv = om_x.empty_cache()
    logits, _, _ = om_x.forward(ids, np.arange(P + G), ck, cv, np.arange(P, P + G))
    yhat, pmax, delta = scores_from_logits(logits, sh.mask_id)
    out["exact"] = [dict(step=0, n_before=G, rows=P + G, L_run=0, L_commit=0, flags=0, tau_used=float("nan"), yhat=yhat,
                         pmax=pmax, delta=delta)]
    log(f"{name}/exact: pass 0 without rounding in {time.time() - t0:.0f} s")
    return out


def write(name, recs_by_policy, path):
    with open(path, "w") as f:
        f.write(f"# CPU oracle, workload {name}, sequence 0, prompt seed {PROMPT_SEED}: first passes per policy.\n")
        f.write("# Written by tests/golden/make_fulldepth_oracle.py (calls only oracle/ and lsp_synth).\n")
        f.write(f"# hash {source_hash()}\n")
        for pname, recs in recs_by_policy.items():
            for r in recs:
                f.write(f"pass {pname} {r['step']} N {r['n_before']} rows {r['rows']} L_run {r['L_run']} L_commit "
                        f"{r['L_commit']} flags {r['flags']} tau {float(r['tau_used'])!r}\n")
                f.write("yhat " + " ".join(str(int(x)) for x in r["yhat"]) + "\n")
                f.write("pmax " + " ".join(repr(float(x)) for x in r["pmax"]) + "\n")
                f.write("delta " + " ".join(repr(float(x)) for x in r["delta"]) + "\n")


def read(path):
    """Returns (hash, {policy: [record]}) or (None, {}) when the file is missing."""
    if not os.path.exists(path):
        return None, {}
    h, out, cur = None, {}, None
    for line in open(path):
        t = line.split()
        if not t:
            continue
        if t[0] == "#":
            if len(t) >= 3 and t[1] == "hash":
                h = t[2]
            continue
        if t[0] == "pass":
            cur = dict(step=int(t[2]), n_before=int(t[4]), rows=int(t[6]), L_run=int(t[8]), L_commit=int(t[10]),
                       flags=int(t[12]), tau_used=float(t[14]))
            out.setdefault(t[1], []).append(cur)
        elif t[0] == "yhat":
            cur["yhat"] = np.array([int(x) for x in t[1:]], dtype=np.int32)
        else:
            cur[t[0]] = np.array([float(x) for x in t[1:]], dtype=np.float64)
    return h, out


def load_or_compute(name, log=print):
    """The stored records when they were written by the current oracle sources, else a fresh computation."""
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), f"fulldepth_{name}.txt")
    h, recs = read(path)
    if h == source_hash():
        return recs, "stored"
    log(f"{path}: written by other oracle sources (or missing); recomputing on the host, this takes minutes")
    return compute(name, log), "recomputed"


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("names", nargs="*", default=["cfg3", "cfg4"])
    ap.add_argument("--out", default=os.path.dirname(os.path.abspath(__file__)))
    a = ap.parse_args()
    os.makedirs(a.out, exist_ok=True)
    for n in a.names:
        write(n, compute(n), os.path.join(a.out, f"fulldepth_{n}.txt"))
