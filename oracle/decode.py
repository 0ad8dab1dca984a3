"""Oracle: the LSP decode loop (Algorithm 1) for one sequence, plus the prefix-cache plumbing.
TEST INFRASTRUCTURE, not a product path.

Reading of the cache append ("one-step lag"; the paper is ambiguous): the pass that predicts a
block sees [MASK] inputs at those positions, so the K/V it computes there do not encode the
committed tokens.  The block committed at step k-1 is therefore *pending* at step k: it is fed
as real tokens in front of the masked suffix, and the K/V computed for it in that pass are
what step k's AppendToCache adds.  The prompt is the pending block of step 0, so CacheInit is
step 0's append.  Cache rows are written once and never change.

A "no-cache" mode (every pass recomputes all positions with committed tokens as real inputs)
exists only to check the plumbing: pass 0 is identical, layer-0 K/V rows always agree, and a
1-layer model gives the same decode in both modes.

Pins: loop invariants (prefix never rewritten, N strictly decreasing, terminates fully
committed, boundaries only at a delimiter / run end / L_min), tau = 0 -> one step, tau = inf
-> G steps, fixed-k -> ceil(G/k) steps (Table 2), the cached/no-cache checks above.
Trajectories of a trained model (Tables 1-3) are "parity unpinned": they need weights and
datasets that are not available.
"""
import numpy as np

from . import scan as _scan
from .scores import scores_from_logits


def make_is_delim(lo, hi):
    return lambda t: lo <= t <= hi


def decode(model, prompt, gen_len, is_delim, policy, score="pmax", use_cache=True,
           exclude_mask=True, max_steps=None, on_step=None):
    """Runs Algorithm 1.  prompt: 1-D int array.  policy: kwargs of oracle.scan.lsp_scan.
    Returns (tokens [P+G], records list).  Each record holds the step's N, rows, L_run,
    L_commit, tau_used, flags and the per-position yhat / p_max / delta arrays."""
    s = model.s
    P, G = len(prompt), int(gen_len)
    tokens = np.full(P + G, s.mask_id, dtype=np.int64)
    tokens[:P] = prompt
    cache_k, cache_v = model.empty_cache()
    F, Fp, pend, N = 0, P, P, G        # cache rows, token boundary, pending block, active length
    recs = []
    step = 0
    while N > 0:                                                        # Alg. 1: loop      
        if use_cache:
            ids = np.concatenate([tokens[F:F + pend], np.full(N, s.mask_id)])
            pos = np.arange(F, F + pend + N)
            head_rows = np.arange(pend, pend + N)
            ck, cv = cache_k, cache_v
        else:
            ids = np.concatenate([tokens[:Fp], np.full(N, s.mask_id)])
            pos = np.arange(0, Fp + N)
            head_rows = np.arange(Fp, Fp + N)
            ck, cv = model.empty_cache()
        logits, k_new, v_new = model.forward(ids, pos, ck, cv, head_rows)   # pass  
        yhat, pmax, delta = scores_from_logits(logits, s.mask_id if exclude_mask else -1)  # scores
        sc = pmax if score == "pmax" else delta
        r = _scan.lsp_scan(sc, yhat, is_delim, margin=delta, **policy)      # tau, snap
        L = r["L_commit"]
        rec = dict(step=step, n_before=N, rows=len(ids), F=F, Fp=Fp, pend=pend, yhat=yhat,
                   pmax=pmax, delta=delta, **r)
        if on_step is not None:
            on_step(rec, logits, k_new, v_new)
        if use_cache:                                                   # append (lagged) 
            for l in range(s.n_layers):
                cache_k[l] = np.concatenate([cache_k[l], k_new[l][:pend]], axis=0)
                cache_v[l] = np.concatenate([cache_v[l], v_new[l][:pend]], axis=0)
            F += pend
        tokens[Fp:Fp + L] = yhat[:L]                                    # commit
        Fp += L
        pend = L
        N -= L
        recs.append(rec)
        step += 1
        if max_steps is not None and step >= max_steps:
            break
    return tokens, recs, (cache_k, cache_v)
