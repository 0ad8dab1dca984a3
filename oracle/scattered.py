"""Oracle: the scattered-acceptance baselines the paper compares LSP with, and the token flip count (Sec. 4:
"Full" decoding = standard confidence-based iterative refinement; the "Scattered-Margin" ablation; Fig. 3's flip
rate).  TEST INFRASTRUCTURE, not a product path.

Scattered acceptance: every step runs the denoiser over the whole generation region (committed positions feed their
token, the others [MASK]) and accepts the most confident masked positions wherever they are.  How many:
  * "top-k": a fixed number k per step (the benchmark's k = 32);
  * "Scattered-Margin": as many as LSP's block sizing would commit (L from the scan over the masked positions in
    order), but taken from anywhere.
The prompt's K/V are computed in the first pass and reused (prefix cache); the generation region is recomputed every
step, so nothing is appended after the first pass.

Readings: ties in confidence go to the lower position (the paper is silent); the flip count of a step is the number
of positions that are masked before both this step and the previous one and whose argmax differs between the two.

Pins: every step accepts exactly min(k, masked) positions, so a decode takes ceil(G / k) steps; accepted positions
are the k best by brute-force sort; k >= G gives one step; a committed position is never rewritten; with k = 1 the
flip base shrinks by one per step; accepting from anywhere with the count of a left-aligned run never commits fewer
tokens per step than LSP itself.
"""
import numpy as np

from . import scan as _scan
from .scores import scores_from_logits


def top_count(score, count):
    """Indices (ascending) of the `count` largest scores; ties go to the lower index."""
    order = sorted(range(len(score)), key=lambda i: (-float(score[i]), i))
    return sorted(order[:count])


def decode_scattered(model, prompt, gen_len, k=32, score="pmax", exclude_mask=True, lsp_policy=None, is_delim=None,
                     max_steps=None):
    """lsp_policy None: top-k with fixed k.  Otherwise kwargs of oracle.scan.lsp_scan: the count is that scan's
    L_commit over the masked positions in order (Scattered-Margin)."""
    s = model.s
    P, G = len(prompt), int(gen_len)
    tokens = np.full(P + G, s.mask_id, dtype=np.int64)
    tokens[:P] = prompt
    cache_k, cache_v = model.empty_cache()
    recs = []
    prev = {}                                     # position -> argmax at the previous step (masked positions only)
    step = 0
    while (tokens[P:] == s.mask_id).any():
        masked = np.nonzero(tokens[P:] == s.mask_id)[0]          # offsets inside the generation region
        if step == 0:
            ids, pos = tokens.copy(), np.arange(P + G)
            head_rows = P + masked
            ck, cv = model.empty_cache()
        else:
            ids, pos = tokens[P:].copy(), np.arange(P, P + G)
            head_rows = masked
            ck, cv = cache_k, cache_v
        logits, k_new, v_new = model.forward(ids, pos, ck, cv, head_rows)
        yhat, pmax, delta = scores_from_logits(logits, s.mask_id if exclude_mask else -1)
        sc = pmax if score == "pmax" else delta
        if lsp_policy is None:
            count, L_run = min(int(k), len(masked)), None
        else:
            r = _scan.lsp_scan(sc, yhat, is_delim or (lambda t: False), margin=delta, **lsp_policy)
            count, L_run = r["L_commit"], r["L_run"]
        sel = top_count(sc, count)
        flips = sum(1 for i, m in enumerate(masked) if int(m) in prev and prev[int(m)] != int(yhat[i]))
        base = sum(1 for m in masked if int(m) in prev)
        prev = {int(m): int(yhat[i]) for i, m in enumerate(masked)}
        if step == 0:                                            # the prompt's K/V become the prefix cache
            for l in range(s.n_layers):
                cache_k[l] = k_new[l][:P]
                cache_v[l] = v_new[l][:P]
        for i in sel:
            tokens[P + masked[i]] = yhat[i]
        recs.append(dict(step=step, n_before=len(masked), rows=len(ids), masked=masked, sel=np.array(sel), yhat=yhat,
                         pmax=pmax, delta=delta, count=count, L_run=L_run, flips=flips, flip_base=base))
        step += 1
        if max_steps is not None and step >= max_steps:
            break
    return tokens, recs


def flip_counts(recs_masked_yhat):
    """Flip counts for any decode: recs_masked_yhat is a list of (absolute masked positions, yhat) per step."""
    out, prev = [], {}
    for pos, yhat in recs_masked_yhat:
        flips = sum(1 for p, y in zip(pos, yhat) if int(p) in prev and prev[int(p)] != int(y))
        base = sum(1 for p in pos if int(p) in prev)
        prev = {int(p): int(y) for p, y in zip(pos, yhat)}
        out.append((flips, base))
    return out
