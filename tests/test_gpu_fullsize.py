"""Parity at the benchmark configurations' full widths, on outputs the oracle can afford to compute.

 * cfg2 (fused LM head + confidence + scan, hidden [8 x 1024, 4096], vocabulary 126464): the oracle computes full
   fp64 logits only for sampled rows and for the left end of every sequence up to one row past the first position that
   fails the threshold, which is all the scan's result depends on.
 * LLaDA-8B- and Dream-7B-shaped layers (full d_model, heads, FFN width; one layer, small vocabulary): teacher-forced
   decode steps whose row counts cover the tiled GEMM (more than 256 rows) and both shapes of the streaming GEMM.
"""
import numpy as np
import pytest
import torch

import lsp_synth as S
from oracle import scan as oscan
from oracle.scores import scores_from_logits
from gpu_util import DEV, tol_for, tol_logit
from test_gpu_decode import _teacher_forced

pytestmark = pytest.mark.gpu
NEAR = oscan.FLAG_NEAR_THRESHOLD | oscan.FLAG_NEAR_TIE


def test_cfg2_full_size_head_and_scan_on_sampled_rows_and_run_prefixes():
    from paper_2603_05454_b200 import LSPDecoder, SchedCfg
    d, V, B, L, tau, scale = 4096, 126464, 8, 1024, 0.9, 6.0
    sh = S.ModelShape(1, d, 32, 32, 128, 64, V, dtype="bf16", head_scale=scale)
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device=DEV)
    w = dict(embed=z(8, d), w_head=S.normal((V, d), 0, S.TID_HEAD, 0.02 * scale, torch.bfloat16, DEV),
             final_norm=torch.ones(d, dtype=torch.bfloat16, device=DEV),
             layers=[dict(attn_norm=z(d), w_qkv=z(3 * d, d), w_o=z(d, d), ffn_norm=z(d), w_gate=z(64, d), w_up=z(64, d),
                          w_down=z(d, 64))])
    hidden = S.normal((B * L, d), 0, 77, 1.0, torch.bfloat16, DEV)
    w64 = w["w_head"].float().cpu().numpy().astype(np.float64)
    h_cpu = hidden.float().cpu().numpy().astype(np.float64)
    tol = tol_for("bf16")
    # identical inputs on both sides: only the accumulation order differs
    tol_z = tol_logit("fp32", 0.02 * scale * np.sqrt(d))
    sched = SchedCfg(tau=tau, delim_bitmap=S.delimiter_bitmap(V, 1, 32).to(DEV), flag_tol=tol, tie_tol=tol_z)
    dec = LSPDecoder(sh, w, sched, B, L, device=DEV)
    off = np.arange(B + 1, dtype=np.int32) * L
    out = dec.head_scan(hidden, off)
    y, p, m = dec.scores()
    dec.close()

    def oracle_rows(rows):
        return scores_from_logits(h_cpu[rows] @ w64.T, sh.mask_id)

    # (a) sampled rows anywhere (several row tiles, both ends)
    rows = np.unique(np.concatenate([[0, 1, 127, 128, 129, B * L - 1], (np.arange(40) * 204 + 7) % (B * L)]))
    yo, po, mo = oracle_rows(rows)
    assert np.abs(p[rows] - po).max() <= 1e-4
    assert np.abs(m[rows] - mo).max() <= tol_z
    assert all(mo[i] <= tol_z for i in np.nonzero(y[rows] != yo)[0])
    # (b) every sequence's run: oracle scores from the left until one row past the first failure
    for b in range(B):
        n = 32
        while True:
            yo, po, mo = oracle_rows(np.arange(off[b], off[b] + n))
            if (po < tau).any() or n >= L:
                break
            n = min(L, 2 * n)
        first_fail = int(np.argmax(po < tau)) if (po < tau).any() else n
        keep = min(n, first_fail + 2)
        r = oscan.lsp_scan(po[:keep], yo[:keep], lambda t: 1 <= t <= 32, tau=float(np.float32(tau)), W=16,
                           flag_tol=float(np.float32(tol)), tie_tol=float(np.float32(tol_z)), margin=mo[:keep])
        if r["flags"] & NEAR:
            continue
        # a truncated sequence can only differ from the full one in the run-to-end rule, which needs L' = keep
        assert r["L_run"] < keep
        assert (out["L_run"][b], out["L_commit"][b]) == (r["L_run"], r["L_commit"]), (b, out, r)


@pytest.mark.parametrize("name", ["llada", "dream"])
def test_full_width_layer_teacher_forced_steps(name):
    from paper_2603_05454_b200 import SchedCfg
    if name == "llada":
        sh = S.ModelShape(1, 4096, 32, 32, 128, 12288, 8192, dtype="bf16", head_scale=4.0)
    else:
        sh = S.ModelShape(1, 3584, 28, 4, 128, 18944, 8192, dtype="bf16", head_scale=4.0, rope_theta=1e6)
    # pass 0 has 300 rows (tiled GEMM, three row tiles), pass 1 about 250 (streaming GEMM, two row tiles); the
    # fixed-k policy then walks the row count down through the one-row-tile regime
    _teacher_forced(sh, 21, 50, 250, SchedCfg(tau=0.9), (1, 64), max_steps=2)
    _teacher_forced(sh, 22, 8, 150, SchedCfg(mode=2, fixed_k=60), (1, 64), max_steps=3)


def test_full_width_layer_teacher_forced_steps_adaptive_threshold():
    """Eq. 2 at full layer width: the adaptive block keeps L' inside [alpha N, beta N], step by step against the oracle."""
    from paper_2603_05454_b200 import SchedCfg
    sh = S.ModelShape(1, 4096, 32, 32, 128, 12288, 8192, dtype="bf16", head_scale=4.0)
    _teacher_forced(sh, 23, 40, 260, SchedCfg(mode=1, alpha=0.25, beta=0.5), (1, 64), max_steps=4)


def test_adaptive_threshold_decode_shrinks_the_suffix_geometrically_at_full_vocabulary():
    """Properties of Eq. 2 that hold at any size, on a free-running decode (two full-width LLaDA-shaped layers, the full
    126464-entry vocabulary, batch 2, 64 + 512): every step's run lies in [ceil(alpha N), floor(beta N)], the committed
    block is the run or a delimiter at most W before it, the suffix therefore shrinks by a constant factor while
    alpha N > W, and the rows touched in total stay far below the quadratic count of one-token steps."""
    import math
    from paper_2603_05454_b200 import LSPDecoder, SchedCfg
    alpha, beta, W = 0.25, 0.5, 16
    sh = S.ModelShape(2, 4096, 32, 32, 128, 12288, 126464, dtype="bf16", head_scale=12.0)
    w = S.make_weights(sh, 5, device=DEV)
    bm = S.delimiter_bitmap(sh.vocab, 1, 32).to(DEV)
    B, P, G = 2, 64, 512
    dec = LSPDecoder(sh, w, SchedCfg(mode=1, alpha=alpha, beta=beta, snap_window=W, delim_bitmap=bm), B, P + G, device=DEV)
    tokens = torch.full((B, P + G), sh.mask_id, dtype=torch.int32, device=DEV)
    tokens[:, :P] = S.make_prompt(B, P, sh, 9).to(DEV)
    dec.begin(tokens, [P] * B, [G] * B)
    n, recs = dec.generate(max_recs=B * (G + 1))
    dec.close()
    assert int((tokens == sh.mask_id).sum()) == 0
    for b in range(B):
        mine = [r for r in recs[b::B] if r["n_before"] > 0]
        N = G
        for r in mine:
            assert r["n_before"] == N
            lo = max(1, math.ceil(alpha * N))
            hi = min(N, max(lo, math.floor(beta * N)))
            assert lo <= r["L_run"] <= hi, r
            assert max(1, r["L_run"] - W) <= r["L_commit"] <= r["L_run"], r
            if alpha * N > 2 * W:                          # the block is at least half the lower end of the range
                assert N - r["L_commit"] <= (1 - alpha / 2) * N
            N -= r["L_commit"]
        assert N == 0
        assert sum(r["n_before"] for r in mine) < G * G / 8     # one-token steps would touch G (G + 1) / 2 masked rows
    assert n == max(len([r for r in recs[b::B] if r["n_before"] > 0]) for b in range(B))


@pytest.mark.parametrize("name,checked_steps", [("cfg3", 12), ("cfg4", 6)])
def test_full_depth_decode_in_the_benchmark_configuration_keeps_its_invariants(name, checked_steps):
    """The LLaDA-8B-shaped decode (cfg3: 32 layers, batch 1, 256 + 256, tau 0.9) and the Dream-7B-shaped one (cfg4: 28
    layers, grouped-query attention 28/4, batch 4, 512 + 512, tau 0.85) exactly as the benchmark runs them (full
    vocabulary, default kernels), checked against what Algorithm 1 fixes at any size: every step's record is the scan of
    that step's own scores (run = leading positions with p_max >= tau; block = run or the last delimiter at most W
    before its end; never 0), the committed tokens are that step's argmaxes, the frozen prefix never changes, the masked
    suffix shrinks by exactly the committed block, and the KV cache holds exactly the committed prefix minus the block
    still pending."""
    from paper_2603_05454_b200 import LSPDecoder, SchedCfg
    wl = S.config(name)
    sh = wl.shape
    W = 16
    w = S.make_weights(sh, 0, device=DEV)
    bm = S.delimiter_bitmap(sh.vocab, *wl.delim).to(DEV)
    B, P, G = wl.batch, wl.prompt_len, wl.gen_len
    dec = LSPDecoder(sh, w, SchedCfg(tau=wl.tau, snap_window=W, delim_bitmap=bm), B, P + G, device=DEV)
    tokens = torch.full((B, P + G), sh.mask_id, dtype=torch.int32, device=DEV)
    tokens[:, :P] = S.make_prompt(B, P, sh, 100).to(DEV)
    dec.begin(tokens, [P] * B, [G] * B)
    tau32 = np.float32(wl.tau)
    N, F, pend = [G] * B, [0] * B, [P] * B
    frozen = [tokens[b, :P].cpu().numpy().copy() for b in range(B)]
    steps = 0
    while max(N) > 0 and steps < checked_steps:
        recs = dec.denoise_step()
        y_all, p_all, m_all = dec.scores()
        assert len(p_all) == sum(N)
        assert (p_all > 0).all() and (p_all <= 1.0 + 1e-6).all() and (m_all >= 0).all()
        assert (y_all >= 0).all() and (y_all != sh.mask_id).all()
        off = 0
        blocks = []
        for b in range(B):
            rec = recs[b]
            if N[b] == 0:
                assert rec["n_before"] == 0
                blocks.append(None)
                continue
            y, p = y_all[off:off + N[b]], p_all[off:off + N[b]]
            off += N[b]
            assert rec["n_before"] == N[b] and rec["rows"] == pend[b] + N[b]
            run = int(np.argmax(p < tau32)) if (p < tau32).any() else N[b]
            assert rec["L_run"] == run
            if run == N[b]:
                want = N[b]
            else:
                delims = [j for j in range(max(1, run - W), run + 1) if wl.delim[0] <= y[j - 1] <= wl.delim[1]]
                want = max(1, delims[-1] if delims else run)
            assert rec["L_commit"] == min(N[b], max(1, want)), (steps, b, rec, run)
            blocks.append(y[:rec["L_commit"]].copy())
        dec.commit()
        tk = tokens.cpu().numpy()
        for b in range(B):
            if blocks[b] is None:
                continue
            L, f = len(blocks[b]), len(frozen[b])
            assert np.array_equal(tk[b, :f], frozen[b])                         # prefix immutability
            assert np.array_equal(tk[b, f:f + L], blocks[b])                    # the block is this step's argmaxes
            assert (tk[b, f + L:] == sh.mask_id).all()
            frozen[b] = tk[b, :f + L].copy()
            F[b], pend[b], N[b] = F[b] + pend[b], L, N[b] - L
        steps += 1
    if max(N) > 0:                                                              # the rest in one call
        n_more, recs = dec.generate(max_recs=B * (G + 1))
        for b in range(B):
            live = [r for r in recs[b::B] if r["n_before"] > 0]
            assert sum(r["L_commit"] for r in live) == N[b] and all(r["L_commit"] >= 1 for r in live)
            if live:
                F[b], pend[b] = F[b] + pend[b] + sum(r["L_commit"] for r in live[:-1]), live[-1]["L_commit"]
            N[b] = 0
    assert dec.active()[1] == 0 and int((tokens == sh.mask_id).sum()) == 0
    kv = dec.kv_view()
    for b in range(B):
        assert np.array_equal(tokens[b, :len(frozen[b])].cpu().numpy(), frozen[b])
        assert F[b] + pend[b] == P + G
        assert bool((kv[:, :, b, :F[b]].float().abs().amax(dim=(-1, -2)) > 0).all())   # every cached row was written ...
        assert not bool(kv[:, :, b, F[b]:].any())                                       # ... and nothing beyond the cache length
    dec.close()


def test_full_depth_decode_is_reproducible_bit_for_bit():
    """Every reduction on the path has a fixed order (split-K partials in K order, vocab tiles in tile order, the scan in
    position order), so repeating a decode must reproduce the tokens and every step record exactly: cfg3 at full depth,
    in the adaptive-threshold mode (11 passes that cross every row regime from 512 rows down to 2)."""
    from paper_2603_05454_b200 import LSPDecoder, SchedCfg
    wl = S.config("cfg3")
    sh = wl.shape
    w = S.make_weights(sh, 0, device=DEV)
    bm = S.delimiter_bitmap(sh.vocab, *wl.delim).to(DEV)
    P, G = wl.prompt_len, wl.gen_len
    dec = LSPDecoder(sh, w, SchedCfg(mode=1, alpha=0.25, beta=0.5, delim_bitmap=bm), 1, P + G, device=DEV)
    prompt = S.make_prompt(1, P, sh, 100).to(DEV)
    runs = []
    for _ in range(3):
        tokens = torch.full((1, P + G), sh.mask_id, dtype=torch.int32, device=DEV)
        tokens[:, :P] = prompt
        dec.begin(tokens, [P], [G])
        n, recs = dec.generate(max_recs=G + 1)
        runs.append((n, tokens.cpu().numpy().copy(), [(r["L_run"], r["L_commit"], r["flags"], r["tau_used"]) for r in recs]))
    dec.close()
    for n, tk, rc in runs[1:]:
        assert n == runs[0][0] and np.array_equal(tk, runs[0][1]) and rc == runs[0][2]
