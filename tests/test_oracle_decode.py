"""Pins for oracle/decode.py: the invariants Algorithm 1 guarantees, the closed-form step
counts, and the cache plumbing checks (cached vs recompute-everything)."""
import math

import numpy as np
import pytest

import lsp_synth as S
from oracle import dlm, scan
from oracle.decode import decode, make_is_delim


def _model(layers=2, dtype="fp32", seed=0, head_scale=2.0):
    # w_std is raised so that a 64-wide model has the same per-projection gain (w_std * sqrt(d)
    # ~ 1) as the 4096-wide benchmark shapes at 0.02; otherwise every masked row predicts alike.
    sh = S.ModelShape(layers, 64, 4, 2, 16, 128, 96, dtype=dtype, head_scale=head_scale, w_std=0.125)
    return sh, dlm.OracleDLM(sh, S.make_weights(sh, seed))


def _check_invariants(sh, prompt, G, tokens, recs, is_delim, l_min=1):
    P = len(prompt)
    assert np.array_equal(tokens[:P], prompt)
    assert (tokens != sh.mask_id).all()                     # terminates fully committed
    N, Fp = G, P
    snapshot = tokens.copy()
    for r in recs:
        assert r["n_before"] == N and r["Fp"] == Fp
        L, Lp = r["L_commit"], r["L_run"]
        assert 1 <= L <= N                                  # monotone progress
        assert np.array_equal(snapshot[Fp:Fp + L], r["yhat"][:L])   # committed block = yhat_{1:L}, never rewritten later
        if L < Lp:                                          # snapped only to a delimiter (or L_min)
            assert is_delim(int(r["yhat"][L - 1])) or L == l_min
        elif L > Lp:
            assert L == max(1, l_min) or L == N
        N -= L
        Fp += L
    assert N == 0 and Fp == P + G


@pytest.mark.parametrize("mode", ["fixed", "adaptive"])
def test_loop_invariants(mode):
    sh, m = _model()
    prompt = S.make_prompt(1, 12, sh, 0)[0].numpy()
    is_d = make_is_delim(1, 40)      # dense delimiters so that snapping fires inside the loop
    pol = dict(tau=0.15, W=16, l_min=1) if mode == "fixed" else dict(mode=scan.MODE_ADAPTIVE, alpha=0.25, beta=0.5)
    tokens, recs, (ck, cv) = decode(m, prompt, 40, is_d, pol)
    _check_invariants(sh, prompt, 40, tokens, recs, is_d)
    assert any(r["flags"] & scan.FLAG_SNAPPED for r in recs)
    rows = [r["rows"] for r in recs]
    assert all(a >= b for a, b in zip(rows, rows[1:]))      # the pass shrinks monotonically
    assert rows[0] == 12 + 40
    # cache = every committed position except the last block, written once
    assert ck[0].shape[0] == 12 + 40 - recs[-1]["L_commit"]
    if mode == "adaptive":
        for r in recs:
            N = r["n_before"]
            lo = max(1, math.ceil(0.25 * N)); hi = min(N, max(lo, math.floor(0.5 * N)))
            assert lo <= r["L_run"] <= hi


def test_tau_zero_one_step_tau_inf_G_steps_fixed_k():
    sh, m = _model()
    prompt = S.make_prompt(1, 8, sh, 1)[0].numpy()
    is_d = make_is_delim(1, 12)
    tokens, recs, _ = decode(m, prompt, 20, is_d, dict(tau=0.0))
    assert len(recs) == 1 and recs[0]["L_commit"] == 20
    tokens, recs, _ = decode(m, prompt, 20, is_d, dict(tau=math.inf))
    assert len(recs) == 20 and all(r["L_commit"] == 1 for r in recs)
    for k in (1, 2, 4, 8, 3):
        _, recs, _ = decode(m, prompt, 20, is_d, dict(mode=scan.MODE_FIXED_K, fixed_k=k))
        assert len(recs) == math.ceil(20 / k)


def test_cache_rows_written_once_and_never_change():
    sh, m = _model()
    prompt = S.make_prompt(1, 10, sh, 2)[0].numpy()
    seen = {}

    def on_step(rec, logits, k_new, v_new):
        seen[rec["step"]] = (rec["F"], rec["pend"], [k[:rec["pend"]].copy() for k in k_new])

    tokens, recs, (ck, cv) = decode(m, prompt, 30, make_is_delim(1, 12), dict(tau=0.15), on_step=on_step)
    for step, (F, pend, ks) in seen.items():
        for l in range(sh.n_layers):
            assert np.array_equal(ck[l][F:F + pend], ks[l])


def test_pass0_and_layer0_rows_equal_in_cached_and_nocache_modes():
    sh, m = _model(layers=2)
    prompt = S.make_prompt(1, 10, sh, 3)[0].numpy()
    grab = {True: [], False: []}
    for uc in (True, False):
        def on_step(rec, logits, k_new, v_new, uc=uc):
            grab[uc].append((rec, logits.copy(), k_new[0].copy()))
        decode(m, prompt, 24, make_is_delim(1, 12), dict(tau=0.15), use_cache=uc, on_step=on_step, max_steps=4)
    r0c, l0c, _ = grab[True][0]
    r0n, l0n, _ = grab[False][0]
    np.testing.assert_allclose(l0c, l0n, rtol=0, atol=0)                 # pass 0 identical
    # layer-0 K of the pending block depends only on (token, position): equal to recomputed rows,
    # as long as both trajectories are still the same
    for (rc, _, kc), (rn, _, kn) in zip(grab[True], grab[False]):
        if rc["Fp"] != rn["Fp"] or not np.array_equal(rc["yhat"][:rc["L_commit"]], rn["yhat"][:rn["L_commit"]]):
            break
        np.testing.assert_allclose(kc[:rc["pend"]], kn[rc["F"]:rc["F"] + rc["pend"]], rtol=1e-12, atol=1e-13)


def test_one_layer_model_cached_equals_nocache():
    """With one layer the cached K/V depend only on a position's own token and index, so
    prefix caching is exact: both modes give the same logits and the same decode."""
    sh, m = _model(layers=1, seed=5)
    prompt = S.make_prompt(1, 10, sh, 4)[0].numpy()
    out = {}
    for uc in (True, False):
        logs = []
        t, recs, _ = decode(m, prompt, 40, make_is_delim(1, 12), dict(tau=0.1), use_cache=uc,
                            on_step=lambda rec, lg, k, v: logs.append(lg.copy()))
        out[uc] = (t, recs, logs)
    assert np.array_equal(out[True][0], out[False][0])
    assert [r["L_commit"] for r in out[True][1]] == [r["L_commit"] for r in out[False][1]]
    for a, b in zip(out[True][2], out[False][2]):
        np.testing.assert_allclose(a, b, rtol=1e-9, atol=1e-10)
    assert len(out[True][1]) > 2          # a real multi-step decode, not a degenerate one


def test_bf16_model_decodes_with_invariants():
    sh, m = _model(dtype="bf16", seed=7)
    prompt = S.make_prompt(1, 6, sh, 5)[0].numpy()
    is_d = make_is_delim(1, 12)
    tokens, recs, _ = decode(m, prompt, 16, is_d, dict(tau=0.15))
    _check_invariants(sh, prompt, 16, tokens, recs, is_d)
