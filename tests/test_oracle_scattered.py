"""Pins for oracle/scattered.py: the scattered-acceptance baselines and the flip count."""
import math

import numpy as np
import pytest

import lsp_synth as S
from oracle import dlm, scan
from oracle.decode import decode, make_is_delim
from oracle.scattered import decode_scattered, flip_counts, top_count


def _model(layers=2, seed=0):
    sh = S.ModelShape(layers, 64, 4, 2, 16, 128, 96, dtype="fp32", head_scale=2.0, w_std=0.125)
    return sh, dlm.OracleDLM(sh, S.make_weights(sh, seed))


def test_top_count_is_the_k_best_with_ties_to_the_lower_index():
    rng = np.random.default_rng(0)
    for _ in range(50):
        n = int(rng.integers(1, 30))
        sc = rng.integers(0, 6, n).astype(np.float64)           # many ties
        k = int(rng.integers(0, n + 1))
        sel = top_count(sc, k)
        assert len(sel) == k and sel == sorted(sel)
        rest = [i for i in range(n) if i not in sel]
        for i in sel:
            for j in rest:
                assert sc[i] > sc[j] or (sc[i] == sc[j] and i < j)


@pytest.mark.parametrize("k", [1, 5, 32, 100])
def test_top_k_step_count_and_immutability(k):
    sh, m = _model()
    prompt = S.make_prompt(1, 10, sh, 1)[0].numpy()
    G = 37
    tokens, recs = decode_scattered(m, prompt, G, k=k)
    assert len(recs) == math.ceil(G / k)                        # closed form: exactly min(k, masked) per step
    assert (tokens != sh.mask_id).all() and np.array_equal(tokens[:10], prompt)
    committed = {}
    for r in recs:
        assert r["count"] == min(k, r["n_before"]) == len(r["sel"])
        assert r["rows"] == (10 + G if r["step"] == 0 else G)   # the generation region never shrinks
        for i in r["sel"]:
            p = int(r["masked"][i])
            assert p not in committed                           # never rewritten
            committed[p] = int(r["yhat"][i])
    assert all(tokens[10 + p] == y for p, y in committed.items())
    if k == 1:
        bases = [r["flip_base"] for r in recs]
        assert bases == [0] + [G - 1 - i for i in range(len(recs) - 1)]
    for r in recs:
        assert 0 <= r["flips"] <= r["flip_base"]


def test_first_pass_equals_the_prefix_decode_first_pass():
    """Pass 0 is the same forward over prompt + masks in both topologies."""
    sh, m = _model()
    prompt = S.make_prompt(1, 9, sh, 2)[0].numpy()
    _, recs = decode_scattered(m, prompt, 20, k=4, max_steps=1)
    _, lrecs, _ = decode(m, prompt, 20, make_is_delim(1, 0), dict(tau=2.0), max_steps=1)
    np.testing.assert_allclose(recs[0]["pmax"], lrecs[0]["pmax"], rtol=0, atol=1e-12)
    assert np.array_equal(recs[0]["yhat"], lrecs[0]["yhat"])


def test_scattered_margin_takes_lsp_sized_counts_from_anywhere():
    sh, m = _model()
    prompt = S.make_prompt(1, 12, sh, 3)[0].numpy()
    pol = dict(mode=scan.MODE_ADAPTIVE, alpha=0.25, beta=0.5, W=-1)
    tokens, recs = decode_scattered(m, prompt, 40, lsp_policy=pol, is_delim=make_is_delim(1, 0))
    assert (tokens != sh.mask_id).all()
    for r in recs:
        N = r["n_before"]
        lo = max(1, math.ceil(0.25 * N)); hi = min(N, max(lo, math.floor(0.5 * N)))
        assert lo <= r["count"] <= hi and len(r["sel"]) == r["count"]
        # the accepted set is at least as confident as the left-aligned block of the same size
        assert r["pmax"][r["sel"]].sum() >= r["pmax"][:r["count"]].sum() - 1e-12


def test_flip_counts_helper_matches_decode_records():
    sh, m = _model()
    prompt = S.make_prompt(1, 8, sh, 4)[0].numpy()
    _, recs = decode_scattered(m, prompt, 25, k=3)
    fc = flip_counts([(r["masked"], r["yhat"]) for r in recs])
    assert fc == [(r["flips"], r["flip_base"]) for r in recs]
    assert flip_counts([([1, 2, 3], [5, 6, 7]), ([2, 3], [6, 9]), ([3], [9])]) == [(0, 0), (1, 2), (0, 1)]


def test_flip_counts_hand_examples():
    """Worked by hand.  A position counts in the base only if it was masked (scored) at the step before as well; it
    flips when its argmax differs between the two."""
    # step 0: nothing scored before.  step 1: positions 10..13 were all scored at step 0 -> base 4; 11 and 13 changed.
    # step 2: 12, 13 carried over, both changed; 20 is new (not in the base).
    assert flip_counts([([10, 11, 12, 13], [1, 2, 3, 4]),
                        ([10, 11, 12, 13], [1, 9, 3, 8]),
                        ([12, 13, 20], [4, 3, 3])]) == [(0, 0), (2, 4), (2, 2)]
    # a position that leaves the masked set and comes back is compared with the step just before only, where it was
    # absent: it is not in the base; an unchanged survivor is in the base and does not flip
    assert flip_counts([([0, 1], [7, 7]), ([1], [7]), ([0, 1], [5, 6])]) == [(0, 0), (0, 1), (1, 1)]
    # prefix decode that commits one position per step with stable predictions: base N-1, N-2, ... and no flips
    steps = [(list(range(k, 6)), [40 + p for p in range(k, 6)]) for k in range(6)]
    assert flip_counts(steps) == [(0, 0)] + [(0, 6 - k) for k in range(1, 6)]
