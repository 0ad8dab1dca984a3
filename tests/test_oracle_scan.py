"""Pins for oracle/scan.py: brute force over every pass/delimiter pattern on tiny suffixes,
the special cases the method fixes, and the adaptive-range invariants."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import scan as S

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def definitional(passes, delims, l_min, W):
    """Written from the definitions, independently of oracle/scan.py: L' by trying every m
    from N down; the snap target as a set-builder maximum."""
    N = len(passes)
    Lp = next(m for m in range(N, -1, -1) if all(passes[:m]))
    if Lp == N:
        return Lp, N
    J = {j for j in range(1, Lp + 1) if delims[j - 1] and (W < 0 or Lp - j <= W)}
    L = max(l_min, max(J)) if J else max(l_min, Lp)
    return Lp, min(N, max(1, L))


def _delimiter_patterns(N):
    """Every delimiter pattern up to N = 8; beyond that five fixed patterns plus eight seeded random ones."""
    if N <= 8:
        return list(itertools.product((0, 1), repeat=N))
    rng = np.random.default_rng(1000 + N)
    fixed = [tuple(int((i * 7 + k) % 3 == 0) for i in range(N)) for k in range(3)] + [(0,) * N, (1,) * N]
    return fixed + [tuple(int(x) for x in rng.integers(0, 2, N)) for _ in range(8)]


@pytest.mark.parametrize("N", list(range(1, 13)))
def test_scan_brute_force_all_patterns(N):
    for W in (0, 1, 2, 16, -1):
        for l_min in (1, 3):
            for passes in itertools.product((0, 1), repeat=N):
                score = [0.95 if p else 0.10 for p in passes]
                for delims in _delimiter_patterns(N):
                    yhat = [1 if d else 100 for d in delims]
                    r = S.lsp_scan(score, yhat, lambda t: t == 1, tau=0.9, l_min=l_min, W=W)
                    Lp, L = definitional(passes, delims, l_min, W)
                    assert (r["L_run"], r["L_commit"]) == (Lp, L), (passes, delims, W, l_min)
                    # properties that must hold for any input
                    assert 1 <= L <= N
                    assert L <= max(Lp, l_min, 1)
                    if L < Lp:
                        assert delims[L - 1] or L == l_min
                        if delims[L - 1] and L > l_min:
                            assert W < 0 or Lp - L <= W
                            # it is the LAST delimiter of the run
                            assert not any(delims[L:Lp])
                    if Lp < N and L > Lp:
                        assert L == min(N, max(1, l_min))


def test_threshold_is_inclusive_and_tau_zero_commits_everything():
    assert S.longest_stable_run([0.9, 0.9, 0.89], 0.9) == 2
    for N in (1, 7, 64):
        score = np.linspace(0.0, 1.0, N)
        yhat = np.arange(N) % 5      # delimiters everywhere
        r = S.lsp_scan(score, yhat, lambda t: t == 1, tau=0.0, W=16)
        assert r["L_commit"] == N and r["L_run"] == N


def test_tau_infinite_commits_exactly_one():
    r = S.lsp_scan([1.0] * 9, [1] * 9, lambda t: t == 1, tau=math.inf)
    assert r["L_run"] == 0 and r["L_commit"] == 1 and r["flags"] & S.FLAG_FALLBACK


def test_snap_window_and_last_delimiter():
    score = [1.0] * 20 + [0.0] * 5
    yhat = [100] * 25
    yhat[2] = 1      # j = 3
    yhat[11] = 1     # j = 12
    is_d = lambda t: t == 1
    assert S.lsp_scan(score, yhat, is_d, W=16)["L_commit"] == 12      # last delimiter in window
    assert S.lsp_scan(score, yhat, is_d, W=8)["L_commit"] == 12       # 20 - 12 = 8 <= W
    assert S.lsp_scan(score, yhat, is_d, W=7)["L_commit"] == 20       # outside: keep the run end
    assert S.lsp_scan(score, yhat, is_d, W=-1)["L_commit"] == 12
    yhat[19] = 1
    assert S.lsp_scan(score, yhat, is_d, W=0)["L_commit"] == 20       # delimiter at the run end
    assert S.lsp_scan(score, yhat, is_d, W=16, l_min=15)["L_commit"] == 20


def test_fixed_k_step_counts_match_table2():
    rows = [l.split() for l in open(os.path.join(GOLD, "table2_fixed_prefix_steps.txt"))
            if l.strip() and not l.startswith("#")]
    for G, k, steps in [(int(a), int(b), int(c)) for a, b, c in rows]:
        N, n = G, 0
        while N > 0:
            r = S.lsp_scan([0.0] * N, [5] * N, lambda t: False, mode=S.MODE_FIXED_K, fixed_k=k)
            N -= r["L_commit"]
            n += 1
        assert n == steps == math.ceil(G / k)


def test_adaptive_range_invariant_and_consistency_with_fixed_run():
    rng = np.random.default_rng(0)
    for _ in range(300):
        N = int(rng.integers(1, 80))
        score = rng.random(N) if rng.random() < 0.7 else np.round(rng.random(N), 1)
        a, b = 0.25, 0.5
        m, tau, unach = S.adaptive_threshold(score, a, b)
        lo = max(1, math.ceil(a * N))
        hi = min(N, max(lo, math.floor(b * N)))
        assert lo <= m <= hi
        assert tau == min(score[:m])
        run_at_tau = S.longest_stable_run(score, tau)
        if unach:
            assert run_at_tau > hi or m == hi
            # truly no achievable length in range: for each m' the run at its own prefix-min overshoots
            for mm in range(lo, hi + 1):
                assert S.longest_stable_run(score, min(score[:mm])) != mm
        else:
            assert run_at_tau == m                       # Eq. 2 holds at the chosen threshold
            for mm in range(m + 1, hi + 1):              # and m is the largest such length
                assert S.longest_stable_run(score, min(score[:mm])) != mm


def test_adaptive_geometric_decay_15_steps():
    """alpha = 0.25, no snapping, scores that make only m = ceil(alpha N) achievable:
    128 -> 96 -> 72 -> ... -> 0 takes 15 steps (ceil(N/4) leaves floor(3N/4))."""
    N, seq = 128, []
    while N > 0:
        lo = math.ceil(0.25 * N)
        score = [1.0] * lo + [0.0] * (N - lo)
        r = S.lsp_scan(score, [7] * N, lambda t: False, mode=S.MODE_ADAPTIVE, alpha=0.25, beta=0.5)
        expect = N if lo == N else lo
        assert r["L_commit"] == expect
        seq.append(N)
        N -= r["L_commit"]
    assert seq == [128, 96, 72, 54, 40, 30, 22, 16, 12, 9, 6, 4, 3, 2, 1]


def test_flags():
    is_d = lambda t: t == 1
    r = S.lsp_scan([1, 1, 1, 1, 0], [9, 1, 9, 9, 9], is_d, tau=0.5)
    assert r["L_commit"] == 2 and r["flags"] & S.FLAG_SNAPPED
    r = S.lsp_scan([1, 1, 1], [9, 1, 9], is_d, tau=0.5)
    assert r["L_commit"] == 3 and r["flags"] & S.FLAG_RUN_TO_END and not r["flags"] & S.FLAG_SNAPPED
    r = S.lsp_scan([0.91, 0.5], [9, 9], is_d, tau=0.9, flag_tol=0.02)
    assert r["flags"] & S.FLAG_NEAR_THRESHOLD
    r = S.lsp_scan([0.99, 0.5], [9, 9], is_d, tau=0.9, flag_tol=0.02)
    assert not r["flags"] & S.FLAG_NEAR_THRESHOLD
