"""Oracle: stability run, adaptive threshold, delimiter snap, fallback (Sec. 3.2, Eq. 2, the
snapping display formula, Algorithm 1, threshold / snap / fallback steps).  TEST INFRASTRUCTURE, not a product path.

Notation follows the paper: positions of the active suffix are 1..N, ``score_i`` is the
stability score (logit margin delta_i of Eq. 1, or the max-probability used by the benchmark
configurations), ``L'`` the candidate run, ``L`` the committed length, ``D`` the delimiter
set, ``W`` the look-back window, ``L_min`` the minimum block.

Readings taken where the paper is silent or inconsistent:
  * the test is ``score_i >= tau`` (the paper says "exceed"; ">=" is what makes tau = 0
    accept everything for either score);
  * adaptive mode picks the LARGEST achievable m in [ceil(alpha N), floor(beta N)]; when no m
    in the range is achievable the range's upper end is used and the step is flagged;
  * a run that reaches the end of the sequence is committed whole (the sequence end is a
    boundary); with no delimiter in the window the run's own end is kept (the prose restricts
    the L_min fallback to blocks shorter than L_min);
  * finally 1 <= L <= N (Algorithm 1's "if L = 0 then L <- 1").

Pins: brute force over all pass patterns for N <= 12 (all delimiter patterns for N <= 8), tau = 0 and
tau = +inf special cases, fixed-k closed form (Table 2), adaptive range invariant and the
15-step geometric sequence.  The choice of m inside the adaptive range is "parity unpinned"
(the paper does not state it).
"""
import math

FLAG_SNAPPED = 1            # L < L' because a delimiter inside the window ended the block
FLAG_FALLBACK = 2           # L' = 0 (or L' < L_min): progress forced by L_min / L <- 1
FLAG_RANGE_UNACHIEVABLE = 4 # adaptive mode: no threshold gives a run inside [alpha N, beta N]
FLAG_RUN_TO_END = 8         # the run covers the whole active suffix
FLAG_NEAR_THRESHOLD = 16    # some decisive score lies within flag_tol of the threshold
FLAG_NEAR_TIE = 32          # some committed position's top-2 logits are within flag_tol

MODE_FIXED_TAU, MODE_ADAPTIVE, MODE_FIXED_K = 0, 1, 2


def longest_stable_run(score, tau):
    """L'(tau): length of the longest run starting at position 1 with score_i >= tau (Sec. 3.2)."""
    N = len(score)
    Lp = 0
    while Lp < N and float(score[Lp]) >= tau:
        Lp += 1
    return Lp


def adaptive_threshold(score, alpha, beta):
    """Eq. 2 via the prefix minimum: returns (m_star, tau_k, range_unachievable).

    pm[m] = min_{i<=m} score_i, pm[N+1] = -inf.  Under ">=" a length m is achievable iff
    pm[m] > pm[m+1] (any tau in (pm[m+1], pm[m]] gives L'(tau) = m)."""
    N = len(score)
    pm = [math.inf] * (N + 2)
    for m in range(1, N + 1):
        pm[m] = min(pm[m - 1], float(score[m - 1]))
    pm[N + 1] = -math.inf
    lo = max(1, math.ceil(float(alpha) * N))
    hi = min(N, max(lo, math.floor(float(beta) * N)))
    for m in range(hi, lo - 1, -1):
        if pm[m] > pm[m + 1]:
            return m, pm[m], False
    return hi, pm[hi], True


def snap_to_delimiter(yhat, L_run, N, is_delim, l_min, W):
    """The snapping rule plus fallback: returns (L, flags)."""
    flags = 0
    if L_run == N:                       # run ends at the end of the sequence
        L = N
        flags |= FLAG_RUN_TO_END
    else:
        lo_j = 1 if W < 0 else max(1, L_run - W)
        J = [j for j in range(lo_j, L_run + 1) if is_delim(int(yhat[j - 1]))]
        if J:
            L = max(l_min, max(J))
            if max(J) < L_run and L < L_run:
                flags |= FLAG_SNAPPED
        else:
            L = max(l_min, L_run)
    if L_run < max(1, l_min) and L_run < N:
        flags |= FLAG_FALLBACK
    L = min(N, max(L, 1))
    return L, flags


def lsp_scan(score, yhat, is_delim, mode=MODE_FIXED_TAU, tau=0.9, alpha=0.25, beta=0.5,
             l_min=1, W=16, fixed_k=1, flag_tol=0.0, tie_tol=0.0, margin=None):
    """One scheduler decision for one sequence.  Returns a dict with L_run (L'), L_commit (L),
    tau_used and flags."""
    N = len(score)
    assert N >= 1
    flags = 0
    if mode == MODE_FIXED_K:             # ablation policy: commit exactly k tokens, no snapping
        L = min(N, max(1, int(fixed_k)))
        return dict(L_run=L, L_commit=L, tau_used=float("nan"), flags=0)
    if mode == MODE_ADAPTIVE:
        L_run, tau_used, unach = adaptive_threshold(score, alpha, beta)
        if unach:
            flags |= FLAG_RANGE_UNACHIEVABLE
    else:
        tau_used = float(tau)
        L_run = longest_stable_run(score, tau_used)
    L, f2 = snap_to_delimiter(yhat, L_run, N, is_delim, l_min, W)
    flags |= f2
    # near-threshold / near-tie flags used by the comparison protocol (not part of the method)
    if flag_tol > 0:
        for i in range(min(N, L_run + 1)):
            if abs(float(score[i]) - tau_used) <= flag_tol:
                flags |= FLAG_NEAR_THRESHOLD
    if tie_tol > 0 and margin is not None:
        for i in range(L):
            if float(margin[i]) <= tie_tol:
                flags |= FLAG_NEAR_TIE
    return dict(L_run=L_run, L_commit=L, tau_used=tau_used, flags=flags)
