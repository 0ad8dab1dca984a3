"""Algorithm 1's loop with the block lengths kept on the device (lsp_set_option key 4): the host enqueues pass k+1 before
it has read L_k, sizes launches from row counts it knows one step late, and reads the records afterwards.  The decode
must be the one the synchronous loop (and the oracle) gives: same tokens, same per-step records."""
import numpy as np
import pytest
import torch

import lsp_synth as S
from oracle import scan as oscan
from oracle.decode import decode, make_is_delim
from gpu_util import DEV, make_pair, oracle_policy

pytestmark = pytest.mark.gpu
NEAR = oscan.FLAG_NEAR_THRESHOLD | oscan.FLAG_NEAR_TIE
KEYS = ("n_before", "rows", "L_run", "L_commit", "flags", "tau_used", "flips", "flip_base")


def _decode(sh, w, sched, Ps, Gs, stride, prompts, lagged, inplace=0, tail=None):
    from paper_2603_05454_b200 import LSPDecoder
    B = len(Ps)
    dec = LSPDecoder(sh, w, sched, B, stride, device=DEV)
    dec.set_option(4, lagged)
    dec.set_option(3, inplace)
    if tail is not None:
        dec.debug_set(31, tail)
    tokens = torch.zeros(B, stride, dtype=torch.int32, device=DEV)
    for b in range(B):
        tokens[b, :Ps[b]] = prompts[b, :Ps[b]]
    dec.begin(tokens, Ps, Gs)
    n, recs = dec.generate(max_recs=B * (max(Gs) + 2))
    assert dec.active()[1] == 0
    tk = tokens.cpu().numpy().copy()
    dec.close()
    return n, recs, tk


def _same_record(x, y):
    return all((x[k] == y[k]) or (k == "tau_used" and np.isnan(x[k]) and np.isnan(y[k])) for k in KEYS)


@pytest.mark.parametrize("sched_kw", [dict(tau=0.05), dict(mode=1, alpha=0.25, beta=0.5), dict(mode=2, fixed_k=7),
                                      dict(tau=0.0), dict(tau=2.0)])
@pytest.mark.parametrize("tail", [1, 8, 1000])
def test_lagged_loop_equals_the_synchronous_loop_fp32(sched_kw, tail):
    """fp32 models run on CUDA-core kernels whose per-row results do not depend on how many rows a launch has, so the
    two loops must agree bit for bit: tokens and every record, for a ragged batch, with the tail threshold at both
    extremes (1: lagged to the very end, so the last step is followed by an empty pass; 1000: every step read first).
    tau = 0 ends every sequence in one pass (the pass enqueued behind it finds nothing to do); tau = 2 commits one
    token per pass."""
    from paper_2603_05454_b200 import SchedCfg
    sh = S.ModelShape(2, 256, 4, 2, 64, 512, 1024, dtype="fp32", head_scale=1.5, w_std=0.0625)
    w = S.make_weights(sh, 9, device=DEV)
    Ps, Gs, stride = [5, 17, 32, 1], [30, 9, 64, 1], 96
    prompts = S.make_prompt(4, 32, sh, 11).to(DEV)
    sched = SchedCfg(delim_bitmap=S.delimiter_bitmap(sh.vocab, 1, 200).to(DEV), **sched_kw)
    n0, r0, t0 = _decode(sh, w, sched, Ps, Gs, stride, prompts, 0)
    n1, r1, t1 = _decode(sh, w, sched, Ps, Gs, stride, prompts, 1, tail=tail)
    assert n0 == n1 and len(r0) == len(r1)
    assert np.array_equal(t0, t1)
    for x, y in zip(r0, r1):
        assert _same_record(x, y), (x, y)
    if sched_kw.get("tau") == 0.0:
        assert n1 == 1
    if sched_kw.get("tau") == 2.0:
        assert n1 == max(Gs)


def test_lagged_loop_matches_the_oracle_free_running():
    from paper_2603_05454_b200 import SchedCfg
    sh = S.ModelShape(2, 256, 4, 2, 64, 512, 1024, dtype="fp32", head_scale=1.5, w_std=0.0625)
    w_gpu, om = make_pair(sh, 9)
    Ps, Gs, stride = [5, 17, 32], [30, 9, 64], 96
    sched = SchedCfg(tau=0.05, delim_bitmap=S.delimiter_bitmap(sh.vocab, 1, 200).to(DEV), flag_tol=1e-4, tie_tol=2e-4)
    prompts = S.make_prompt(3, 32, sh, 11)
    n, recs, tk = _decode(sh, w_gpu, sched, Ps, Gs, stride, prompts.to(DEV), 1)
    for b in range(3):
        otok, orecs, _ = decode(om, prompts[b, :Ps[b]].numpy(), Gs[b], make_is_delim(1, 200), oracle_policy(sched))
        mine = [r for r in recs[b::3] if r["n_before"] > 0]
        ok = True
        for r, o in zip(mine, orecs):
            if o["flags"] & NEAR:
                ok = False
                break
            assert (r["L_run"], r["L_commit"], r["n_before"], r["rows"]) == (o["L_run"], o["L_commit"], o["n_before"], o["rows"])
        if ok:
            assert len(mine) == len(orecs) and np.array_equal(tk[b, :Ps[b] + Gs[b]], otok)


@pytest.mark.parametrize("inplace", [0, 1])
def test_lagged_loop_bf16_tensor_core_kernels(inplace):
    """bf16, head_dim 128 (tcgen05 GEMMs, attention and fused head).  The LM-head launch of a lagged pass has more rows
    than the synchronous one, which can move a tile boundary and with it the last bits of a sum: the loops must agree
    up to the first step flagged near a threshold or tie."""
    from paper_2603_05454_b200 import SchedCfg
    sh = S.ModelShape(2, 512, 4, 2, 128, 1024, 4096, dtype="bf16", head_scale=1.5, w_std=0.044)
    w = S.make_weights(sh, 7, device=DEV)
    Ps, Gs, stride = [20, 150, 64], [100, 31, 130], 200
    prompts = S.make_prompt(3, 150, sh, 8).to(DEV)
    sched = SchedCfg(tau=0.04, delim_bitmap=S.delimiter_bitmap(sh.vocab, 1, 400).to(DEV), flag_tol=2e-2, tie_tol=0.1)
    n0, r0, t0 = _decode(sh, w, sched, Ps, Gs, stride, prompts, 0, inplace)
    n1, r1, t1 = _decode(sh, w, sched, Ps, Gs, stride, prompts, 1, inplace)
    assert (t1 != sh.mask_id)[[0, 1, 2], [Ps[0], Ps[1], Ps[2]]].all()
    for b in range(3):
        a = [r for r in r0[b::3] if r["n_before"] > 0]
        c = [r for r in r1[b::3] if r["n_before"] > 0]
        same = True
        for x, y in zip(a, c):
            if not _same_record(x, y):
                assert (x["flags"] | y["flags"]) & NEAR, (b, x, y)
                same = False
                break
            if (x["flags"] | y["flags"]) & NEAR:
                same = False
                break
        if same:
            assert len(a) == len(c) and np.array_equal(t0[b, :Ps[b] + Gs[b]], t1[b, :Ps[b] + Gs[b]])
        assert (t1[b, :Ps[b] + Gs[b]] != sh.mask_id).all()
        assert sum(r["L_commit"] for r in c) == Gs[b]
