"""K6 parity: the single-warp scan kernel against oracle/scan.py, bit-exact, through lsp_scan."""
import numpy as np
import pytest
import torch

import lsp_synth as S
from oracle import scan as oscan
from gpu_util import DEV

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dec():
    from paper_2603_05454_b200 import LSPDecoder, SchedCfg
    sh = S.ModelShape(1, 64, 1, 1, 64, 64, 4096, dtype="fp32")
    w = S.make_weights(sh, 0, device=DEV)
    d = LSPDecoder(sh, w, SchedCfg(), 64, 2048, device=DEV)
    yield d
    d.close()


def _case(dec, lens, seed, sched, p_pass=0.8, dens=0.12):
    from paper_2603_05454_b200 import SchedCfg
    V = 4096
    lo, hi = 1, 32
    bm = S.delimiter_bitmap(V, lo, hi).to(DEV)
    sched.delim_bitmap = bm
    dec.set_sched(sched)
    scores, yhats = [], []
    for i, n in enumerate(lens):
        sc, yh = S.synthetic_scores(n, seed, 10 * i, p_pass, float(np.float32(sched.tau)), dens, lo, hi, V)
        scores.append(sc); yhats.append(yh)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    sc_all = torch.cat(scores).to(DEV) if sum(lens) else torch.zeros(0, device=DEV)
    yh_all = torch.cat(yhats).to(DEV) if sum(lens) else torch.zeros(0, dtype=torch.int32, device=DEV)
    mg_all = (sc_all * 3).contiguous()
    out = dec.scan(sc_all, yh_all, mg_all, off)
    for b, n in enumerate(lens):
        if n == 0:
            assert out["L_commit"][b] == 0
            continue
        r = oscan.lsp_scan(scores[b].numpy(), yhats[b].numpy(), lambda t: lo <= t <= hi, mode=sched.mode,
                           tau=float(np.float32(sched.tau)), alpha=float(np.float32(sched.alpha)),
                           beta=float(np.float32(sched.beta)), l_min=sched.l_min, W=sched.snap_window,
                           fixed_k=sched.fixed_k, flag_tol=float(np.float32(sched.flag_tol)),
                           tie_tol=float(np.float32(sched.tie_tol)),
                           margin=(scores[b] * 3).numpy())
        assert out["L_run"][b] == r["L_run"], (b, n, out["L_run"][b], r)
        assert out["L_commit"][b] == r["L_commit"], (b, n, out["L_commit"][b], r)
        assert int(out["flags"][b]) == r["flags"], (b, n, int(out["flags"][b]), r)
        if sched.mode != 2:
            assert np.float32(out["tau_used"][b]) == np.float32(r["tau_used"])


LENS = [1, 2, 31, 32, 33, 64, 65, 100, 255, 256, 257, 1024, 1000, 7, 0, 513]


@pytest.mark.parametrize("W", [0, 1, 16, 40, -1])
@pytest.mark.parametrize("l_min", [1, 5])
def test_fixed_tau(dec, W, l_min):
    from paper_2603_05454_b200 import SchedCfg
    for seed, pp in ((0, 0.8), (1, 0.97), (2, 0.3), (3, 1.0)):
        _case(dec, LENS, seed, SchedCfg(tau=0.9, snap_window=W, l_min=l_min, flag_tol=0.01, tie_tol=0.4), p_pass=pp)


def test_adaptive_and_fixed_k(dec):
    from paper_2603_05454_b200 import SchedCfg
    for seed in range(4):
        _case(dec, LENS, seed, SchedCfg(mode=1, alpha=0.25, beta=0.5, snap_window=16), p_pass=0.6)
        _case(dec, LENS, seed, SchedCfg(mode=1, alpha=0.1, beta=0.9, snap_window=4, l_min=3), p_pass=0.9)
        _case(dec, LENS, seed, SchedCfg(mode=2, fixed_k=4))


def test_tau_zero_commits_everything_and_empty_delimiter_set(dec):
    from paper_2603_05454_b200 import SchedCfg
    _case(dec, LENS, 5, SchedCfg(tau=0.0), p_pass=0.5)
    dec.set_sched(SchedCfg(tau=0.5, delim_bitmap=None))
    sc = torch.tensor([0.9, 0.9, 0.1, 0.9], device=DEV)
    yh = torch.tensor([1, 1, 1, 1], dtype=torch.int32, device=DEV)
    out = dec.scan(sc, yh, None, [0, 4])
    assert out["L_commit"][0] == 2 and out["L_run"][0] == 2
