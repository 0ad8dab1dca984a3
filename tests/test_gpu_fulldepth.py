"""Full-depth parity (Algorithm 1 and Eq. 1 at the benchmark's sizes): the first decode passes of the LLaDA-8B-shaped
workload (cfg3: 32 layers, vocabulary 126464, batch 1) and of the Dream-7B-shaped one (cfg4: 28 layers, grouped-query
attention 28/4, batch 4) in the launch configuration bench.py times, teacher-forced against the CPU oracle.

The oracle's records come from tests/golden/fulldepth_<workload>.txt (written by the script beside it, which calls only
oracle/ and the shared input generator) or, when the oracle's sources changed since, from a fresh computation on the
host.  Sequences of a batch are independent, so the oracle follows sequence 0 only; the other sequences of the cfg4
batch run along on the GPU (they shape the launches) and commit their own proposals.

Two policies per workload: the benchmark's fixed threshold (passes of 2 P rows, then about P + G/2) and a fixed block
size that walks the row count down through the two-row-tile regime into the one-row-tile regime.

Every pass is compared element by element: yhat, p_max, delta, and - outside the flagged band - L' and L.

What "equal" can mean at this depth.  Two correct bf16 pipelines do not agree to 2e-2 on p_max after 28-32 layers: a
last-bit difference in an fp32 sum flips a bf16 rounding, and some three hundred rounding points later the hidden state
differs by about 2 % of its norm, which on logits of RMS 15 is several tenths.  The oracle measures that effect on
itself: its records hold pass 0 twice, with bf16 rounding at the declared points and with none at all (block "exact").
The yardstick is E = oracle_bf16 - exact.  The CUDA path is held to it:
  * pass 0:  rms(gpu - exact) <= 1.5 rms(E) and max|gpu - exact| <= 2 max|E|, for p_max and for delta: the kernels sit
    as close to exact arithmetic as the oracle's own bf16 model does;
  * every pass:  max|gpu - oracle_bf16| <= 3 max|E| (two independent roundings of the same quantity);
  * an argmax may differ from the oracle's only where the oracle's own margin delta is below 2 max|E_delta|.
The measured figures are printed (pytest -s) and written to $LSP_PARITY_REPORT when set.
"""
import importlib.util
import os

import numpy as np
import pytest
import torch

import lsp_synth as S
from oracle import scan as oscan
from gpu_util import DEV

pytestmark = pytest.mark.gpu

_spec = importlib.util.spec_from_file_location(
    "make_fulldepth_oracle", os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "make_fulldepth_oracle.py"))
gold = importlib.util.module_from_spec(_spec)
_spec.loader.exec_module(gold)

RMS_FACTOR, MAX_FACTOR, PAIR_FACTOR, FLIP_FACTOR = 1.5, 2.0, 3.0, 2.0


def _rms(x):
    return float(np.sqrt(np.mean(np.square(x))))


def _sched(pol, wl, bm, tol_p, tol_d):
    from paper_2603_05454_b200 import SchedCfg
    return SchedCfg(mode=pol.get("mode", 0), fixed_k=pol.get("fixed_k", 1), tau=wl.tau, snap_window=16, l_min=1,
                    delim_bitmap=bm, flag_tol=tol_p, tie_tol=tol_d)


@pytest.mark.parametrize("name", ["cfg3", "cfg4"])
def test_full_depth_passes_teacher_forced_against_the_oracle(name):
    from paper_2603_05454_b200 import LSPDecoder
    recs_by_policy, how = gold.load_or_compute(name)
    wl = S.config(name)
    sh = wl.shape
    B, P, G = wl.batch, wl.prompt_len, wl.gen_len
    exact = recs_by_policy["exact"][0]
    ref0 = next(iter(v for k, v in recs_by_policy.items() if k != "exact"))[0]       # oracle with bf16 rounding, pass 0
    E_p, E_d = ref0["pmax"] - exact["pmax"], ref0["delta"] - exact["delta"]
    yard = dict(p_rms=_rms(E_p), p_max=float(np.abs(E_p).max()), d_rms=_rms(E_d), d_max=float(np.abs(E_d).max()),
                flips=int((ref0["yhat"] != exact["yhat"]).sum()))
    print(f"{name} yardstick (oracle bf16 - oracle exact, pass 0): p_max rms {yard['p_rms']:.3e} max {yard['p_max']:.3e}; "
          f"delta rms {yard['d_rms']:.3e} max {yard['d_max']:.3e}; argmax differs at {yard['flips']} of {len(E_p)}")
    tol_p, tol_d = PAIR_FACTOR * yard["p_max"], PAIR_FACTOR * yard["d_max"]
    tie_d = FLIP_FACTOR * yard["d_max"]
    w = S.make_weights(sh, 0, device=DEV)
    bm = S.delimiter_bitmap(sh.vocab, *wl.delim).to(DEV)
    prompts = S.make_prompt(B, P, sh, gold.PROMPT_SEED).to(DEV)
    is_delim = lambda t: wl.delim[0] <= t <= wl.delim[1]
    dec = None
    worst = dict(yardstick=yard, p=0.0, delta=0.0, flips=[], flagged=0, passes=0, rows=[], pass0=None)
    for pname, orecs in recs_by_policy.items():
        if pname == "exact":
            continue
        pol = gold.POLICIES[name][pname][0]
        sched = _sched(pol, wl, bm, tol_p, tie_d)
        if dec is None:
            dec = LSPDecoder(sh, w, sched, B, P + G, device=DEV)
        else:
            dec.set_sched(sched)
        tokens = torch.full((B, P + G), sh.mask_id, dtype=torch.int32, device=DEV)
        tokens[:, :P] = prompts
        dec.begin(tokens, [P] * B, [G] * B)
        for o in orecs:
            rec = dec.denoise_step()
            y, p, m = dec.scores()
            N0 = o["n_before"]
            assert rec[0]["n_before"] == N0 and rec[0]["rows"] == o["rows"]
            y0, p0, m0 = y[:N0], p[:N0].astype(np.float64), m[:N0].astype(np.float64)
            dp, dd = np.abs(p0 - o["pmax"]), np.abs(m0 - o["delta"])
            flips = np.nonzero(y0 != o["yhat"])[0]
            worst["p"], worst["delta"] = max(worst["p"], float(dp.max())), max(worst["delta"], float(dd.max()))
            worst["flips"] += [float(o["delta"][i]) for i in flips]
            worst["passes"] += 1
            worst["rows"].append(sum(r["rows"] for r in rec))
            print(f"{name}/{pname} pass {o['step']}: rows {sum(r['rows'] for r in rec)}, N {N0}: gpu - oracle: p_max rms "
                  f"{_rms(dp):.3e} max {dp.max():.3e}; delta rms {_rms(dd):.3e} max {dd.max():.3e}; argmax differs at "
                  f"{len(flips)} (oracle delta there up to {max([float(o['delta'][i]) for i in flips], default=0):.3f})")
            if o["step"] == 0:
                g_p, g_d = p0 - exact["pmax"], m0 - exact["delta"]
                st = dict(p_rms=_rms(g_p), p_max=float(np.abs(g_p).max()), d_rms=_rms(g_d), d_max=float(np.abs(g_d).max()),
                          flips=int((y0 != exact["yhat"]).sum()))
                print(f"{name}/{pname} pass 0: gpu - exact: p_max rms {st['p_rms']:.3e} max {st['p_max']:.3e}; delta rms "
                      f"{st['d_rms']:.3e} max {st['d_max']:.3e}; argmax differs at {st['flips']}")
                worst["pass0"] = st
                assert st["p_rms"] <= RMS_FACTOR * yard["p_rms"] and st["d_rms"] <= RMS_FACTOR * yard["d_rms"], (st, yard)
                assert st["p_max"] <= MAX_FACTOR * yard["p_max"] and st["d_max"] <= MAX_FACTOR * yard["d_max"], (st, yard)
            assert dp.max() <= tol_p, (pname, o["step"], float(dp.max()), tol_p)
            assert dd.max() <= tol_d, (pname, o["step"], float(dd.max()), tol_d)
            # an argmax may differ only where the oracle's own two largest logits are closer than the rounding noise
            assert all(o["delta"][i] <= tie_d for i in flips), ([float(o["delta"][i]) for i in flips], tie_d)
            # the oracle's decision, re-derived from its stored scores with this test's flag band
            r = oscan.lsp_scan(o["pmax"], o["yhat"], is_delim, mode=pol.get("mode", 0), fixed_k=pol.get("fixed_k", 1),
                               tau=float(np.float32(wl.tau)), W=16, l_min=1, flag_tol=float(np.float32(tol_p)),
                               tie_tol=float(np.float32(tie_d)), margin=o["delta"])
            assert (r["L_run"], r["L_commit"]) == (o["L_run"], o["L_commit"])
            near = oscan.FLAG_NEAR_THRESHOLD | oscan.FLAG_NEAR_TIE
            if r["flags"] & near or len(flips):
                worst["flagged"] += 1
            else:
                assert (rec[0]["L_run"], rec[0]["L_commit"]) == (o["L_run"], o["L_commit"]), (pname, o["step"], rec[0])
            # teacher forcing: sequence 0 commits the oracle's block and tokens, the others their own proposals
            L = [o["L_commit"]] + [rec[b]["L_commit"] for b in range(1, B)]
            dec.commit(L)
            Fp = P + G - N0
            tokens[0, Fp:Fp + o["L_commit"]] = torch.tensor(o["yhat"][:o["L_commit"]], dtype=torch.int32, device=DEV)
            torch.cuda.synchronize()
    dec.close()
    print(f"{name} ({how} oracle records): {worst['passes']} passes, rows {worst['rows']}: max|dp_max| {worst['p']:.3e}, "
          f"max|ddelta| {worst['delta']:.3e}, argmax flips {len(worst['flips'])} at oracle delta "
          f"{[round(x, 4) for x in worst['flips']]}, flagged passes {worst['flagged']}")
    out_dir = os.environ.get("LSP_PARITY_REPORT")
    if out_dir:
        os.makedirs(out_dir, exist_ok=True)
        with open(os.path.join(out_dir, f"fulldepth_{name}.txt"), "w") as f:
            f.write(repr(worst) + "\n")
