"""K5 (+K6) parity: fused LM head + confidence reduction against the oracle's full-vocabulary scores."""
import numpy as np
import pytest
import torch

import lsp_synth as S
from oracle import scan as oscan
from oracle.scores import scores_from_logits
from gpu_util import DEV, tol_for, tol_logit

pytestmark = pytest.mark.gpu


def _run(dtype, d, V, lens, head_scale, tau, seed=0, exclude=1, impl=None):
    from paper_2603_05454_b200 import LSPDecoder, SchedCfg
    sh = S.ModelShape(1, d, max(1, d // 64), max(1, d // 64), 64, 64, V, dtype=dtype, head_scale=head_scale)
    w = {"embed": torch.zeros(V, d, dtype=torch.float32 if dtype == "fp32" else torch.bfloat16, device=DEV)}
    tdt = w["embed"].dtype
    w["w_head"] = S.normal((V, d), seed, S.TID_HEAD, sh.w_std * head_scale, tdt, DEV)
    w["final_norm"] = torch.ones(d, dtype=tdt, device=DEV)
    z = lambda *s: torch.zeros(*s, dtype=tdt, device=DEV)
    w["layers"] = [dict(attn_norm=z(d), w_qkv=z(3 * d, d), w_o=z(d, d), ffn_norm=z(d), w_gate=z(64, d), w_up=z(64, d),
                        w_down=z(d, 64))]
    rows = int(sum(lens))
    bm = S.delimiter_bitmap(V, 1, 32).to(DEV)
    tol = tol_for(dtype)
    # oracle: full logits in fp64 from the same (dtype-rounded) values
    hidden = S.normal((rows, d), seed, 77, 1.0, tdt, DEV)
    h64 = hidden.float().cpu().numpy().astype(np.float64)
    w64 = w["w_head"].float().cpu().numpy().astype(np.float64)
    logits = h64 @ w64.T
    # inputs are identical on both sides here, so only accumulation order differs: fp32 accumulation of d
    # products of magnitude ~z_rms/sqrt(d) keeps logits within 1e-4 * z_rms even in bf16
    tol_z = tol_logit("fp32", float(np.sqrt((logits * logits).mean())))
    sched = SchedCfg(tau=tau, delim_bitmap=bm, exclude_mask_logit=exclude, flag_tol=tol, tie_tol=tol_z)
    dec = LSPDecoder(sh, w, sched, len(lens), max(2, max(lens)), device=DEV)
    if impl is not None:
        dec.set_option(0, impl)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    out = dec.head_scan(hidden, off)
    y, p, m = dec.scores()
    dec.close()
    yo, po, mo = scores_from_logits(logits, sh.mask_id if exclude else -1)
    assert np.abs(p - po).max() <= 1e-4
    assert np.abs(m - mo).max() <= tol_z
    bad = np.nonzero(y != yo)[0]
    assert all(mo[i] <= tol_z for i in bad), "argmax differs away from a near-tie"
    n_flag = 0
    for b in range(len(lens)):
        a, e = off[b], off[b + 1]
        if e == a:
            continue
        r = oscan.lsp_scan(po[a:e], yo[a:e], lambda t: 1 <= t <= 32, tau=float(np.float32(tau)), W=16,
                           flag_tol=float(np.float32(tol)), tie_tol=float(np.float32(tol_z)), margin=mo[a:e])
        if r["flags"] & (oscan.FLAG_NEAR_THRESHOLD | oscan.FLAG_NEAR_TIE):
            n_flag += 1
            continue
        assert (out["L_run"][b], out["L_commit"][b]) == (r["L_run"], r["L_commit"]), (b, out, r)
    return n_flag


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_head_small_shapes_span_tiles_and_ragged_tails(dtype):
    # vocab not a multiple of any tile width, rows not a multiple of the row tile
    _run(dtype, 256, 2048, [64, 1, 130, 5], head_scale=30.0, tau=0.3)
    _run(dtype, 128, 1000, [3, 200], head_scale=40.0, tau=0.2, seed=1)
    _run(dtype, 256, 4099, [257], head_scale=30.0, tau=0.3, seed=2, exclude=0)


@pytest.mark.parametrize("impl", [0, 1])
def test_head_bf16_wide_model_both_gemm_paths(impl):
    _run("bf16", 4096, 8192, [100, 300], head_scale=5.0, tau=0.5, seed=3, impl=impl)


def test_head_all_equal_rows_pick_lowest_id():
    from paper_2603_05454_b200 import LSPDecoder, SchedCfg
    d, V = 64, 512
    sh = S.ModelShape(1, d, 1, 1, 64, 64, V, dtype="fp32", mask_id=0)
    z = lambda *s: torch.zeros(*s, device=DEV)
    w = dict(embed=z(V, d), w_head=z(V, d), final_norm=torch.ones(d, device=DEV),
             layers=[dict(attn_norm=z(d), w_qkv=z(3 * d, d), w_o=z(d, d), ffn_norm=z(d), w_gate=z(64, d),
                          w_up=z(64, d), w_down=z(d, 64))])
    dec = LSPDecoder(sh, w, SchedCfg(tau=0.0), 1, 8, device=DEV)
    dec.head_scan(torch.ones(5, d, device=DEV), [0, 5])
    y, p, m = dec.scores()
    assert (y == 1).all() and (m == 0).all() and np.allclose(p, 1.0 / (V - 1), rtol=1e-5)
    dec.close()
