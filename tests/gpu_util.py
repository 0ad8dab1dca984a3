"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

import lsp_synth as S
from oracle import dlm, scan as oscan
from oracle.decode import decode, make_is_delim

DEV = "cuda:0"


def tol_for(dtype):
    return 1e-4 if dtype == "fp32" else 2e-2


def make_pair(shape, seed):
    """Weights on the GPU (for the library) and the oracle model built from the CPU copy of the same values."""
    w_gpu = S.make_weights(shape, seed, device=DEV)
    w_cpu = S.make_weights(shape, seed, device="cpu")
    return w_gpu, dlm.OracleDLM(shape, w_cpu)


def oracle_policy(s, flag_tol):
    """kwargs of oracle.scan.lsp_scan that mirror a binding SchedCfg (thresholds as the fp32 values the GPU sees)."""
    return dict(mode=s.mode, tau=float(np.float32(s.tau)), alpha=float(np.float32(s.alpha)),
                beta=float(np.float32(s.beta)), l_min=s.l_min, W=s.snap_window, fixed_k=s.fixed_k, flag_tol=flag_tol)
