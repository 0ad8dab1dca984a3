"""lsp_linear_static: the GEMM entry point for callers that may not allocate device memory (its scratch is a static
array inside the library).  Collected last on purpose: a failure here cannot hide the other tests' results."""
import numpy as np
import pytest
import torch

import lsp_synth as S
from gpu_util import DEV

pytestmark = pytest.mark.gpu


def _reference(A, W):
    """The same product through the existing entry point (lsp_op_linear with a context and a caller workspace)."""
    from paper_2603_05454_b200 import LSPDecoder, SchedCfg
    sh = S.ModelShape(1, 64, 1, 1, 64, 64, 128, dtype="bf16")
    dec = LSPDecoder(sh, S.make_weights(sh, 0, device=DEV), SchedCfg(), 1, 8, device=DEV)
    out = torch.empty(A.shape[0], W.shape[0], dtype=torch.bfloat16, device=DEV)
    dec.op_linear(0, A, W, None, out)
    dec.close()
    return out


# the last four reach the paths the large shapes do not: one weight row group narrower than a TMA box and a single
# one-atom K chunk; a ragged last column tile; K not a multiple of 128; more column tiles than CTAs, so that a CTA's
# share of the (tile, K chunk) units starts and ends in the middle of a tile
@pytest.mark.parametrize("shape", [(37, 4096, 4096), (128, 1152, 512), (3, 12288, 4096),
                                   (1, 16, 64), (5, 144, 192), (128, 2064, 320), (8, 8320, 256)])
def test_static_scratch_gemm_matches_workspace_gemm_twice_in_a_row(shape):
    """Two calls in a row (the second finds the first call's leftovers in the static array), each checked against the
    existing entry point and against the fp64 product of the same bf16 inputs rounded to bf16."""
    from paper_2603_05454_b200 import linear_static
    from oracle.dlm import round_bf16
    M, N, K = shape
    W = S.normal((N, K), 5, 2, 0.05, torch.bfloat16, DEV)
    out = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    for call in range(2):
        A = S.normal((M, K), 5 + call, 1, 1.0, torch.bfloat16, DEV)
        ref = _reference(A, W).float().cpu().numpy()
        exact = f64(A) @ f64(W).T
        out.fill_(float("nan"))
        linear_static(A, W, out)
        torch.cuda.synchronize()
        got = out.float().cpu().numpy()
        rtol = 1.0 / 128                                # one bf16 ulp: the two paths sum their K slices in different orders
        atol = rtol * np.abs(exact).max() * 0.05
        np.testing.assert_allclose(got, ref, rtol=rtol, atol=atol)
        np.testing.assert_allclose(got, round_bf16(exact), rtol=rtol, atol=atol)


def test_static_scratch_gemm_rejects_sizes_beyond_its_limits():
    from paper_2603_05454_b200 import linear_static, LSPError
    A = torch.zeros(129, 128, dtype=torch.bfloat16, device=DEV)
    W = torch.zeros(64, 128, dtype=torch.bfloat16, device=DEV)
    out = torch.zeros(129, 64, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(LSPError) as e:
        linear_static(A, W, out)                        # M > 128
    assert e.value.code == -2 and "limits" in str(e.value)
    with pytest.raises(LSPError):
        linear_static(A[:4, :96].contiguous(), W[:, :96].contiguous(), out[:4])     # K not a multiple of 64
