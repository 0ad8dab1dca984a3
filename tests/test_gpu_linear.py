"""K3 parity: the GEMM kernels with their fused epilogues against fp64 matrix products."""
import numpy as np
import pytest
import torch

import lsp_synth as S
from oracle import dlm
from gpu_util import DEV

pytestmark = pytest.mark.gpu


def _dec(dtype):
    from paper_2603_05454_b200 import LSPDecoder, SchedCfg
    sh = S.ModelShape(1, 64, 1, 1, 64, 64, 128, dtype=dtype)
    return LSPDecoder(sh, S.make_weights(sh, 0, device=DEV), SchedCfg(), 1, 8, device=DEV)


def _check(dtype, impl, M, N, K, seed):
    tdt = torch.float32 if dtype == "fp32" else torch.bfloat16
    dec = _dec(dtype)
    dec.set_option(0, impl)
    A = S.normal((M, K), seed, 1, 1.0, tdt, DEV)
    W = S.normal((N, K), seed, 2, 0.05, tdt, DEV)
    W2 = S.normal((N, K), seed, 3, 0.05, tdt, DEV)
    X0 = S.normal((M, N), seed, 4, 1.0, tdt, DEV)
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    rnd = dlm.round_bf16 if dtype == "bf16" else (lambda x: x.astype(np.float32).astype(np.float64))
    a, w, w2, x0 = f64(A), f64(W), f64(W2), f64(X0)
    rtol = 2e-5 if dtype == "fp32" else 1.0 / 128   # one bf16 ulp of the result (rounding point may flip)
    out = torch.empty(M, N, dtype=tdt, device=DEV)
    dec.op_linear(0, A, W, None, out)
    ref = a @ w.T
    np.testing.assert_allclose(f64(out), rnd(ref), rtol=rtol, atol=rtol * np.abs(ref).max() * 0.05)
    xr = X0.clone()
    dec.op_linear(1, A, W, None, xr)
    ref = x0 + a @ w.T
    np.testing.assert_allclose(f64(xr), rnd(ref), rtol=rtol, atol=rtol * np.abs(ref).max() * 0.05)
    dec.op_linear(2, A, W, W2, out)
    g, u = a @ w.T, a @ w2.T
    ref = g / (1 + np.exp(-g)) * u
    np.testing.assert_allclose(f64(out), rnd(ref), rtol=rtol * 2, atol=rtol * np.abs(ref).max() * 0.05)
    dec.close()


@pytest.mark.parametrize("shape", [(1, 64, 64), (70, 144, 192), (129, 256, 128), (300, 512, 1024)])
def test_linear_fp32(shape):
    _check("fp32", 0, *shape, seed=0)


@pytest.mark.parametrize("impl", [0, 1])
@pytest.mark.parametrize("shape", [(1, 64, 64), (70, 144, 192), (129, 256, 128), (300, 512, 1024),
                                   (512, 4096, 4096), (37, 12288, 4096), (257, 4096, 12288)])
def test_linear_bf16(impl, shape):
    _check("bf16", impl, *shape, seed=1)


@pytest.mark.parametrize("grid_mode", [1, 2])
@pytest.mark.parametrize("shape", [(1, 256, 128), (5, 384, 256), (64, 1152, 512), (128, 4096, 4096), (100, 12288, 4096),
                                   (17, 4096, 12288), (129, 384, 256), (200, 4096, 4096), (256, 12288, 4096),
                                   (190, 1152, 576)])
def test_linear_bf16_weight_streaming_kernel(grid_mode, shape):
    """M <= 256 takes the persistent streaming kernel (one or two row tiles per CTA): tiles split between CTAs
    (partials in scratch, summed by the last arriver) with both ways of dealing out the work."""
    M, N, K = shape
    tdt = torch.bfloat16
    dec = _dec("bf16")
    dec.debug_set(17, grid_mode)
    A = S.normal((M, K), 2, 1, 1.0, tdt, DEV)
    W = S.normal((N, K), 2, 2, 0.05, tdt, DEV)
    W2 = S.normal((N, K), 2, 3, 0.05, tdt, DEV)
    X0 = S.normal((M, N), 2, 4, 1.0, tdt, DEV)
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    a, w, w2, x0 = f64(A), f64(W), f64(W2), f64(X0)
    rtol = 1.0 / 128
    out = torch.empty(M, N, dtype=tdt, device=DEV)
    outs = []
    for rep in range(2):                       # twice: the tile counters must be back at zero after a launch
        dec.op_linear(0, A, W, None, out)
        ref = a @ w.T
        np.testing.assert_allclose(f64(out), dlm.round_bf16(ref), rtol=rtol, atol=rtol * np.abs(ref).max() * 0.05)
        outs.append(out.clone())
    assert torch.equal(outs[0], outs[1])       # deterministic summation order
    xr = X0.clone()
    dec.op_linear(1, A, W, None, xr)
    ref = x0 + a @ w.T
    np.testing.assert_allclose(f64(xr), dlm.round_bf16(ref), rtol=rtol, atol=rtol * np.abs(ref).max() * 0.05)
    dec.op_linear(2, A, W, W2, out)
    g, u = a @ w.T, a @ w2.T
    ref = g / (1 + np.exp(-g)) * u
    np.testing.assert_allclose(f64(out), dlm.round_bf16(ref), rtol=rtol * 2, atol=rtol * np.abs(ref).max() * 0.05)
    dec.close()


@pytest.mark.parametrize("case", [
    # (M, N, K, options): 256 x 256 tiles whose K slices run as one cluster; the fp32 partial tile (256 KB) is larger
    # than the pipeline's shared memory, so it is reduced one row tile at a time
    (200, 4096, 4096, {20: 256}), (256, 12288, 4096, {20: 256}), (130, 4096, 12288, {20: 256}),
    (640, 4096, 12288, {}), (1000, 3584, 3584, {}), (300, 2048, 1024, {}), (257, 512, 2048, {}),
    (640, 4096, 4096, {29: 0}),
    (640, 4096, 12288, {33: 0}), (200, 12288, 1024, {20: 256, 33: 0}),      # clusters of 2 without the half-tile exchange
    # SwiGLU GEMM with 192-wide tiles (96 pairs): one and two row tiles, several row groups, a forced 256 for contrast
    (100, 12288, 256, {}), (200, 12288, 320, {}), (600, 12288, 256, {32: 192}), (100, 12288, 256, {32: 256}),
    (300, 9600, 192, {32: 192}),
])
def test_linear_bf16_cluster_split_of_two_row_tiles(case):
    M, N, K, opts = case
    tdt = torch.bfloat16
    dec = _dec("bf16")
    for k, v in opts.items():
        dec.debug_set(k, v)
    A = S.normal((M, K), 3, 1, 1.0, tdt, DEV)
    W = S.normal((N, K), 3, 2, 0.05, tdt, DEV)
    W2 = S.normal((N, K), 3, 3, 0.05, tdt, DEV)
    X0 = S.normal((M, N), 3, 4, 1.0, tdt, DEV)
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    a, w, w2, x0 = f64(A), f64(W), f64(W2), f64(X0)
    rtol = 1.0 / 128
    out = torch.empty(M, N, dtype=tdt, device=DEV)
    outs = []
    for rep in range(2):
        dec.op_linear(0, A, W, None, out)
        ref = a @ w.T
        np.testing.assert_allclose(f64(out), dlm.round_bf16(ref), rtol=rtol, atol=rtol * np.abs(ref).max() * 0.05)
        outs.append(out.clone())
    assert torch.equal(outs[0], outs[1])       # rank-order summation: the same bits every time
    xr = X0.clone()
    dec.op_linear(1, A, W, None, xr)
    ref = x0 + a @ w.T
    np.testing.assert_allclose(f64(xr), dlm.round_bf16(ref), rtol=rtol, atol=rtol * np.abs(ref).max() * 0.05)
    dec.op_linear(2, A, W, W2, out)
    g, u = a @ w.T, a @ w2.T
    ref = g / (1 + np.exp(-g)) * u
    np.testing.assert_allclose(f64(out), dlm.round_bf16(ref), rtol=rtol * 2, atol=rtol * np.abs(ref).max() * 0.05)
    dec.close()


def test_linear_bf16_seeded_random_shapes_and_kernel_options():
    """Sixty seeded random (rows, columns, K, option) combinations across the row regimes (one tile, two tiles, row
    groups), the split paths (clusters of 2..8, half-tile exchange, rounds, global scratch), the tile widths, and the
    operand-swapped kernel forced on."""
    import random
    rng = random.Random(7)
    dec = _dec("bf16")
    defaults = {29: 1, 33: 1, 20: 0, 23: 0, 32: 0, 17: 2, 24: 3, 36: 129, 38: 0}
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    rows = [1, 2, 5, 17, 32, 33, 64, 100, 128, 129, 190, 256, 257, 300, 400, 512, 640, 768, 1000, 1100, 1536, 2100]
    done = 0
    while done < 60:
        M, N, K = rng.choice(rows), rng.choice([96, 128, 384, 1152, 2048, 3584, 4096, 4608, 9600, 12288]), \
            rng.choice([64, 192, 320, 1024, 2048, 3584, 4096])
        if M * N * K > 2e10:
            continue
        opts = {}
        for key, p, vals in ((29, 0.2, [0]), (33, 0.2, [0]), (20, 0.15, [128, 256]), (23, 0.15, [128, 256]),
                             (32, 0.15, [192, 256]), (17, 0.1, [1]), (24, 0.1, [1, 2]), (38, 0.3, [1])):
            if rng.random() < p:
                opts[key] = rng.choice(vals)
        if opts.get(38):
            opts[36] = 1                    # the operand-swapped kernel at every row count up to 256, on any shape it can run
        for k, v in {**defaults, **opts}.items():
            dec.debug_set(k, v)
        A = S.normal((M, K), done, 1, 1.0, torch.bfloat16, DEV)
        W = S.normal((N, K), done, 2, 0.05, torch.bfloat16, DEV)
        W2 = S.normal((N, K), done, 3, 0.05, torch.bfloat16, DEV)
        X0 = S.normal((M, N), done, 4, 1.0, torch.bfloat16, DEV)
        a, w, w2, x0 = f64(A), f64(W), f64(W2), f64(X0)
        rtol = 1.0 / 128
        out = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
        tag = f"M={M} N={N} K={K} options={opts}"
        dec.op_linear(0, A, W, None, out)
        ref = a @ w.T
        np.testing.assert_allclose(f64(out), dlm.round_bf16(ref), rtol=rtol, atol=rtol * np.abs(ref).max() * 0.05, err_msg=tag)
        xr = X0.clone()
        dec.op_linear(1, A, W, None, xr)
        ref = x0 + a @ w.T
        np.testing.assert_allclose(f64(xr), dlm.round_bf16(ref), rtol=rtol, atol=rtol * np.abs(ref).max() * 0.05, err_msg=tag)
        dec.op_linear(2, A, W, W2, out)
        g, u = a @ w.T, a @ w2.T
        ref = g / (1 + np.exp(-g)) * u
        np.testing.assert_allclose(f64(out), dlm.round_bf16(ref), rtol=rtol * 2, atol=rtol * np.abs(ref).max() * 0.05, err_msg=tag)
        done += 1
    dec.close()


def test_bounded_wait_expiry_is_reported_and_the_context_stays_usable():
    """A device-side wait that runs out (a barrier nothing arrives at, 200 microseconds) comes back as
    LSP_ERR_DEVICE_TIMEOUT with the site in the message; the status word is cleared, and the next GEMM is correct."""
    from paper_2603_05454_b200 import LSPError
    dec = _dec("bf16")
    A = S.normal((70, 192), 3, 1, 1.0, torch.bfloat16, DEV)
    W = S.normal((144, 192), 3, 2, 0.05, torch.bfloat16, DEV)
    out = torch.empty(70, 144, dtype=torch.bfloat16, device=DEV)
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    ref = dlm.round_bf16(f64(A) @ f64(W).T)
    for _ in range(2):
        with pytest.raises(LSPError) as e:
            dec.wait_selftest(200)
        assert e.value.code == -6 and "site 99" in str(e.value)
        dec.op_linear(0, A, W, None, out)               # synchronises and checks the status word: must be clean again
        np.testing.assert_allclose(f64(out), ref, rtol=1.0 / 128, atol=np.abs(ref).max() / 128 * 0.05)
    dec.close()


@pytest.mark.parametrize("M", [1, 48, 128, 200, 256, 384, 640, 1500])
def test_linear_bf16_third_model_shape(M):
    """A model shape none of the tile heuristics were fitted on (d 5120, 40/8 heads of 128, FFN 13824): the fused QKV
    width 7168, the O and down projections, the SwiGLU pair GEMM, at row counts of every regime."""
    dec = _dec("bf16")
    d, qd, kvd, f = 5120, 40 * 128, 8 * 128, 13824
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    rtol = 1.0 / 128
    for (N, K, op) in ((qd + 2 * kvd, d, 0), (d, qd, 1), (f, d, 2), (d, f, 1)):
        A = S.normal((M, K), 5, 1, 1.0, torch.bfloat16, DEV)
        W = S.normal((N, K), 5, 2, 0.03, torch.bfloat16, DEV)
        W2 = S.normal((N, K), 5, 3, 0.03, torch.bfloat16, DEV) if op == 2 else None
        out = S.normal((M, N), 5, 4, 1.0, torch.bfloat16, DEV)
        x0 = f64(out)
        dec.op_linear(op, A, W, W2, out)
        a, w = f64(A), f64(W)
        if op == 0:
            ref = a @ w.T
        elif op == 1:
            ref = x0 + a @ w.T
        else:
            g, u = a @ w.T, a @ f64(W2).T
            ref = g / (1 + np.exp(-g)) * u
        np.testing.assert_allclose(f64(out), dlm.round_bf16(ref), rtol=rtol * (2 if op == 2 else 1),
                                   atol=rtol * np.abs(ref).max() * 0.05, err_msg=f"M={M} N={N} K={K} op={op}")
    dec.close()


@pytest.mark.parametrize("M", [1, 16, 17, 100, 129, 144, 177, 200, 256])
def test_linear_bf16_operand_swapped_kernel(M):
    """The operand-swapped kernel (weights as the 128-row MMA operand, activation rows as N in steps of 16), forced on for
    every row count up to 256: one and two accumulators, K slices on clusters of 1, 2 and 4, ragged last tiles, all three
    epilogues, twice (bit-identical: the K slices are summed in rank order)."""
    dec = _dec("bf16")
    dec.debug_set(36, 1)
    dec.debug_set(37, 256)
    dec.debug_set(38, 1)
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    rtol = 1.0 / 128
    for (N, K) in ((4096, 4096), (12288, 4096), (1152, 512), (384, 256), (3584, 18944), (4608, 3584), (144, 192)):
        A = S.normal((M, K), 7, 1, 1.0, torch.bfloat16, DEV)
        W = S.normal((N, K), 7, 2, 0.03, torch.bfloat16, DEV)
        W2 = S.normal((N, K), 7, 3, 0.03, torch.bfloat16, DEV)
        X0 = S.normal((M, N), 7, 4, 1.0, torch.bfloat16, DEV)
        a, w, w2, x0 = f64(A), f64(W), f64(W2), f64(X0)
        tag = f"M={M} N={N} K={K}"
        out = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
        outs = []
        for _ in range(2):
            out.fill_(float("nan"))
            dec.op_linear(0, A, W, None, out)
            ref = a @ w.T
            np.testing.assert_allclose(f64(out), dlm.round_bf16(ref), rtol=rtol, atol=rtol * np.abs(ref).max() * 0.05, err_msg=tag)
            outs.append(out.clone())
        assert torch.equal(outs[0], outs[1]), tag
        xr = X0.clone()
        dec.op_linear(1, A, W, None, xr)
        ref = x0 + a @ w.T
        np.testing.assert_allclose(f64(xr), dlm.round_bf16(ref), rtol=rtol, atol=rtol * np.abs(ref).max() * 0.05, err_msg=tag)
        dec.op_linear(2, A, W, W2, out)
        g, u = a @ w.T, a @ w2.T
        ref = g / (1 + np.exp(-g)) * u
        np.testing.assert_allclose(f64(out), dlm.round_bf16(ref), rtol=rtol * 2, atol=rtol * np.abs(ref).max() * 0.05, err_msg=tag)
    dec.close()


@pytest.mark.parametrize("case", [(130, 12288, 256, {}), (150, 12288, 320, {}), (192, 12288, 256, {}), (177, 9600, 192, {}),
                                  (160, 12288, 256, {32: 256}), (193, 12288, 256, {}), (150, 12288, 256, {39: 0}),
                                  (140, 12288, 512, {37: 0})])
def test_linear_bf16_second_row_tile_of_64_rows(case):
    """129..192 rows on two row tiles with unsplit tiles (the SwiGLU GEMM of a wide FFN): the second row tile runs 64-row
    MMAs, whose accumulator rows sit in the lower half of every warp's tensor-memory lanes.  Also the neighbouring cases
    that must not take that path (193 rows; the option off; plain epilogues with the operand-swapped kernel off)."""
    M, N, K, opts = case
    dec = _dec("bf16")
    for k, v in opts.items():
        dec.debug_set(k, v)
    A = S.normal((M, K), 9, 1, 1.0, torch.bfloat16, DEV)
    W = S.normal((N, K), 9, 2, 0.05, torch.bfloat16, DEV)
    W2 = S.normal((N, K), 9, 3, 0.05, torch.bfloat16, DEV)
    X0 = S.normal((M, N), 9, 4, 1.0, torch.bfloat16, DEV)
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    a, w, w2, x0 = f64(A), f64(W), f64(W2), f64(X0)
    rtol = 1.0 / 128
    out = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=DEV)
    dec.op_linear(2, A, W, W2, out)
    g, u = a @ w.T, a @ w2.T
    ref = g / (1 + np.exp(-g)) * u
    np.testing.assert_allclose(f64(out), dlm.round_bf16(ref), rtol=rtol * 2, atol=rtol * np.abs(ref).max() * 0.05)
    out.fill_(float("nan"))
    dec.op_linear(0, A, W, None, out)
    ref = a @ w.T
    np.testing.assert_allclose(f64(out), dlm.round_bf16(ref), rtol=rtol, atol=rtol * np.abs(ref).max() * 0.05)
    xr = X0.clone()
    dec.op_linear(1, A, W, None, xr)
    ref = x0 + a @ w.T
    np.testing.assert_allclose(f64(xr), dlm.round_bf16(ref), rtol=rtol, atol=rtol * np.abs(ref).max() * 0.05)
    dec.close()
