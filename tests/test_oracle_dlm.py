"""Pins for oracle/dlm.py: closed forms, library routines (torch CPU float64) and structural cases."""
import numpy as np
import torch
import torch.nn.functional as F

import lsp_synth as S
from oracle import dlm


def test_round_bf16_matches_torch():
    x = np.random.default_rng(0).normal(size=1000) * 3
    ref = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).double().numpy()
    assert np.array_equal(dlm.round_bf16(x), ref)
    assert dlm.round_bf16(np.array([1.00390625]))[0] == 1.0      # tie -> even
    assert dlm.round_bf16(np.array([1.01171875]))[0] == 1.015625  # tie -> even (up)


def test_rms_norm_closed_form_and_library():
    x = np.full((2, 8), -3.0)
    np.testing.assert_allclose(dlm.rms_norm(x, np.ones(8), 0.0), -np.ones((2, 8)), atol=1e-15)
    rng = np.random.default_rng(3)
    x, g = rng.normal(size=(5, 32)), rng.normal(size=32)
    ref = F.rms_norm(torch.tensor(x), (32,), torch.tensor(g), 1e-5).numpy()
    np.testing.assert_allclose(dlm.rms_norm(x, g, 1e-5), ref, rtol=1e-12)


def test_rope_identity_norm_and_relative_property():
    rng = np.random.default_rng(4)
    x = rng.normal(size=(6, 2, 16))
    np.testing.assert_allclose(dlm.rope(x, np.zeros(6), 10000.0), x, atol=0)
    y = dlm.rope(x, np.arange(6) * 37, 10000.0)
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    # <rope(q,m), rope(k,n)> depends only on m - n
    q, k = rng.normal(size=(1, 1, 16)), rng.normal(size=(1, 1, 16))
    d1 = (dlm.rope(q, [5], 1e4) * dlm.rope(k, [2], 1e4)).sum()
    d2 = (dlm.rope(q, [105], 1e4) * dlm.rope(k, [102], 1e4)).sum()
    assert abs(d1 - d2) < 1e-10
    # the first pair rotates by exactly pos radians (frequency index 0 has unit frequency)
    e = np.zeros((1, 1, 16)); e[0, 0, 0] = 1.0
    r = dlm.rope(e, [1.0], 1e4)
    assert abs(r[0, 0, 0] - np.cos(1.0)) < 1e-15 and abs(r[0, 0, 8] - np.sin(1.0)) < 1e-15
    # last pair's frequency is theta^(-(dh-2)/dh)
    e = np.zeros((1, 1, 16)); e[0, 0, 7] = 1.0
    r = dlm.rope(e, [3.0], 1e4)
    assert abs(r[0, 0, 15] - np.sin(3.0 * 1e4 ** (-14 / 16))) < 1e-15


def test_attention_uniform_scores_and_library():
    rng = np.random.default_rng(5)
    v = rng.normal(size=(9, 2, 8))
    out = dlm.attention(np.zeros((3, 4, 8)), rng.normal(size=(9, 2, 8)), v)
    for h in range(4):
        np.testing.assert_allclose(out[:, h], np.tile(v[:, h // 2].mean(0), (3, 1)), atol=1e-14)
    q, k = rng.normal(size=(5, 4, 8)), rng.normal(size=(9, 2, 8))
    tq = torch.tensor(q).permute(1, 0, 2)[None]
    tk = torch.tensor(k).permute(1, 0, 2)[None].repeat_interleave(2, dim=1)
    tv = torch.tensor(v).permute(1, 0, 2)[None].repeat_interleave(2, dim=1)
    ref = F.scaled_dot_product_attention(tq, tk, tv)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(dlm.attention(q, k, v), ref, rtol=1e-10, atol=1e-12)


def _tiny(dtype="fp32", layers=2, hkv=2):
    return S.ModelShape(layers, 32, 4, hkv, 8, 64, 50, dtype=dtype, head_scale=8.0)


def test_forward_with_zero_output_projections_is_head_of_embedding():
    sh = _tiny()
    w = S.make_weights(sh, 0)
    for lw in w["layers"]:
        lw["w_o"].zero_(); lw["w_down"].zero_()
    m = dlm.OracleDLM(sh, w)
    ids = np.array([3, 7, 49, 49])
    ck, cv = m.empty_cache()
    logits, _, _ = m.forward(ids, np.arange(4), ck, cv, [2, 3])
    e = m.embed[ids[[2, 3]]]
    ref = (e / np.sqrt((e * e).mean(-1, keepdims=True) + sh.rms_eps)) @ m.w_head.T
    np.testing.assert_allclose(logits, ref, rtol=1e-12)


def test_forward_matches_torch_restatement_fp64():
    """The whole pass against library ops (torch CPU, float64): linear, rms_norm, sdpa, silu."""
    sh = _tiny(hkv=2)
    w = S.make_weights(sh, 1)
    m = dlm.OracleDLM(sh, w)
    ids = np.array([1, 2, 3, 49, 49, 49]); Q = len(ids)
    ck, cv = m.empty_cache()
    logits, k_new, v_new = m.forward(ids, np.arange(Q) + 4, ck, cv, [3, 4, 5])
    T = lambda a: torch.tensor(np.asarray(a), dtype=torch.float64)
    x = T(m.embed)[torch.tensor(ids)]
    half = sh.head_dim // 2
    inv = sh.rope_theta ** (-torch.arange(half, dtype=torch.float64) * 2 / sh.head_dim)
    ang = (torch.arange(Q, dtype=torch.float64) + 4)[:, None] * inv
    cos, sin = torch.cat([ang.cos(), ang.cos()], -1)[:, None], torch.cat([ang.sin(), ang.sin()], -1)[:, None]
    rot = lambda t: t * cos + torch.cat([-t[..., half:], t[..., :half]], -1) * sin
    for l, lw in enumerate(m.layers):
        n = F.rms_norm(x, (sh.d_model,), T(lw["attn_norm"]), sh.rms_eps)
        q = rot(F.linear(n, T(lw["w_q"])).view(Q, sh.n_heads, sh.head_dim))
        k = rot(F.linear(n, T(lw["w_k"])).view(Q, sh.n_kv_heads, sh.head_dim))
        v = F.linear(n, T(lw["w_v"])).view(Q, sh.n_kv_heads, sh.head_dim)
        np.testing.assert_allclose(k_new[l], k.numpy(), rtol=1e-9, atol=1e-12)
        g = sh.n_heads // sh.n_kv_heads
        a = F.scaled_dot_product_attention(q.permute(1, 0, 2)[None],
                                           k.permute(1, 0, 2)[None].repeat_interleave(g, 1),
                                           v.permute(1, 0, 2)[None].repeat_interleave(g, 1))[0]
        x = x + F.linear(a.permute(1, 0, 2).reshape(Q, -1), T(lw["w_o"]))
        n2 = F.rms_norm(x, (sh.d_model,), T(lw["ffn_norm"]), sh.rms_eps)
        x = x + F.linear(F.silu(F.linear(n2, T(lw["w_gate"]))) * F.linear(n2, T(lw["w_up"])), T(lw["w_down"]))
    ref = F.linear(F.rms_norm(x[3:], (sh.d_model,), T(m.final_norm), sh.rms_eps), T(m.w_head))
    np.testing.assert_allclose(logits, ref.numpy(), rtol=1e-9, atol=1e-11)


def test_bf16_mode_rounds_at_declared_points():
    sh = _tiny(dtype="bf16")
    w = S.make_weights(sh, 2)
    m = dlm.OracleDLM(sh, w)
    ck, cv = m.empty_cache()
    _, k_new, v_new = m.forward(np.array([1, 2, 49]), np.arange(3), ck, cv, [2])
    for a in k_new + v_new:
        assert np.array_equal(a, dlm.round_bf16(a))


def test_bf16_mode_rounding_points_are_exactly_the_declared_ones(monkeypatch):
    """One forward pass of a bf16 model, with every call of the rounding hook recorded and the inputs of the norm and
    attention routines captured.  Declared points, per layer: norm output, Q, K, V (after the rotation), attention
    output, residual update, second norm output, SwiGLU product, second residual update; then the final norm.  Logits
    and softmax weights stay unrounded.  A dropped (or added) rounding changes the recorded sequence."""
    sh = _tiny(dtype="bf16")
    sh.n_layers = 2
    m = dlm.OracleDLM(sh, S.make_weights(sh, 2))
    Q, head_rows = 5, [2, 4]
    is_bf16 = lambda a: np.array_equal(a, dlm.round_bf16(a))
    calls = []
    orig_r = m.r
    m.r = lambda x: calls.append((np.shape(x), is_bf16(x))) or orig_r(x)
    seen = {"norm_in": [], "attn_in": []}
    o_norm, o_attn = dlm.rms_norm, dlm.attention
    monkeypatch.setattr(dlm, "rms_norm", lambda x, g, e: seen["norm_in"].append(is_bf16(x)) or o_norm(x, g, e))
    monkeypatch.setattr(dlm, "attention",
                        lambda q, k, v: seen["attn_in"].append(is_bf16(q) and is_bf16(k) and is_bf16(v)) or o_attn(q, k, v))
    ck, cv = m.empty_cache()
    logits, k_new, v_new = m.forward(np.array([1, 2, 49, 7, 49]), np.arange(Q), ck, cv, head_rows)
    d, f = sh.d_model, sh.d_ffn
    hq, hkv, dh = sh.n_heads, sh.n_kv_heads, sh.head_dim
    per_layer = [(Q, d), (Q, hq, dh), (Q, hkv, dh), (Q, hkv, dh), (Q, hq, dh), (Q, d), (Q, d), (Q, f), (Q, d)]
    assert [c[0] for c in calls] == per_layer * sh.n_layers + [(len(head_rows), d)]
    assert not any(c[1] for c in calls)                   # every rounding did something: its input was not bf16 yet
    assert all(seen["norm_in"]) and len(seen["norm_in"]) == 2 * sh.n_layers + 1     # residual stream is bf16 at every norm
    assert all(seen["attn_in"]) and len(seen["attn_in"]) == sh.n_layers             # Q, K, V are bf16 when attention reads them
    assert not is_bf16(logits)                            # logits are accumulators, never rounded
    for a in k_new + v_new:
        assert is_bf16(a)
    # softmax weights are not rounded: attention() never reaches the rounding routine
    def boom(x):
        raise AssertionError("attention rounded something")
    monkeypatch.setattr(dlm, "round_bf16", boom)
    rng = np.random.default_rng(0)
    o_attn(rng.normal(size=(3, hq, dh)), rng.normal(size=(4, hkv, dh)), rng.normal(size=(4, hkv, dh)))


def test_fp32_mode_rounds_nothing():
    sh = _tiny(dtype="fp32")
    m = dlm.OracleDLM(sh, S.make_weights(sh, 2))
    ck, cv = m.empty_cache()
    x = np.random.default_rng(1).normal(size=(3, 7))
    assert m.r(x) is x


def test_one_layer_at_a_time_mode_is_the_same_arithmetic():
    sh = _tiny(dtype="bf16")
    w = S.make_weights(sh, 3)
    a, b = dlm.OracleDLM(sh, w), dlm.OracleDLM(sh, w, one_layer_at_a_time=True)
    ids, pos = np.array([5, 9, 49, 49]), np.arange(4) + 3
    ck, cv = a.empty_cache()
    la, ka, va = a.forward(ids, pos, ck, cv, [2, 3])
    lb, kb, vb = b.forward(ids, pos, ck, cv, [2, 3])
    assert np.array_equal(la, lb) and all(np.array_equal(x, y) for x, y in zip(ka + va, kb + vb))
