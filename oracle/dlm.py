"""Oracle: one denoiser pass p_theta(X_F, X_A; K) (Algorithm 1, the forward pass) for the transformer
shape the benchmark configurations fix (the paper treats the model as a black box): a
pre-norm bidirectional transformer with RMSNorm, rotary positions (rotate-half pairing),
multi-head / grouped-query attention without any mask, SwiGLU feed-forward, no biases and an
untied LM head.  TEST INFRASTRUCTURE, not a product path.

All arithmetic is numpy float64.  For a bf16 model the weights and the embedding arrive
already rounded to bf16 and activations are rounded (nearest-even) to bf16 at the points a
bf16 inference path materialises them: each RMSNorm output, Q/K/V after the rotation, the
attention output, every residual-stream update and the SwiGLU product.  Softmax weights and
logits are never rounded.  For an fp32 model nothing is rounded.

Pins: closed forms per op (uniform scores -> mean of V; rotation is norm-preserving and the
identity at position 0; RMSNorm of a constant vector), library routines (torch CPU
scaled-dot-product attention and rms_norm in float64), a model with zero output projections,
and the cache checks in the decode tests.
"""
import numpy as np


def round_bf16(x):
    """Round float64 -> nearest-even bfloat16, returned as float64."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


def rms_norm(x, g, eps):
    """x / sqrt(mean(x^2) + eps) * g over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def rope(x, pos, theta):
    """x: [Q, H, dh]; pos: [Q] absolute positions.  Pair (i, i + dh/2) is rotated by the angle
    pos * theta^(-2i/dh)."""
    dh = x.shape[-1]
    half = dh // 2
    inv = theta ** (-2.0 * np.arange(half, dtype=np.float64) / dh)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv[None, :]      # [Q, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def attention(q, k, v):
    """Non-causal softmax(q k^T / sqrt(dh)) v.  q: [Q, Hq, dh]; k, v: [S, Hkv, dh]; query head
    h reads key/value head h // (Hq / Hkv).  Every query sees every key."""
    Q, Hq, dh = q.shape
    S, Hkv, _ = k.shape
    grp = Hq // Hkv
    out = np.empty_like(q)
    for h in range(Hq):
        kh, vh = k[:, h // grp, :], v[:, h // grp, :]
        s = (q[:, h, :] @ kh.T) / np.sqrt(float(dh))                     # [Q, S]
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=1, keepdims=True)
        out[:, h, :] = p @ vh
    return out


def silu(x):
    return x / (1.0 + np.exp(-x))


def _f64(t):
    return np.asarray(t.float().cpu().numpy() if hasattr(t, "cpu") else t, dtype=np.float64)


class OracleDLM:
    """Holds float64 copies of the (already dtype-rounded) weights.  Linear weights are
    [out_features, in_features]."""

    def __init__(self, shape, weights, one_layer_at_a_time=False):
        """one_layer_at_a_time: weights["layers"][l] is converted to float64 when layer l runs and dropped afterwards
        (an 8B-parameter model is 64 GB in float64), and only the embedding rows a pass reads are converted.  Same
        arithmetic either way."""
        self.s = shape
        self.bf16 = (shape.dtype == "bf16")
        self.w_head = _f64(weights["w_head"])
        self.final_norm = _f64(weights["final_norm"])
        if one_layer_at_a_time:
            self.embed, self.layers, self._src = None, None, weights
        else:
            self.embed = _f64(weights["embed"])
            self.layers = [{k: _f64(v) for k, v in lw.items()} for lw in weights["layers"]]

    def layer(self, l):
        if self.layers is not None:
            return self.layers[l]
        return {k: _f64(v) for k, v in self._src["layers"][l].items()}

    def embed_rows(self, ids):
        ids = np.asarray(ids, dtype=np.int64)
        return self.embed[ids] if self.embed is not None else _f64(self._src["embed"][ids])

    def r(self, x):
        return round_bf16(x) if self.bf16 else x

    def empty_cache(self):
        s = self.s
        z = lambda: np.zeros((0, s.n_kv_heads, s.head_dim))
        return [z() for _ in range(s.n_layers)], [z() for _ in range(s.n_layers)]

    def forward(self, ids, pos, cache_k, cache_v, head_rows):
        """ids, pos: [Q] input token ids and absolute positions of this pass's rows.
        cache_k/v: per layer [F, Hkv, dh] (fixed context, not recomputed).
        Returns (logits [len(head_rows), V], k_new per layer [Q, Hkv, dh], v_new per layer)."""
        s = self.s
        Q = len(ids)
        x = self.embed_rows(ids)                                         # [Q, d]
        k_new, v_new = [], []
        for l in range(s.n_layers):
            w = self.layer(l)
            n = self.r(rms_norm(x, w["attn_norm"], s.rms_eps))
            q = (n @ w["w_q"].T).reshape(Q, s.n_heads, s.head_dim)
            k = (n @ w["w_k"].T).reshape(Q, s.n_kv_heads, s.head_dim)
            v = (n @ w["w_v"].T).reshape(Q, s.n_kv_heads, s.head_dim)
            q = self.r(rope(q, pos, s.rope_theta))
            k = self.r(rope(k, pos, s.rope_theta))
            v = self.r(v)
            k_new.append(k)
            v_new.append(v)
            k_all = np.concatenate([cache_k[l], k], axis=0)
            v_all = np.concatenate([cache_v[l], v], axis=0)
            a = self.r(attention(q, k_all, v_all)).reshape(Q, s.n_heads * s.head_dim)
            x = self.r(x + a @ w["w_o"].T)
            n2 = self.r(rms_norm(x, w["ffn_norm"], s.rms_eps))
            h = self.r(silu(n2 @ w["w_gate"].T) * (n2 @ w["w_up"].T))
            x = self.r(x + h @ w["w_down"].T)
        hn = self.r(rms_norm(x[np.asarray(head_rows, dtype=np.int64)], self.final_norm, s.rms_eps))
        return hn @ self.w_head.T, k_new, v_new
