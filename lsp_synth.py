"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests/bench.

This module holds no arithmetic of the decoding method. It only defines a counter-based
generator: element ``i`` of tensor ``tensor_id`` under ``seed`` is a pure function of
``(seed, tensor_id, i)``, evaluated with integer operations that give the same bits on
every device torch runs on, so a tensor made on the GPU and one made on the CPU are equal.

Recipe
------
* ``key = seed * G + tensor_id * T + i`` (wrapping 64-bit), ``G = 0x9E3779B97F4A7C15``,
  ``T = 0xD1B54A32D192ED03``.
* ``h1 = mix(key + G)``, ``h2 = mix(key + 2G)`` with the splitmix64 finaliser ``mix``.
* Approximate standard normal: the eight 16-bit lanes of ``h1, h2`` are summed (an
  Irwin-Hall variate with n = 8: mean 262140, variance 8 * (65536**2 - 1) / 12), centred
  and scaled in one fp32 multiply.  Support is about +-4.9 sigma, excess kurtosis -0.15.
  No transcendental function is used, so there is no libm dependence.
* Uniform integers: ``(h1 >>> 32) mod n``.

Tensors are indexed in their *logical* row-major shape (e.g. a linear layer's weight is
``[out_features, in_features]``), independent of any storage layout a consumer picks.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, Tuple

import torch

_M64 = (1 << 64) - 1
_G = 0x9E3779B97F4A7C15
_T = 0xD1B54A32D192ED03
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB
_IH_MEAN = 8 * 65535 // 2  # 262140
_IH_SIGMA = math.sqrt(8 * (65536 ** 2 - 1) / 12.0)
_CHUNK = 1 << 25


def _s64(x: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant as a Python int in int64 range."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift on int64 (torch's >> is arithmetic)."""
    return torch.bitwise_and(torch.bitwise_right_shift(x, s), (1 << (64 - s)) - 1)


def _mix(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _s64(_C1)
    z = (z ^ _lsr(z, 27)) * _s64(_C2)
    return z ^ _lsr(z, 31)


def _keys(seed: int, tensor_id: int, start: int, n: int, device) -> torch.Tensor:
    base = _s64(seed * _G + tensor_id * _T + start)
    return torch.arange(n, dtype=torch.int64, device=device) + base


def _lanes16(h: torch.Tensor) -> torch.Tensor:
    return (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + _lsr(h, 48)


def normal(shape, seed: int, tensor_id: int, scale: float = 1.0, dtype=torch.float32,
           device="cpu") -> torch.Tensor:
    """Approximately N(0, scale^2) values, rounded (nearest-even) to ``dtype`` last."""
    n = int(math.prod(shape)) if len(shape) else 1
    out = torch.empty(n, dtype=dtype, device=device)
    c = torch.tensor(1.0 / _IH_SIGMA, dtype=torch.float32, device=device)
    sc = torch.tensor(scale, dtype=torch.float32, device=device)
    for s in range(0, n, _CHUNK):
        m = min(_CHUNK, n - s)
        k = _keys(seed, tensor_id, s, m, device)
        acc = _lanes16(_mix(k + _s64(_G))) + _lanes16(_mix(k + _s64(2 * _G)))
        x = (acc - _IH_MEAN).to(torch.float32) * c
        out[s:s + m] = (x * sc).to(dtype)
    return out.reshape(shape)


def randint(shape, seed: int, tensor_id: int, high: int, device="cpu") -> torch.Tensor:
    """Uniform int32 in [0, high)."""
    n = int(math.prod(shape)) if len(shape) else 1
    out = torch.empty(n, dtype=torch.int32, device=device)
    for s in range(0, n, _CHUNK):
        m = min(_CHUNK, n - s)
        k = _keys(seed, tensor_id, s, m, device)
        out[s:s + m] = (_lsr(_mix(k + _s64(_G)), 32) % high).to(torch.int32)
    return out.reshape(shape)


# --- pure-Python restatement of the same recipe, used by the tests to pin the torch version ---

def _mix_py(z: int) -> int:
    z &= _M64
    z = ((z ^ (z >> 30)) * _C1) & _M64
    z = ((z ^ (z >> 27)) * _C2) & _M64
    return z ^ (z >> 31)


def normal_py(seed: int, tensor_id: int, i: int) -> float:
    key = (seed * _G + tensor_id * _T + i) & _M64
    acc = 0
    for j in (1, 2):
        h = _mix_py(key + j * _G)
        acc += (h & 0xFFFF) + ((h >> 16) & 0xFFFF) + ((h >> 32) & 0xFFFF) + (h >> 48)
    return (acc - _IH_MEAN) / _IH_SIGMA


def randint_py(seed: int, tensor_id: int, i: int, high: int) -> int:
    key = (seed * _G + tensor_id * _T + i) & _M64
    return (_mix_py(key + _G) >> 32) % high


# --- model-shaped bundles ---------------------------------------------------------------

@dataclass
class ModelShape:
    """Shape of a pre-norm bidirectional transformer denoiser (no biases, untied head)."""
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    dtype: str = "bf16"          # "fp32" or "bf16"
    mask_id: int = -1            # -1 -> vocab - 1
    w_std: float = 0.02
    head_scale: float = 1.0

    def __post_init__(self):
        if self.mask_id < 0:
            self.mask_id = self.vocab - 1


# tensor ids: 1 embed, 2 head, 3 final norm (unused: gains are 1), 16*(layer+1)+k per layer
TID_EMBED, TID_HEAD = 1, 2
_LAYER_K = {"w_q": 0, "w_k": 1, "w_v": 2, "w_o": 3, "w_gate": 4, "w_up": 5, "w_down": 6}


def layer_tid(layer: int, name: str) -> int:
    return 16 * (layer + 1) + _LAYER_K[name]


def make_weights(shape: ModelShape, seed: int, device="cpu") -> Dict[str, object]:
    """Random-init weights. Linear weights are logical [out_features, in_features]; the
    embedding is [vocab, d]; norm gains are all ones.  Values are N(0, w_std) (the head
    additionally times head_scale), rounded to the model dtype."""
    dt = torch.float32 if shape.dtype == "fp32" else torch.bfloat16
    d, hq, hkv, dh, f, v = (shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim,
                            shape.d_ffn, shape.vocab)
    w: Dict[str, object] = {
        "embed": normal((v, d), seed, TID_EMBED, shape.w_std, dt, device),
        "w_head": normal((v, d), seed, TID_HEAD, shape.w_std * shape.head_scale, dt, device),
        "final_norm": torch.ones(d, dtype=dt, device=device),
        "layers": [],
    }
    for l in range(shape.n_layers):
        w["layers"].append(make_layer(shape, seed, l, device))
    return w


def make_layer(shape: ModelShape, seed: int, l: int, device="cpu") -> Dict[str, torch.Tensor]:
    """The weights of layer l alone (the same values make_weights gives), for consumers that hold one layer at a time."""
    dt = torch.float32 if shape.dtype == "fp32" else torch.bfloat16
    d, hq, hkv, dh, f = shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn
    dims: Dict[str, Tuple[int, int]] = {
        "w_q": (hq * dh, d), "w_k": (hkv * dh, d), "w_v": (hkv * dh, d), "w_o": (d, hq * dh),
        "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f)}
    lw = {n: normal(s, seed, layer_tid(l, n), shape.w_std, dt, device) for n, s in dims.items()}
    lw["attn_norm"] = torch.ones(d, dtype=dt, device=device)
    lw["ffn_norm"] = torch.ones(d, dtype=dt, device=device)
    return lw


def make_prompt(batch: int, prompt_len: int, shape: ModelShape, seed: int, device="cpu") -> torch.Tensor:
    """Uniform-random prompt ids in [0, vocab) that avoid mask_id (drawn from vocab-1 ids)."""
    t = randint((batch, prompt_len), seed, 1000, shape.vocab - 1, device)
    return torch.where(t >= shape.mask_id, t + 1, t).to(torch.int32)


def delimiter_bitmap(vocab: int, lo: int, hi: int) -> torch.Tensor:
    """Bitmap (uint8, ceil(vocab/8) bytes; bit v%8 of byte v//8) of delimiter ids lo..hi inclusive."""
    bm = torch.zeros((vocab + 7) // 8, dtype=torch.uint8)
    for v in range(lo, hi + 1):
        bm[v // 8] |= 1 << (v % 8)
    return bm


def synthetic_scores(n: int, seed: int, tensor_id: int, p_pass: float, tau: float,
                     delim_density: float, delim_lo: int, delim_hi: int, vocab: int):
    """Per-position (score, yhat) arrays for scan tests with text-like structure: a position
    passes the threshold tau with probability p_pass and predicts a delimiter id with
    probability delim_density (the paper's delimiters are punctuation/newlines, roughly one
    token in seven to ten of natural text)."""
    u = randint((n,), seed, tensor_id, 1 << 20).to(torch.float64) / float(1 << 20)
    u2 = randint((n,), seed, tensor_id + 1, 1 << 20).to(torch.float64) / float(1 << 20)
    u3 = randint((n,), seed, tensor_id + 2, 1 << 20).to(torch.float64) / float(1 << 20)
    passing = u < p_pass
    score = torch.where(passing, tau + (1.0 - tau) * u2, tau * u2 * 0.999).to(torch.float32)
    is_d = u3 < delim_density
    dl = randint((n,), seed, tensor_id + 3, delim_hi - delim_lo + 1) + delim_lo
    other = randint((n,), seed, tensor_id + 4, vocab - delim_hi - 2) + delim_hi + 1
    yhat = torch.where(is_d, dl, other).to(torch.int32)
    return score, yhat


@dataclass
class Workload:
    name: str
    shape: ModelShape
    batch: int
    prompt_len: int
    gen_len: int
    tau: float
    delim: Tuple[int, int]
    extra: dict = field(default_factory=dict)


def config(name: str) -> Workload:
    """The workloads named by the benchmark configuration list (1-based as 'cfg1'..'cfg5')."""
    if name == "cfg1":
        return Workload(name, ModelShape(2, 256, 4, 4, 64, 1024, 2048, dtype="fp32", head_scale=8.0),
                        1, 32, 64, 0.9, (1, 8))
    if name == "cfg3":
        return Workload(name, ModelShape(32, 4096, 32, 32, 128, 12288, 126464, head_scale=12.0),
                        1, 256, 256, 0.9, (1, 32))
    if name == "cfg4":
        return Workload(name, ModelShape(28, 3584, 28, 4, 128, 18944, 152064, rope_theta=1e6,
                                         head_scale=12.0), 4, 512, 512, 0.85, (1, 64))
    if name == "cfg5":
        return Workload(name, ModelShape(32, 4096, 32, 32, 128, 12288, 126464, head_scale=12.0),
                        16, 1024, 1024, 0.9, (1, 32))
    raise KeyError(name)
