"""ctypes binding with the same names as include/lsp.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.environ.get("LSP_LIB") or os.path.join(_HERE, "liblsp_b200.so")   # LSP_LIB: another build of the library

FLAG_SNAPPED, FLAG_FALLBACK, FLAG_RANGE_UNACHIEVABLE = 1, 2, 4
FLAG_RUN_TO_END, FLAG_NEAR_THRESHOLD, FLAG_NEAR_TIE = 8, 16, 32

EXPORTS = ["lsp_workspace_bytes", "lsp_kv_cache_bytes", "lsp_init", "lsp_set_sched", "lsp_set_option",
           "lsp_begin", "lsp_denoise_step", "lsp_commit", "lsp_generate", "lsp_generate_host", "lsp_active", "lsp_score_rows",
           "lsp_get_scores", "lsp_head_scan", "lsp_scan", "lsp_op_linear", "lsp_op_attention", "lsp_last_timing", "lsp_get_counters", "lsp_reset_counters",
           "lsp_linear_static", "lsp_last_error", "lsp_destroy"]


class LSPError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"lsp error {code}: {msg}")
        self.code = code


class ModelCfg(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("dtype", C.c_int), ("mask_id", C.c_int)]


class SchedCfgC(C.Structure):
    _fields_ = [("score", C.c_int), ("mode", C.c_int), ("tau", C.c_float), ("alpha", C.c_float), ("beta", C.c_float),
                ("l_min", C.c_int), ("snap_window", C.c_int), ("fixed_k", C.c_int), ("delim_bitmap", C.c_void_p),
                ("exclude_mask_logit", C.c_int), ("flag_tol", C.c_float), ("tie_tol", C.c_float), ("topology", C.c_int)]


class WeightsC(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("final_norm", C.c_void_p), ("w_head", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm", "w_qkv", "w_o", "ffn_norm", "w_gate", "w_up", "w_down")]


class StepRec(C.Structure):
    _fields_ = [("step", C.c_int), ("n_before", C.c_int), ("rows", C.c_int), ("l_run", C.c_int), ("l_commit", C.c_int),
                ("tau_used", C.c_float), ("flags", C.c_uint), ("ms", C.c_float), ("flips", C.c_int), ("flip_base", C.c_int)]


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2603_05454_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    l = C.CDLL(_LIB_PATH)
    l.lsp_workspace_bytes.restype = C.c_size_t
    l.lsp_workspace_bytes.argtypes = [C.POINTER(ModelCfg), C.c_int, C.c_int]
    l.lsp_kv_cache_bytes.restype = C.c_size_t
    l.lsp_kv_cache_bytes.argtypes = [C.POINTER(ModelCfg), C.c_int, C.c_int]
    l.lsp_init.argtypes = [C.POINTER(C.c_void_p), C.POINTER(ModelCfg), C.POINTER(SchedCfgC), C.POINTER(WeightsC),
                           C.c_void_p, C.c_void_p, C.c_size_t, C.c_int, C.c_int, C.c_void_p]
    l.lsp_set_sched.argtypes = [C.c_void_p, C.POINTER(SchedCfgC)]
    l.lsp_set_option.argtypes = [C.c_void_p, C.c_int, C.c_int]
    l.lsp_debug_set.argtypes = [C.c_void_p, C.c_int, C.c_int]      # internal (csrc/lsp_tuning.h), not in EXPORTS
    l.lsp_debug_wait_selftest.argtypes = [C.c_void_p, C.c_int]
    l.lsp_begin.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int]
    l.lsp_denoise_step.argtypes = [C.c_void_p, C.POINTER(StepRec)]
    l.lsp_commit.argtypes = [C.c_void_p, C.c_void_p]
    l.lsp_generate.argtypes = [C.c_void_p, C.POINTER(StepRec), C.c_int, C.POINTER(C.c_int)]
    l.lsp_generate_host.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                    C.POINTER(StepRec), C.c_int, C.POINTER(C.c_int)]
    l.lsp_active.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int)]
    l.lsp_score_rows.argtypes = [C.c_void_p]
    l.lsp_get_scores.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    l.lsp_head_scan.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int] + [C.c_void_p] * 4
    l.lsp_scan.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int] + [C.c_void_p] * 4
    l.lsp_op_linear.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int]
    l.lsp_op_attention.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.c_int]
    l.lsp_last_timing.argtypes = [C.c_void_p, C.c_void_p]
    l.lsp_get_counters.argtypes = [C.c_void_p, C.c_void_p]
    l.lsp_reset_counters.argtypes = [C.c_void_p]
    l.lsp_linear_static.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_char_p,
                                    C.c_size_t]
    l.lsp_last_error.restype = C.c_char_p
    l.lsp_last_error.argtypes = [C.c_void_p]
    l.lsp_destroy.argtypes = [C.c_void_p]
    return l


lib = _load()


@dataclass
class SchedCfg:
    score: int = 0            # 0 = max-prob, 1 = logit margin
    mode: int = 0             # 0 fixed tau, 1 adaptive, 2 fixed-k
    tau: float = 0.9
    alpha: float = 0.25
    beta: float = 0.50
    l_min: int = 1
    snap_window: int = 16
    fixed_k: int = 1
    delim_bitmap: Optional[torch.Tensor] = None   # uint8 CUDA tensor, vocab bits
    exclude_mask_logit: int = 1
    flag_tol: float = 0.0
    tie_tol: float = 0.0
    topology: int = 0         # 0 prefix (LSP), 1 scattered acceptance (baseline)

    def to_c(self) -> SchedCfgC:
        p = self.delim_bitmap.data_ptr() if self.delim_bitmap is not None else None
        return SchedCfgC(self.score, self.mode, self.tau, self.alpha, self.beta, self.l_min, self.snap_window,
                         self.fixed_k, p, self.exclude_mask_logit, self.flag_tol, self.tie_tol, self.topology)


def _ptr_array(tensors: Sequence[torch.Tensor]):
    arr = (C.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])
    return arr


class LSPDecoder:
    """Owns the device buffers (allocated through torch) and a library context.

    shape: any object with the fields of lsp_model_cfg (n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn,
    vocab, rms_eps, rope_theta, dtype in {"fp32","bf16"}, mask_id).
    weights: dict with CUDA tensors embed, w_head, final_norm and a list "layers" of dicts with attn_norm, w_q,
    w_k, w_v (or w_qkv), w_o, ffn_norm, w_gate, w_up, w_down; linear weights are [out_features, in_features].
    """

    def __init__(self, shape, weights, sched: SchedCfg, max_batch: int, max_len: int, device="cuda:0", stream=None):
        self.device = torch.device(device)
        self.shape = shape
        self.tdtype = torch.float32 if shape.dtype == "fp32" else torch.bfloat16
        self.mc = ModelCfg(shape.n_layers, shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim,
                           shape.d_ffn, shape.vocab, shape.rms_eps, shape.rope_theta,
                           0 if shape.dtype == "fp32" else 1, shape.mask_id)
        self.max_batch, self.max_len = max_batch, max_len
        ws = lib.lsp_workspace_bytes(C.byref(self.mc), max_batch, max_len)
        kv = lib.lsp_kv_cache_bytes(C.byref(self.mc), max_batch, max_len)
        if ws == 0 or kv == 0:
            raise LSPError(-2, "unsupported model shape")
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=self.device)
        self.kv_cache = torch.zeros(kv, dtype=torch.uint8, device=self.device)
        self._keep = []
        layers = []
        for lw in weights["layers"]:
            lw = dict(lw)
            if "w_qkv" not in lw:
                lw["w_qkv"] = torch.cat([lw["w_q"], lw["w_k"], lw["w_v"]], dim=0).contiguous()
            layers.append(lw)
        self._layers = layers
        self._w = weights
        names = ("attn_norm", "w_qkv", "w_o", "ffn_norm", "w_gate", "w_up", "w_down")
        arrs = {n: _ptr_array([lw[n] for lw in layers]) for n in names}
        self._keep.append(arrs)
        wc = WeightsC(weights["embed"].data_ptr(), weights["final_norm"].data_ptr(), weights["w_head"].data_ptr(),
                      *[C.cast(arrs[n], C.POINTER(C.c_void_p)) for n in names])
        self.sched = sched
        sc = sched.to_c()
        self.stream = stream
        sptr = stream.cuda_stream if stream is not None else torch.cuda.current_stream(self.device).cuda_stream
        self._h = C.c_void_p()
        with torch.cuda.device(self.device):
            rc = lib.lsp_init(C.byref(self._h), C.byref(self.mc), C.byref(sc), C.byref(wc), self.kv_cache.data_ptr(),
                              self.workspace.data_ptr(), ws, max_batch, max_len, sptr)
        if rc != 0:
            raise LSPError(rc, "lsp_init failed")
        self.batch = 0

    # -- helpers
    def _check(self, rc):
        if rc != 0:
            raise LSPError(rc, lib.lsp_last_error(self._h).decode())

    def close(self):
        if self._h:
            lib.lsp_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def layer_weights(self):
        """Per-layer weight tensors as the library holds them (w_qkv is the packed [q; k; v] projection)."""
        return self._layers

    def set_sched(self, sched: SchedCfg):
        self.sched = sched
        sc = sched.to_c()
        self._check(lib.lsp_set_sched(self._h, C.byref(sc)))

    def set_option(self, key: int, value: int):
        self._check(lib.lsp_set_option(self._h, key, value))

    def debug_set(self, key: int, value: int):
        """Internal tuning and benchmark knobs (csrc/lsp_tuning.h); not part of the public interface."""
        self._check(lib.lsp_debug_set(self._h, key, value))

    def wait_selftest(self, limit_us: int = 200):
        """Internal (csrc/lsp_tuning.h): lets a bounded device-side wait run out; raises LSPError(-6)."""
        self._check(lib.lsp_debug_wait_selftest(self._h, limit_us))

    # -- Algorithm 1
    def begin(self, tokens: torch.Tensor, prompt_len, gen_len):
        assert tokens.dtype == torch.int32 and tokens.is_cuda and tokens.dim() == 2 and tokens.is_contiguous()
        batch = tokens.shape[0]
        pl = np.ascontiguousarray(prompt_len, dtype=np.int32)
        gl = np.ascontiguousarray(gen_len, dtype=np.int32)
        if pl.shape != (batch,) or gl.shape != (batch,):
            raise ValueError(f"prompt_len and gen_len need one entry per row of tokens ({batch})")
        self._check(lib.lsp_begin(self._h, tokens.data_ptr(), tokens.shape[1], pl.ctypes.data, gl.ctypes.data, batch))
        self.tokens = tokens          # the library state changed only now (a rejected call leaves the old decode in place)
        self.batch = batch

    def denoise_step(self):
        recs = (StepRec * self.batch)()
        self._check(lib.lsp_denoise_step(self._h, recs))
        return [_rec(r) for r in recs]

    def commit(self, L=None):
        if L is None:
            self._check(lib.lsp_commit(self._h, None))
        else:
            a = np.ascontiguousarray(L, dtype=np.int32)
            if a.shape != (self.batch,):
                raise ValueError(f"L needs one entry per sequence ({self.batch})")
            self._check(lib.lsp_commit(self._h, a.ctypes.data))

    def generate(self, max_recs: int = 0):
        n = C.c_int(0)
        recs = (StepRec * max_recs)() if max_recs else None
        self._check(lib.lsp_generate(self._h, recs, max_recs, C.byref(n)))
        out = [_rec(r) for r in recs][: n.value * self.batch] if recs is not None else []
        return n.value, out

    def generate_host(self, tokens_dev: torch.Tensor, tokens_in: torch.Tensor, tokens_out: torch.Tensor, prompt_len,
                      gen_len, max_recs: int = 0):
        """Algorithm 1 from host memory: tokens_in / tokens_out are CPU int32 tensors [batch, stride] (pinned or
        not), tokens_dev the device buffer of the same shape the decode runs in."""
        assert tokens_dev.dtype == torch.int32 and tokens_dev.is_cuda and tokens_dev.is_contiguous()
        for t in (tokens_in, tokens_out):
            assert t.dtype == torch.int32 and not t.is_cuda and t.is_contiguous() and t.shape == tokens_dev.shape
        batch = tokens_dev.shape[0]
        pl = np.ascontiguousarray(prompt_len, dtype=np.int32)
        gl = np.ascontiguousarray(gen_len, dtype=np.int32)
        if pl.shape != (batch,) or gl.shape != (batch,):
            raise ValueError(f"prompt_len and gen_len need one entry per row of tokens ({batch})")
        self.tokens = tokens_dev
        self.batch = batch
        n = C.c_int(0)
        recs = (StepRec * max_recs)() if max_recs else None
        self._check(lib.lsp_generate_host(self._h, tokens_dev.data_ptr(), tokens_dev.shape[1], tokens_in.data_ptr(),
                                          tokens_out.data_ptr(), pl.ctypes.data, gl.ctypes.data, self.batch, recs,
                                          max_recs, C.byref(n)))
        out = [_rec(r) for r in recs][: n.value * self.batch] if recs is not None else []
        return n.value, out

    def active(self):
        a = np.zeros(self.batch, dtype=np.int32)
        u = C.c_int(0)
        self._check(lib.lsp_active(self._h, a.ctypes.data, C.byref(u)))
        return a, u.value

    def scores(self):
        n = lib.lsp_score_rows(self._h)
        y = np.zeros(n, dtype=np.int32)
        p = np.zeros(n, dtype=np.float32)
        m = np.zeros(n, dtype=np.float32)
        self._check(lib.lsp_get_scores(self._h, y.ctypes.data, p.ctypes.data, m.ctypes.data))
        return y, p, m

    def _scan_out(self, batch):
        return (np.zeros(batch, np.int32), np.zeros(batch, np.int32), np.zeros(batch, np.uint32), np.zeros(batch, np.float32))

    def head_scan(self, hidden: torch.Tensor, seq_offsets):
        assert hidden.is_cuda and hidden.is_contiguous() and hidden.dtype == self.tdtype
        so = np.ascontiguousarray(seq_offsets, dtype=np.int32)
        batch = len(so) - 1
        lr, lc, fl, tu = self._scan_out(batch)
        self._check(lib.lsp_head_scan(self._h, hidden.data_ptr(), so.ctypes.data, batch, lr.ctypes.data, lc.ctypes.data,
                                      fl.ctypes.data, tu.ctypes.data))
        return dict(L_run=lr, L_commit=lc, flags=fl, tau_used=tu)

    def scan(self, score: torch.Tensor, yhat: torch.Tensor, margin: Optional[torch.Tensor], seq_offsets):
        assert score.dtype == torch.float32 and yhat.dtype == torch.int32 and score.is_cuda and yhat.is_cuda
        so = np.ascontiguousarray(seq_offsets, dtype=np.int32)
        batch = len(so) - 1
        lr, lc, fl, tu = self._scan_out(batch)
        self._check(lib.lsp_scan(self._h, score.data_ptr(), yhat.data_ptr(), margin.data_ptr() if margin is not None else None,
                                 so.ctypes.data, batch, lr.ctypes.data, lc.ctypes.data, fl.ctypes.data, tu.ctypes.data))
        return dict(L_run=lr, L_commit=lc, flags=fl, tau_used=tu)

    def op_linear(self, op: int, A: torch.Tensor, W: torch.Tensor, W2: Optional[torch.Tensor], out: torch.Tensor):
        M, K = A.shape
        N = W.shape[0]
        self._check(lib.lsp_op_linear(self._h, op, A.data_ptr(), W.data_ptr(), W2.data_ptr() if W2 is not None else None,
                                      out.data_ptr(), M, N, K))
        return out

    def op_attention(self, layer: int, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, out: torch.Tensor,
                     cache_len, rows):
        """One layer's suffix-over-prefix attention on packed rows; the cached K/V are read from kv_view()."""
        cl = np.ascontiguousarray(cache_len, dtype=np.int32)
        rw = np.ascontiguousarray(rows, dtype=np.int32)
        assert cl.shape == rw.shape and q.shape[0] == int(rw.sum()) == k_new.shape[0] == v_new.shape[0] == out.shape[0]
        for t in (q, k_new, v_new, out):
            assert t.is_cuda and t.is_contiguous() and t.dtype == self.tdtype
        self._check(lib.lsp_op_attention(self._h, layer, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), out.data_ptr(),
                                         cl.ctypes.data, rw.ctypes.data, len(cl)))
        return out

    def last_timing(self):
        a = np.zeros(8, dtype=np.float32)
        self._check(lib.lsp_last_timing(self._h, a.ctypes.data))
        return a

    def counters(self):
        a = np.zeros(18, dtype=np.float64)
        self._check(lib.lsp_get_counters(self._h, a.ctypes.data))
        return dict(zip(("launches", "gemm_bytes", "gemm_flops", "attn_bytes", "append_bytes", "head_bytes",
                         "head_flops", "steps", "launches_misc", "launches_gemm", "launches_attn", "launches_head",
                         "launches_scan", "launches_commit", "attn_flops", "tokens", "attn_kernel", "attn_cluster"),
                        a.tolist()))

    def reset_counters(self):
        self._check(lib.lsp_reset_counters(self._h))

    # views of the caller-visible state (device memory owned here)
    def kv_view(self):
        s = self.shape
        return self.kv_cache.view(self.tdtype).view(s.n_layers, 2, self.max_batch, self.max_len, s.n_kv_heads, s.head_dim)


def linear_static(A: torch.Tensor, W: torch.Tensor, out: torch.Tensor, stream=None):
    """out = A W^T through lsp_linear_static: no context, no workspace; the library's static scratch is used.
    A [M, K], W [N, K], out [M, N]: contiguous bfloat16 CUDA tensors on the current device."""
    M, K = A.shape
    N = W.shape[0]
    sptr = stream.cuda_stream if stream is not None else torch.cuda.current_stream(A.device).cuda_stream
    buf = C.create_string_buffer(256)
    with torch.cuda.device(A.device):
        rc = lib.lsp_linear_static(A.data_ptr(), W.data_ptr(), out.data_ptr(), M, N, K, sptr, buf, len(buf))
    if rc != 0:
        raise LSPError(rc, buf.value.decode())
    return out


def _rec(r: StepRec):
    return dict(step=r.step, n_before=r.n_before, rows=r.rows, L_run=r.l_run, L_commit=r.l_commit,
                tau_used=r.tau_used, flags=r.flags, ms=r.ms, flips=r.flips, flip_base=r.flip_base)
