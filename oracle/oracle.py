"""ctypes driver of the C oracle: one request at a time, layer by layer.

TEST INFRASTRUCTURE (see synera_oracle.c).  Requests are independent, so a batch is a loop
over requests.  Weights are supplied by a ``layer_weights(l)`` callable so that a large model
can be regenerated one layer at a time instead of being held in memory.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Callable, Dict, List, Optional, Sequence

import numpy as np

from . import build as _build


class _Desc(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ffn", C.c_int32),
                ("vocab", C.c_int32), ("rope_base", C.c_double), ("rms_eps", C.c_double),
                ("bf16_operands", C.c_int32)]


class _LayerW(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2")]


def _u16(t) -> np.ndarray:
    """bf16 torch tensor (or uint16 array) -> contiguous uint16 numpy bit pattern."""
    if isinstance(t, np.ndarray):
        assert t.dtype == np.uint16
        return np.ascontiguousarray(t)
    import torch
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


@dataclass
class OracleResult:
    top1: np.ndarray            # [n] int32
    top2: np.ndarray            # [n] int32
    gap: np.ndarray             # [n] top1 logit - top2 logit
    logits: Optional[np.ndarray]  # [n, V] or None
    accept_len: int
    correction: int


def verify_greedy(top1: Sequence[int], chunk: Sequence[int], u: int = 1):
    """Pure-integer greedy verification (the C routine, callable on injected argmax arrays)."""
    lib = Oracle._load(False)
    t = np.ascontiguousarray(np.asarray(top1, dtype=np.int32))
    c = np.ascontiguousarray(np.asarray(chunk, dtype=np.int32))
    a, k = C.c_int32(), C.c_int32()
    lib.orc_verify(_p(t), _p(c), C.c_int(len(c)), C.c_int(u), C.byref(a), C.byref(k))
    return a.value, k.value


class Oracle:
    """shape: any object with n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab,
    rope_base, rms_eps attributes."""

    _libs: Dict[bool, C.CDLL] = {}

    @classmethod
    def _load(cls, f32: bool) -> C.CDLL:
        if f32 not in cls._libs:
            _build.build()
            lib = C.CDLL(_build.lib_path(f32))
            lib.orc_real_bytes.restype = C.c_int
            for fn in ("orc_bf16_round_array", "orc_embed", "orc_rmsnorm", "orc_linear", "orc_rope", "orc_kv_write", "orc_attention",
                       "orc_layer", "orc_logits", "orc_verify", "orc_slot"):
                getattr(lib, fn).restype = None
            cls._libs[f32] = lib
        return cls._libs[f32]

    def __init__(self, shape, page_size: int = 16, f32: bool = False, bf16_operands: bool = False):
        """bf16_operands: model the network as a bf16 model (bf16 weights and activations, wide
        accumulation): every activation entering a matrix product or the KV cache is rounded to bf16.
        False keeps every intermediate in double (or float): the plain mathematical definition."""
        self.lib = self._load(f32)
        self.real = np.float32 if f32 else np.float64
        assert self.lib.orc_real_bytes() == np.dtype(self.real).itemsize
        self.shape = shape
        self.P = page_size
        self.desc = _Desc(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                          shape.d_ffn, shape.vocab, float(shape.rope_base), float(shape.rms_eps),
                          1 if bf16_operands else 0)

    # ------------------------------------------------------------------ storage
    def new_pool(self, n_pages: int) -> List[np.ndarray]:
        """Per-layer KV pools, [n_pages][2][Hkv][P][hd], zero-filled."""
        s = self.shape
        return [np.zeros((n_pages, 2, s.n_kv_heads, self.P, s.head_dim), dtype=self.real)
                for _ in range(s.n_layers)]

    def load_kv(self, pool_layer: np.ndarray, page_table: np.ndarray, pos0: int, k, v) -> None:
        """Place externally produced K/V ([npos][Hkv][hd], any float type) at logical positions pos0.."""
        k = np.asarray(k, dtype=self.real)
        v = np.asarray(v, dtype=self.real)
        pos = pos0 + np.arange(k.shape[0])
        pages = np.asarray(page_table, dtype=np.int64)[pos // self.P][:, None]
        rows = (pos % self.P)[:, None]
        heads = np.arange(self.shape.n_kv_heads)[None, :]
        pool_layer[pages, 0, heads, rows, :] = k
        pool_layer[pages, 1, heads, rows, :] = v

    # ------------------------------------------------------------------ single ops (exposed for pins)
    def bf16_round(self, a) -> np.ndarray:
        a = np.ascontiguousarray(a, dtype=self.real).ravel()
        out = np.empty_like(a)
        self.lib.orc_bf16_round_array(_p(a), _p(out), C.c_int(a.size))
        return out

    def embed(self, E, tokens) -> np.ndarray:
        tok = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        x = np.empty((len(tok), self.shape.d_model), dtype=self.real)
        Eb = _u16(E)
        self.lib.orc_embed(_p(Eb), C.c_int(self.shape.d_model), _p(tok), C.c_int(len(tok)), _p(x))
        return x

    def rmsnorm(self, x: np.ndarray, g) -> np.ndarray:
        x = np.ascontiguousarray(x, dtype=self.real)
        out = np.empty_like(x)
        gb = _u16(g)
        self.lib.orc_rmsnorm(_p(x), _p(gb), C.c_int(x.shape[0]), C.c_int(x.shape[1]),
                             C.c_double(self.shape.rms_eps), _p(out))
        return out

    def linear(self, x: np.ndarray, W) -> np.ndarray:
        x = np.ascontiguousarray(x, dtype=self.real)
        Wb = _u16(W)
        N, K = Wb.shape
        assert x.shape[1] == K
        y = np.empty((x.shape[0], N), dtype=self.real)
        self.lib.orc_linear(_p(x), _p(Wb), C.c_int(x.shape[0]), C.c_int(K), C.c_int(N), _p(y))
        return y

    def rope(self, v: np.ndarray, n_heads: int, pos: int) -> np.ndarray:
        out = np.ascontiguousarray(v, dtype=self.real).copy()
        self.lib.orc_rope(_p(out), C.c_int(n_heads), C.c_int(self.shape.head_dim), C.c_int(pos),
                          C.c_double(self.shape.rope_base))
        return out

    def attention(self, q: np.ndarray, pool_layer: np.ndarray, page_table, ctx: int) -> np.ndarray:
        q = np.ascontiguousarray(q, dtype=self.real)
        pt = np.ascontiguousarray(np.asarray(page_table, dtype=np.int32))
        out = np.empty_like(q)
        self.lib.orc_attention(C.byref(self.desc), _p(q), _p(pool_layer), _p(pt), C.c_int(self.P),
                               C.c_int(ctx), C.c_int(q.shape[0]), _p(out))
        return out

    def slot(self, page_table, pos: int):
        pt = np.ascontiguousarray(np.asarray(page_table, dtype=np.int32))
        a, b = C.c_int32(), C.c_int32()
        self.lib.orc_slot(_p(pt), C.c_int(self.P), C.c_int(pos), C.byref(a), C.byref(b))
        return a.value, b.value

    # ------------------------------------------------------------------ the step, one request
    def layer(self, w: Dict[str, object], x: np.ndarray, pool_layer: np.ndarray, page_table: np.ndarray,
              ctx: int) -> None:
        """x [n, d] updated in place; the chunk's K/V land in pool_layer."""
        keep = {k: _u16(w[k]) for k in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2")}
        lw = _LayerW(*[keep[k].ctypes.data for k in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2")])
        assert x.dtype == self.real and x.flags.c_contiguous and pool_layer.dtype == self.real
        pt = np.ascontiguousarray(np.asarray(page_table, dtype=np.int32))
        self.lib.orc_layer(C.byref(self.desc), C.byref(lw), _p(x), _p(pool_layer), _p(pt), C.c_int(self.P),
                           C.c_int(ctx), C.c_int(x.shape[0]))

    def logits(self, glob: Dict[str, object], x: np.ndarray, want_logits: bool = True):
        n = x.shape[0]
        fn, lm = _u16(glob["final_norm"]), _u16(glob["lm_head"])
        lg = np.empty((n, self.shape.vocab), dtype=self.real) if want_logits else None
        t1 = np.empty(n, dtype=np.int32)
        t2 = np.empty(n, dtype=np.int32)
        gap = np.empty(n, dtype=self.real)
        self.lib.orc_logits(C.byref(self.desc), _p(fn), _p(lm), _p(x), C.c_int(n),
                            _p(lg) if want_logits else None, _p(t1), _p(t2), _p(gap))
        return lg, t1, t2, gap

    def forward_chunk(self, glob, layer_weights: Callable[[int], Dict[str, object]], pools: List[np.ndarray],
                      page_table, ctx: int, chunk: Sequence[int], u: int = 1, want_logits: bool = True,
                      taps: Optional[dict] = None) -> OracleResult:
        """Partial prefill of one request's chunk against its cached prefix, then greedy verify."""
        x = self.embed(glob["embed"], chunk)
        for l in range(self.shape.n_layers):
            self.layer(layer_weights(l), x, pools[l], page_table, ctx)
            if taps is not None:
                taps[("x", l)] = x.copy()
        lg, t1, t2, gap = self.logits(glob, x, want_logits)
        a, c = verify_greedy(t1, chunk, u)
        return OracleResult(t1, t2, gap, lg, a, c)
