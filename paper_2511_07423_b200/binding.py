"""ctypes binding of include/synera.h and include/synera_sched.h: argument marshalling only.

PyTorch supplies device memory and streams; every pointer handed to the library is a raw
``data_ptr()``.  There is no CPU fallback: if the library is missing or a call fails, a
:class:`SynError` is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import torch

HERE = os.path.dirname(os.path.abspath(__file__))


def lib_path() -> str:
    return os.path.join(HERE, "libsynera.so")


class SynError(RuntimeError):
    def __init__(self, code: int, what: str):
        detail = ""
        if code in (-8, -10):
            try:
                detail = " [" + load_library().syn_last_cuda_error().decode() + "]"
            except Exception:  # pragma: no cover
                pass
        super().__init__(f"{what}: {code} ({_strerror(code)}){detail}")
        self.code = code


class _Desc(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] \
        + [("rope_base", C.c_float), ("rms_eps", C.c_float), ("flags", C.c_uint32)]


class _Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] \
        + [(n, C.POINTER(C.c_void_p)) for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2")] \
        + [("location", C.c_int32)]


class StepStats(C.Structure):
    _fields_ = [("n_req", C.c_int32), ("n_tokens", C.c_int32), ("ctx_tokens", C.c_int64),
                ("weight_bytes", C.c_int64), ("kv_read_bytes", C.c_int64), ("kv_write_bytes", C.c_int64),
                ("dense_flops", C.c_double), ("attn_flops", C.c_double), ("attn_items", C.c_int32),
                ("attn_split_items", C.c_int32), ("kernel_launches", C.c_int32), ("attn_rows", C.c_int32), ("h2d_bytes", C.c_int64),
                ("t_gpu_ms", C.c_double), ("t_wall_ms", C.c_double)]

KERNEL_CLASSES = ("prep", "qkv_gemm", "attention", "attention_merge", "o_gemm", "gate_up_gemm", "down_gemm",
                  "lm_head_gemm", "verify", "unused")


_LIB: Optional[C.CDLL] = None

EXPORTS = ["syn_model_load", "syn_model_free", "syn_kv_alloc", "syn_kv_free", "syn_kv_import", "syn_kv_export",
           "syn_verify_batch", "syn_plan_create", "syn_plan_free", "syn_verify_run", "syn_model_status",
           "syn_last_step_stats", "syn_plan_stats", "syn_plan_host", "syn_strerror", "syn_last_cuda_error", "syn_op_linear",
           "syn_op_linear_as", "syn_op_linear_reset", "syn_debug_set_spin_limit", "syn_debug_linear_counter", "syn_debug_set_schedule",
           "syn_debug_set_attention",
           "syn_op_attention", "syn_op_attention_static",
           "syn_set_profile", "syn_get_profile", "syn_verify_batch_sampled", "syn_op_sample_verify",
           "syn_gemm_plan_host", "syn_gemm_work_host", "syn_gemm2_plan_host", "syn_gemm2_work_host"]
SCHED_EXPORTS = ["syn_sched_create", "syn_sched_free", "syn_sched_add_request", "syn_sched_add_verify", "syn_sched_finish",
                 "syn_sched_peek", "syn_sched_commit", "syn_sched_step", "syn_sched_get_stats"]


def load_library() -> C.CDLL:
    global _LIB
    if _LIB is None:
        path = lib_path()
        if not os.path.exists(path):
            raise SynError(-1, f"{path} is missing: run `python -m paper_2511_07423_b200.build`")
        lib = C.CDLL(path)
        lib.syn_strerror.restype = C.c_char_p
        lib.syn_strerror.argtypes = [C.c_int]
        lib.syn_last_cuda_error.restype = C.c_char_p
        lib.syn_last_cuda_error.argtypes = []
        for fn in ("syn_model_free", "syn_kv_free", "syn_plan_free", "syn_sched_free"):
            getattr(lib, fn).restype = None
            getattr(lib, fn).argtypes = [C.c_void_p]
        _LIB = lib
    return _LIB


def _strerror(code: int) -> str:
    try:
        return load_library().syn_strerror(code).decode()
    except Exception:  # pragma: no cover
        return "?"


def _check(code: int, what: str) -> None:
    if code != 0:
        raise SynError(code, what)


def _i32(t) -> torch.Tensor:
    t = torch.as_tensor(t, dtype=torch.int32, device="cpu").contiguous()
    return t


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> C.c_void_p:
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


class Model:
    """syn_model_load / syn_model_free."""

    def __init__(self, shape, glob: Dict[str, torch.Tensor], layers: Sequence[Dict[str, torch.Tensor]]):
        lib = load_library()
        L = shape.n_layers
        assert len(layers) == L
        dev = glob["embed"].is_cuda
        keep: List[torch.Tensor] = []

        def ptr(t: torch.Tensor) -> int:
            assert t.dtype == torch.bfloat16 and t.is_cuda == dev
            t = t.contiguous()
            keep.append(t)
            return t.data_ptr()

        w = _Weights()
        w.embed, w.lm_head, w.final_norm = ptr(glob["embed"]), ptr(glob["lm_head"]), ptr(glob["final_norm"])
        arrays = {}
        for name in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2"):
            arr = (C.c_void_p * L)(*[ptr(layers[l][name]) for l in range(L)])
            arrays[name] = arr
            setattr(w, name, C.cast(arr, C.POINTER(C.c_void_p)))
        w.location = 1 if dev else 0
        d = _Desc(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                  shape.vocab, float(shape.rope_base), float(shape.rms_eps), 0)
        self._h = C.c_void_p()
        _check(lib.syn_model_load(C.byref(d), C.byref(w), C.byref(self._h)), "syn_model_load")
        self.shape = shape
        self._lib = lib

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.syn_model_free(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def status(self) -> int:
        return int(self._lib.syn_model_status(self._h))

    def set_profile(self, on: bool) -> None:
        _check(self._lib.syn_set_profile(self._h, C.c_int(1 if on else 0)), "syn_set_profile")

    def last_step_stats(self) -> "StepStats":
        """syn_last_step_stats: counters of the last step launched on this model; with profiling on
        also its device time and, for the blocking calls, the wall time."""
        s = StepStats()
        _check(self._lib.syn_last_step_stats(self._h, C.byref(s)), "syn_last_step_stats")
        return s

    def get_profile(self):
        """{class name: (total ms, launches)} since the last call (synchronises the device)."""
        n = len(KERNEL_CLASSES)
        ms, cnt = (C.c_double * n)(), (C.c_int32 * n)()
        _check(self._lib.syn_get_profile(self._h, ms, cnt), "syn_get_profile")
        return {KERNEL_CLASSES[i]: (ms[i], cnt[i]) for i in range(n)}


class KVCache:
    """syn_kv_alloc / syn_kv_import / syn_kv_export / syn_kv_free."""

    def __init__(self, model: Model, n_pages: int, page_size: int = 16):
        self._lib = load_library()
        self.model = model
        self.n_pages, self.page_size = n_pages, page_size
        self._h = C.c_void_p()
        _check(self._lib.syn_kv_alloc(model._h, C.c_uint32(n_pages), C.c_uint32(page_size), C.byref(self._h)),
               "syn_kv_alloc")

    def import_kv(self, layer: int, page_table, pos0: int, k: torch.Tensor, v: torch.Tensor, stream=None) -> None:
        pt = _i32(page_table)
        assert k.is_cuda and v.is_cuda and k.dtype == torch.bfloat16 and k.is_contiguous() and v.is_contiguous()
        _check(self._lib.syn_kv_import(self._h, C.c_uint32(layer), C.c_void_p(pt.data_ptr()), C.c_int32(pos0),
                                       C.c_int32(k.shape[0]), C.c_void_p(k.data_ptr()), C.c_void_p(v.data_ptr()),
                                       _stream_ptr(stream)), "syn_kv_import")

    def export_kv(self, layer: int, page_table, pos0: int, n_pos: int, stream=None):
        s = self.model.shape
        pt = _i32(page_table)
        k = torch.empty(n_pos, s.n_kv_heads, s.head_dim, dtype=torch.bfloat16, device="cuda")
        v = torch.empty_like(k)
        _check(self._lib.syn_kv_export(self._h, C.c_uint32(layer), C.c_void_p(pt.data_ptr()), C.c_int32(pos0),
                                       C.c_int32(n_pos), C.c_void_p(k.data_ptr()), C.c_void_p(v.data_ptr()),
                                       _stream_ptr(stream)), "syn_kv_export")
        return k, v

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.syn_kv_free(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -------------------------------------------------------------- the step
    def verify_batch(self, chunk_tokens, chunk_offsets, page_tables, ctx_lens, n_uncached=None,
                     want_logits: bool = False, req_ids=None, stream=None, out=None):
        """syn_verify_batch with HOST metadata.  Returns (accept_len, correction_token[, logits]).
        `out`: optional pair of int32 CPU tensors [n_req] to receive the results."""
        tok, off, ctx = _i32(chunk_tokens), _i32(chunk_offsets), _i32(ctx_lens)
        pt = _i32(page_tables)
        assert pt.dim() == 2
        n_req = ctx.numel()
        unc = _i32(n_uncached) if n_uncached is not None else None
        acc, cor = out if out is not None else (torch.empty(n_req, dtype=torch.int32), torch.empty(n_req, dtype=torch.int32))
        assert acc.dtype == torch.int32 and cor.dtype == torch.int32 and not acc.is_cuda and acc.numel() >= n_req
        logits = None
        if want_logits:
            logits = torch.empty(int(off[-1]), self.model.shape.vocab, dtype=torch.float32, device="cuda")
        ids = torch.as_tensor(req_ids, dtype=torch.int64).contiguous() if req_ids is not None else None
        _check(self._lib.syn_verify_batch(
            self.model._h, self._h, C.c_int32(n_req), C.c_void_p(ids.data_ptr()) if ids is not None else None,
            C.c_void_p(tok.data_ptr()), C.c_void_p(off.data_ptr()), C.c_void_p(pt.data_ptr()), C.c_int32(pt.shape[1]),
            C.c_void_p(ctx.data_ptr()), C.c_void_p(unc.data_ptr()) if unc is not None else None,
            C.c_void_p(acc.data_ptr()), C.c_void_p(cor.data_ptr()),
            C.c_void_p(logits.data_ptr()) if logits is not None else None, _stream_ptr(stream)), "syn_verify_batch")
        return (acc, cor, logits) if want_logits else (acc, cor)


class Sampling(C.Structure):
    """syn_sampling: the LLM's sampling method and the width of the transmitted SLM rows."""
    _fields_ = [("top_k", C.c_int32), ("top_p", C.c_float), ("temperature", C.c_float), ("slm_k", C.c_int32)]


def _f32(t) -> torch.Tensor:
    return torch.as_tensor(t, dtype=torch.float32, device="cpu").contiguous()


def verify_batch_sampled(kv: "KVCache", chunk_tokens, chunk_offsets, page_tables, ctx_lens, n_uncached, cfg: Sampling,
                         slm_ids, slm_probs, rand_accept, rand_sample, want_logits: bool = False, stream=None):
    """syn_verify_batch_sampled with HOST metadata.  Returns (accept_len, correction_token[, logits])."""
    tok, off, ctx, pt = _i32(chunk_tokens), _i32(chunk_offsets), _i32(ctx_lens), _i32(page_tables)
    n_req = ctx.numel()
    unc = _i32(n_uncached) if n_uncached is not None else None
    sid, sp, ra, rs = _i32(slm_ids), _f32(slm_probs), _f32(rand_accept), _f32(rand_sample)
    acc = torch.empty(n_req, dtype=torch.int32)
    cor = torch.empty(n_req, dtype=torch.int32)
    logits = torch.empty(int(off[-1]), kv.model.shape.vocab, dtype=torch.float32, device="cuda") if want_logits else None
    _check(load_library().syn_verify_batch_sampled(
        kv.model._h, kv._h, C.c_int32(n_req), None, C.c_void_p(tok.data_ptr()), C.c_void_p(off.data_ptr()),
        C.c_void_p(pt.data_ptr()), C.c_int32(pt.shape[1]), C.c_void_p(ctx.data_ptr()),
        C.c_void_p(unc.data_ptr()) if unc is not None else None, C.byref(cfg), C.c_void_p(sid.data_ptr()),
        C.c_void_p(sp.data_ptr()), C.c_void_p(ra.data_ptr()), C.c_void_p(rs.data_ptr()), C.c_void_p(acc.data_ptr()),
        C.c_void_p(cor.data_ptr()), C.c_void_p(logits.data_ptr()) if logits is not None else None, _stream_ptr(stream)),
        "syn_verify_batch_sampled")
    return (acc, cor, logits) if want_logits else (acc, cor)


def syn_op_sample_verify(logits: torch.Tensor, chunk_tokens, chunk_offsets, n_uncached, cfg: Sampling, slm_ids, slm_probs,
                         rand_accept, rand_sample, stream=None):
    """The sampling stage alone on device logits fp32 [T, vocab].  Returns (accept_len, correction_token)."""
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
    tok, off, unc = _i32(chunk_tokens), _i32(chunk_offsets), _i32(n_uncached)
    sid, sp, ra, rs = _i32(slm_ids), _f32(slm_probs), _f32(rand_accept), _f32(rand_sample)
    n_req = unc.numel()
    acc = torch.empty(n_req, dtype=torch.int32)
    cor = torch.empty(n_req, dtype=torch.int32)
    _check(load_library().syn_op_sample_verify(
        C.c_void_p(logits.data_ptr()), C.c_int32(logits.shape[0]), C.c_int32(logits.shape[1]), C.c_int32(n_req),
        C.c_void_p(tok.data_ptr()), C.c_void_p(off.data_ptr()), C.c_void_p(unc.data_ptr()), C.byref(cfg),
        C.c_void_p(sid.data_ptr()), C.c_void_p(sp.data_ptr()), C.c_void_p(ra.data_ptr()), C.c_void_p(rs.data_ptr()),
        C.c_void_p(acc.data_ptr()), C.c_void_p(cor.data_ptr()), _stream_ptr(stream)), "syn_op_sample_verify")
    return acc, cor


class Plan:
    """syn_plan_create / syn_verify_run / syn_op_attention / syn_plan_stats / syn_plan_free."""

    def __init__(self, kv: KVCache, chunk_tokens, chunk_offsets, page_tables, ctx_lens, n_uncached=None):
        self._lib = load_library()
        self.kv = kv
        tok, off, ctx, pt = _i32(chunk_tokens), _i32(chunk_offsets), _i32(ctx_lens), _i32(page_tables)
        unc = _i32(n_uncached) if n_uncached is not None else None
        self.n_req, self.n_tokens = ctx.numel(), int(off[-1])
        self._h = C.c_void_p()
        _check(self._lib.syn_plan_create(
            kv.model._h, kv._h, C.c_int32(self.n_req), C.c_void_p(tok.data_ptr()), C.c_void_p(off.data_ptr()),
            C.c_void_p(pt.data_ptr()), C.c_int32(pt.shape[1]), C.c_void_p(ctx.data_ptr()),
            C.c_void_p(unc.data_ptr()) if unc is not None else None, C.byref(self._h)), "syn_plan_create")

    def stats(self) -> StepStats:
        s = StepStats()
        _check(self._lib.syn_plan_stats(self._h, C.byref(s)), "syn_plan_stats")
        return s

    def run(self, accept_len: torch.Tensor, correction: torch.Tensor, top1: Optional[torch.Tensor] = None,
            logits: Optional[torch.Tensor] = None, stream=None) -> None:
        """syn_verify_run: asynchronous, DEVICE int32 outputs."""
        assert accept_len.is_cuda and correction.is_cuda and accept_len.dtype == torch.int32
        _check(self._lib.syn_verify_run(
            self.kv.model._h, self.kv._h, self._h, C.c_void_p(accept_len.data_ptr()), C.c_void_p(correction.data_ptr()),
            C.c_void_p(top1.data_ptr()) if top1 is not None else None,
            C.c_void_p(logits.data_ptr()) if logits is not None else None, _stream_ptr(stream)), "syn_verify_run")

    def attention(self, layer: int, q: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """syn_op_attention: q and the result are half precision [T, n_q_heads * head_dim]."""
        assert q.is_cuda and q.dtype == torch.float16 and q.is_contiguous()
        if out is None:
            out = torch.empty_like(q)
        _check(self._lib.syn_op_attention(self.kv.model._h, self.kv._h, self._h, C.c_uint32(layer),
                                          C.c_void_p(q.data_ptr()), C.c_void_p(out.data_ptr()), _stream_ptr(stream)),
               "syn_op_attention")
        return out

    def attention_static(self, layer: int, q: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """syn_op_attention_static: the attention of the step for callers that cannot allocate while
        they run; its partial results live in a fixed array inside the library.  Pass `out` to keep
        the call itself free of allocations on the Python side too."""
        assert q.is_cuda and q.dtype == torch.float16 and q.is_contiguous()
        if out is None:
            out = torch.empty_like(q)
        _check(self._lib.syn_op_attention_static(self.kv.model._h, self.kv._h, self._h, C.c_uint32(layer),
                                                 C.c_void_p(q.data_ptr()), C.c_void_p(out.data_ptr()),
                                                 _stream_ptr(stream)), "syn_op_attention_static")
        return out

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.syn_plan_free(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


PLAN_ITEM_FIELDS = ("q_tok", "nj", "kvh", "req", "kv_begin", "kv_end", "q_pos0", "part", "grp")


def plan_host(shape, n_pages: int, chunk_tokens, chunk_offsets, page_tables, ctx_lens, n_uncached=None,
              n_sm: int = 148, page_size: int = 16):
    """syn_plan_host: the host planner without a device.  Returns a dict with pos, slot [T],
    items [n_items, 9] (columns PLAN_ITEM_FIELDS), cta_begin [n_cta + 1] and stats."""
    lib = load_library()
    tok, off, ctx, pt = _i32(chunk_tokens), _i32(chunk_offsets), _i32(ctx_lens), _i32(page_tables)
    assert pt.dim() == 2
    unc = _i32(n_uncached) if n_uncached is not None else None
    n_req = ctx.numel()
    T = max(0, int(off[-1])) if off.numel() else 0
    d = _Desc(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
              shape.vocab, float(shape.rope_base), float(shape.rms_eps), 0)
    pos = torch.zeros(max(T, 1), dtype=torch.int32)
    slot = torch.zeros(max(T, 1), dtype=torch.int32)
    cta = torch.zeros(n_sm + 1, dtype=torch.int32)
    n_items, n_cta = C.c_int32(0), C.c_int32(0)
    st = StepStats()
    cap = 0
    items = torch.zeros(1, len(PLAN_ITEM_FIELDS), dtype=torch.int32)
    for _ in range(2):
        code = lib.syn_plan_host(
            C.byref(d), C.c_uint32(n_pages), C.c_uint32(page_size), C.c_int32(n_sm), C.c_int32(n_req),
            C.c_void_p(tok.data_ptr()), C.c_void_p(off.data_ptr()), C.c_void_p(pt.data_ptr()), C.c_int32(pt.shape[1]),
            C.c_void_p(ctx.data_ptr()), C.c_void_p(unc.data_ptr()) if unc is not None else None,
            C.c_void_p(pos.data_ptr()), C.c_void_p(slot.data_ptr()), C.c_void_p(items.data_ptr()) if cap else None,
            C.c_int32(cap), C.byref(n_items), C.c_void_p(cta.data_ptr()), C.byref(n_cta), C.byref(st))
        _check(code, "syn_plan_host")
        if cap:
            break
        cap = n_items.value
        items = torch.zeros(max(cap, 1), len(PLAN_ITEM_FIELDS), dtype=torch.int32)
    return {"pos": pos[:T], "slot": slot[:T], "items": items[:n_items.value], "cta_begin": cta[:n_cta.value + 1],
            "n_cta": n_cta.value, "stats": st}


# ------------------------------------------------------------------------------------------ scheduler

SCHED_KINDS = ("idle", "prefill", "verify")


class _SchedBatch(C.Structure):
    _fields_ = [("kind", C.c_int32), ("n_req", C.c_int32), ("n_tokens", C.c_int32), ("max_pages", C.c_int32),
                ("req_ids", C.POINTER(C.c_int64)), ("chunk_tokens", C.POINTER(C.c_int32)),
                ("chunk_offsets", C.POINTER(C.c_int32)), ("page_tables", C.POINTER(C.c_int32)),
                ("ctx_lens", C.POINTER(C.c_int32)), ("n_uncached", C.POINTER(C.c_int32))]


class _SchedResult(C.Structure):
    _fields_ = [("req_id", C.c_int64)] + [(n, C.c_int32) for n in ("kind", "n_tokens", "accept_len", "correction_token",
                                                                    "ctx_len", "prompt_done")]


class SchedStats(C.Structure):
    _fields_ = [("iterations", C.c_int64 * 3), ("tokens", C.c_int64 * 3), ("requests", C.c_int64 * 3),
                ("deferred", C.c_int64), ("host_seconds", C.c_double), ("execute_seconds", C.c_double),
                ("live_requests", C.c_int32), ("free_pages", C.c_int32)]


class Scheduler:
    """syn_sched_*: the verification-aware scheduler over one KV cache, or, with ``kv=None``, its
    policy alone (peek / commit without a device)."""

    def __init__(self, kv: Optional["KVCache"], n_pages: Optional[int] = None, page_size: int = 16,
                 max_batch_tokens: int = 2048):
        self._lib = load_library()
        self.kv = kv
        if kv is not None:
            n_pages, page_size = kv.n_pages, kv.page_size
        self._h = C.c_void_p()
        _check(self._lib.syn_sched_create(kv.model._h if kv is not None else None, kv._h if kv is not None else None,
                                          C.c_uint32(n_pages), C.c_uint32(page_size), C.c_int32(max_batch_tokens),
                                          C.byref(self._h)), "syn_sched_create")
        self._cap = 0
        self._res = None

    def add_request(self, req_id: int, prompt) -> None:
        p = _i32(prompt)
        _check(self._lib.syn_sched_add_request(self._h, C.c_int64(req_id), C.c_void_p(p.data_ptr()), C.c_int32(p.numel())),
               "syn_sched_add_request")

    def add_verify(self, req_id: int, tokens, n_uncached: int = 1) -> None:
        t = _i32(tokens)
        _check(self._lib.syn_sched_add_verify(self._h, C.c_int64(req_id), C.c_void_p(t.data_ptr()), C.c_int32(t.numel()),
                                              C.c_int32(n_uncached)), "syn_sched_add_verify")

    def finish(self, req_id: int) -> None:
        _check(self._lib.syn_sched_finish(self._h, C.c_int64(req_id)), "syn_sched_finish")

    def peek(self) -> Dict[str, object]:
        """The next iteration's batch, copied into tensors (page_tables [n_req, max_pages])."""
        b = _SchedBatch()
        _check(self._lib.syn_sched_peek(self._h, C.byref(b)), "syn_sched_peek")
        out = {"kind": SCHED_KINDS[b.kind], "n_req": b.n_req, "n_tokens": b.n_tokens, "max_pages": b.max_pages}
        if b.kind == 0:
            return out
        B = b.n_req
        out["req_ids"] = [b.req_ids[i] for i in range(B)]
        out["chunk_offsets"] = torch.tensor([b.chunk_offsets[i] for i in range(B + 1)], dtype=torch.int32)
        out["chunk_tokens"] = torch.tensor([b.chunk_tokens[i] for i in range(b.n_tokens)], dtype=torch.int32)
        out["page_tables"] = torch.tensor([b.page_tables[i] for i in range(B * b.max_pages)],
                                          dtype=torch.int32).view(B, b.max_pages)
        out["ctx_lens"] = torch.tensor([b.ctx_lens[i] for i in range(B)], dtype=torch.int32)
        out["n_uncached"] = torch.tensor([b.n_uncached[i] for i in range(B)], dtype=torch.int32)
        return out

    def _results(self, n: int) -> List[Dict[str, int]]:
        return [{f: getattr(self._res[i], f) for f, _ in _SchedResult._fields_} for i in range(n)]

    def _room(self, n: int) -> None:
        if n > self._cap:
            self._cap = max(n, 64)
            self._res = (_SchedResult * self._cap)()

    def commit(self, accept_len=None, correction_token=None) -> List[Dict[str, int]]:
        a = _i32(accept_len) if accept_len is not None else None
        c = _i32(correction_token) if correction_token is not None else None
        self._room(a.numel() if a is not None else 1)
        n = C.c_int32(0)
        _check(self._lib.syn_sched_commit(self._h, C.c_void_p(a.data_ptr()) if a is not None else None,
                                          C.c_void_p(c.data_ptr()) if c is not None else None, self._res,
                                          C.c_int32(self._cap), C.byref(n)), "syn_sched_commit")
        return self._results(n.value)

    def step(self, stream=None, max_results: int = 4096):
        """One iteration: (kind, results)."""
        self._room(max_results)
        n, kind = C.c_int32(0), C.c_int32(0)
        sp = _stream_ptr(stream) if self.kv is not None else None   # without a model the library refuses the call
        _check(self._lib.syn_sched_step(self._h, self._res, C.c_int32(self._cap), C.byref(n), C.byref(kind), sp),
               "syn_sched_step")
        return SCHED_KINDS[kind.value], self._results(n.value)

    def stats(self) -> SchedStats:
        st = SchedStats()
        _check(self._lib.syn_sched_get_stats(self._h, C.byref(st)), "syn_sched_get_stats")
        return st

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.syn_sched_free(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


GEMM_PLAN_FIELDS = ("n_pairs", "n_tt", "TN", "num_kb", "n_cta", "pair_mode", "splits", "kb_per_split", "ksplit", "kper")
GEMM_WORK_FIELDS = ("pair", "tt", "mt_lo", "mt_hi", "kb0", "kb1", "split", "role", "rtile", "hpart")
GEMM_EPILOGUES = {"plain": 0, "qkv": 1, "resid": 2, "swiglu": 3, "lmhead": 4}
# syn_op_linear_as only: the CTA-pair kernel with 512-feature (quad) or 256-feature (duo) items, as a
# plain projection or as a residual projection (K shared between clusters where the shape allows it)
LINEAR_SCHEDULES = dict(GEMM_EPILOGUES, pair_quad=5, pair_duo=6, pair_quad_resid=7, pair_duo_resid=8)


def gemm_plan_host(T: int, N: int, K: int, epilogue: str, n_sm: int = 148) -> Dict[str, int]:
    """syn_gemm_plan_host: the launch shape of one projection, without a device."""
    out = (C.c_int32 * len(GEMM_PLAN_FIELDS))()
    _check(load_library().syn_gemm_plan_host(C.c_int32(T), C.c_int32(N), C.c_int32(K), C.c_int32(n_sm),
                                             C.c_int32(GEMM_EPILOGUES[epilogue]), out), "syn_gemm_plan_host")
    return dict(zip(GEMM_PLAN_FIELDS, out))


def gemm_work_host(T: int, N: int, K: int, epilogue: str, cta: int, i: int, n_sm: int = 148) -> Optional[Dict[str, int]]:
    """syn_gemm_work_host: work item i of CTA cta, or None."""
    out = (C.c_int32 * len(GEMM_WORK_FIELDS))()
    r = load_library().syn_gemm_work_host(C.c_int32(T), C.c_int32(N), C.c_int32(K), C.c_int32(n_sm),
                                          C.c_int32(GEMM_EPILOGUES[epilogue]), C.c_int32(cta), C.c_int32(i), out)
    if r < 0:
        _check(r, "syn_gemm_work_host")
    return dict(zip(GEMM_WORK_FIELDS, out)) if r == 1 else None


GEMM2_PLAN_FIELDS = ("kind", "n_groups", "n_tt", "TN", "num_kb", "n_clusters", "splits", "kb_per_split", "rem_base", "rem_extra")
GEMM2_WORK_FIELDS = ("grp", "tt", "kb0", "kb1", "tile", "split", "nsplit", "first_cl", "counter")
GEMM2_KINDS = {"auto": 0, "quad": 1, "duo": 2}


def gemm2_plan_host(T: int, N: int, K: int, epilogue: str, force: str = "auto", n_sm: int = 148) -> Dict[str, int]:
    """syn_gemm2_plan_host: the launch shape of one projection on CTA pairs, without a device."""
    out = (C.c_int32 * len(GEMM2_PLAN_FIELDS))()
    _check(load_library().syn_gemm2_plan_host(C.c_int32(T), C.c_int32(N), C.c_int32(K), C.c_int32(n_sm),
                                              C.c_int32(GEMM_EPILOGUES[epilogue]), C.c_int32(GEMM2_KINDS[force]), out),
           "syn_gemm2_plan_host")
    return dict(zip(GEMM2_PLAN_FIELDS, out))


def gemm2_work_host(T: int, N: int, K: int, epilogue: str, cluster: int, i: int, force: str = "auto",
                    n_sm: int = 148) -> Optional[Dict[str, int]]:
    """syn_gemm2_work_host: work item i of a cluster, or None."""
    out = (C.c_int32 * len(GEMM2_WORK_FIELDS))()
    r = load_library().syn_gemm2_work_host(C.c_int32(T), C.c_int32(N), C.c_int32(K), C.c_int32(n_sm),
                                           C.c_int32(GEMM_EPILOGUES[epilogue]), C.c_int32(GEMM2_KINDS[force]),
                                           C.c_int32(cluster), C.c_int32(i), out)
    if r < 0:
        _check(r, "syn_gemm2_work_host")
    return dict(zip(GEMM2_WORK_FIELDS, out)) if r == 1 else None


def syn_op_linear(x: torch.Tensor, w: torch.Tensor, stream=None, schedule_as: str = "plain",
                  reuse_pack: bool = False) -> torch.Tensor:
    """y[T, N] fp32 = x[T, K] half @ w[N, K]^T bf16 through the library's tcgen05 GEMM, under the
    schedule the step uses for the projection with epilogue `schedule_as`.  The library keeps a packed
    copy of the last w keyed by address and shape; unless `reuse_pack` says the matrix is the one of the
    previous call, the copy is dropped first (a new tensor may sit at a freed tensor's address)."""
    assert x.is_cuda and w.is_cuda and x.dtype == torch.float16 and w.dtype == torch.bfloat16
    x, w = x.contiguous(), w.contiguous()
    T, K = x.shape
    N = w.shape[0]
    y = torch.empty(T, N, dtype=torch.float32, device="cuda")
    lib = load_library()
    if not reuse_pack:
        _check(lib.syn_op_linear_reset(), "syn_op_linear_reset")
    _check(lib.syn_op_linear_as(C.c_void_p(x.data_ptr()), C.c_void_p(w.data_ptr()), C.c_void_p(y.data_ptr()),
                                C.c_int32(T), C.c_int32(N), C.c_int32(K), C.c_int32(LINEAR_SCHEDULES[schedule_as]),
                                _stream_ptr(stream)), "syn_op_linear_as")
    return y


def debug_set_spin_limit(cycles: int) -> None:
    """syn_debug_set_spin_limit: SM cycles after which a wait inside the projection kernels gives up (0: default)."""
    _check(load_library().syn_debug_set_spin_limit(C.c_int64(cycles)), "syn_debug_set_spin_limit")


def debug_set_schedule(which: int) -> None:
    """syn_debug_set_schedule: 0 automatic, 1 every projection on the one-CTA kernel."""
    _check(load_library().syn_debug_set_schedule(C.c_int32(which)), "syn_debug_set_schedule")


def debug_set_attention(which: int) -> None:
    """syn_debug_set_attention: 0 default, 1 warp-level-MMA kernel, 2 tcgen05 kernel; applies to plans made afterwards."""
    _check(load_library().syn_debug_set_attention(C.c_int32(which)), "syn_debug_set_attention")


def debug_linear_counter(index: int, value: int) -> None:
    """syn_debug_linear_counter: overwrite one arrival counter of syn_op_linear's workspace."""
    _check(load_library().syn_debug_linear_counter(C.c_int32(index), C.c_int32(value)), "syn_debug_linear_counter")
