"""Seeded synthetic inputs: weights, request lengths, page tables, cached KV, tokens, drafts.

Everything is keyed, not sequential, so any slice can be regenerated anywhere
(per layer, per request) without holding the whole workload.  No arithmetic of
the verification step lives here: a draft is built from an argmax that the
caller supplies.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Dict, List, Optional

import torch

from . import rng
from .configs import ModelShape, Workload

# stream purposes
S_WEIGHT, S_GAIN, S_CTXLEN, S_CHUNKLEN, S_PAGES, S_KV, S_CTXTOK, S_ANCHOR, S_DRAFT_U, S_DRAFT_T, S_MIX = range(11)

_WNAMES = {"embed": 0, "lm_head": 1, "wq": 2, "wk": 3, "wv": 4, "wo": 5, "wg": 6, "wu": 7, "wd": 8}
_GNAMES = {"final_norm": 0, "norm1": 1, "norm2": 2}
_CHUNK = 1 << 24


def weight_shape(shape: ModelShape, name: str):
    """[out_features, in_features] of a projection; tables are [vocab, d_model]."""
    d, f = shape.d_model, shape.d_ffn
    return {"embed": (shape.vocab, d), "lm_head": (shape.vocab, d),
            "wq": (shape.q_dim, d), "wk": (shape.kv_dim, d), "wv": (shape.kv_dim, d),
            "wo": (d, shape.q_dim), "wg": (f, d), "wu": (f, d), "wd": (d, f)}[name]


def gen_weight(shape: ModelShape, seed: int, name: str, layer: int = 0, device="cpu") -> torch.Tensor:
    """bf16 [out, in] matrix, N(0, weight_std) drawn in fp32 then rounded to nearest-even."""
    rows, cols = weight_shape(shape, name)
    key = rng.stream_key(seed, S_WEIGHT, _WNAMES[name], layer)
    n = rows * cols
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    for s in range(0, n, _CHUNK):
        c = min(_CHUNK, n - s)
        out[s:s + c] = rng.normal_f32(key, s, c, shape.weight_std, device=device).to(torch.bfloat16)
    return out.view(rows, cols)


def gen_gain(shape: ModelShape, seed: int, name: str, layer: int = 0, device="cpu") -> torch.Tensor:
    """bf16 [d_model] RMSNorm gain, 1 + gain_std * N(0,1)."""
    key = rng.stream_key(seed, S_GAIN, _GNAMES[name], layer)
    return rng.normal_f32(key, 0, shape.d_model, shape.gain_std, 1.0, device=device).to(torch.bfloat16)


LAYER_WEIGHTS = ("wq", "wk", "wv", "wo", "wg", "wu", "wd")
LAYER_GAINS = ("norm1", "norm2")


def gen_layer(shape: ModelShape, seed: int, layer: int, device="cpu") -> Dict[str, torch.Tensor]:
    out = {n: gen_weight(shape, seed, n, layer, device) for n in LAYER_WEIGHTS}
    out.update({n: gen_gain(shape, seed, n, layer, device) for n in LAYER_GAINS})
    return out


def gen_globals(shape: ModelShape, seed: int, device="cpu") -> Dict[str, torch.Tensor]:
    return {"embed": gen_weight(shape, seed, "embed", 0, device),
            "lm_head": gen_weight(shape, seed, "lm_head", 0, device),
            "final_norm": gen_gain(shape, seed, "final_norm", 0, device)}


# ----------------------------------------------------------------------------- request mix

def _draw_lengths(recipe, key_u: int, key_mix: int, n: int) -> List[int]:
    kind = recipe[0]
    if kind == "list":
        vals = list(recipe[1])
        assert len(vals) == n
        return vals
    if kind == "const":
        return [int(recipe[1])] * n
    if kind == "uniform":
        return rng.randint(key_u, 0, n, recipe[1], recipe[2]).tolist()
    if kind == "loguniform":
        lo, hi = recipe[1], recipe[2]
        u = rng.uniform01(key_u, 0, n)
        v = torch.exp(math.log(lo) + u * (math.log(hi) - math.log(lo))).round().clamp(lo, hi)
        return [int(x) for x in v.tolist()]
    if kind == "mix":
        u = rng.uniform01(key_mix, 0, n).tolist()
        r = rng.uniform01(key_u, 0, n).tolist()
        out = []
        for ui, ri in zip(u, r):
            acc = 0.0
            for w, lo, hi in recipe[1]:
                acc += w
                if ui < acc or (w, lo, hi) == recipe[1][-1]:
                    out.append(lo + min(int(ri * (hi - lo + 1)), hi - lo))
                    break
        return out
    raise ValueError(kind)


@dataclass
class Batch:
    """Host-side description of one verification batch (all int32 CPU tensors)."""
    n_req: int
    page_size: int
    n_pages: int
    ctx_lens: torch.Tensor        # [B]
    chunk_lens: torch.Tensor      # [B]
    chunk_offsets: torch.Tensor   # [B+1]
    page_tables: torch.Tensor     # [B, max_pages]
    max_pages: int
    n_uncached: torch.Tensor      # [B]
    scale: float = 1.0            # common context factor applied by the fit rule

    @property
    def n_tokens(self) -> int:
        return int(self.chunk_offsets[-1])


def gen_batch(wl: Workload, pool_tokens: Optional[int] = None, n_req: Optional[int] = None) -> Batch:
    """Draw lengths and lay out pages.

    Pages: one seeded permutation of all physical page ids, dealt round-robin (logical
    page k of each request in turn), so logical neighbours are never physical neighbours
    and every request's pages are interleaved with everyone else's.  Unused table
    entries hold -1.
    ``pool_tokens`` (fit rule): if the demand exceeds it, every context is multiplied
    by the common factor capacity/demand (floored).
    """
    B = wl.n_req if n_req is None else n_req
    P = wl.page_size
    ctx = _draw_lengths(wl.ctx, rng.stream_key(wl.seed, S_CTXLEN), rng.stream_key(wl.seed, S_MIX, 0), wl.n_req)[:B]
    chunk = _draw_lengths(wl.chunk, rng.stream_key(wl.seed, S_CHUNKLEN), rng.stream_key(wl.seed, S_MIX, 1), wl.n_req)[:B]
    scale = 1.0
    if wl.fit_to_pool and pool_tokens is not None:
        need = sum(-(-(c + n) // P) * P for c, n in zip(ctx, chunk))
        if need > pool_tokens:
            scale = pool_tokens / need
            while True:
                ctx2 = [max(1, int(c * scale)) for c in ctx]
                if sum(-(-(c + n) // P) * P for c, n in zip(ctx2, chunk)) <= pool_tokens:
                    break
                scale *= 0.999
            ctx = ctx2
    pages_per_req = [-(-(c + n) // P) for c, n in zip(ctx, chunk)]
    max_pages = max(pages_per_req)
    n_pages = sum(pages_per_req)
    perm = rng.permutation(rng.stream_key(wl.seed, S_PAGES), n_pages).to(torch.int32)
    # deal the permuted ids round-robin: logical page k of every request that still needs one
    need = torch.tensor(pages_per_req)
    live = (torch.arange(max_pages).view(-1, 1) < need.view(1, -1))          # [max_pages, B]
    table = torch.full((max_pages, B), -1, dtype=torch.int32)
    table[live] = perm
    table = table.t().contiguous()                                          # [B, max_pages], -1 = unused
    offs = [0]
    for n in chunk:
        offs.append(offs[-1] + n)
    return Batch(B, P, n_pages, torch.tensor(ctx, dtype=torch.int32), torch.tensor(chunk, dtype=torch.int32),
                 torch.tensor(offs, dtype=torch.int32), table, max_pages,
                 torch.tensor([1 if wl.n_drafts is None else max(1, n - wl.n_drafts) for n in chunk], dtype=torch.int32),
                 scale)


# ----------------------------------------------------------------------------- cached KV and tokens

def gen_kv(shape: ModelShape, seed: int, layer: int, req: int, pos0: int, npos: int, device="cpu"):
    """Synthetic cached K and V for positions [pos0, pos0+npos) of one request and layer.

    bf16 [npos, n_kv_heads, head_dim] each, i.i.d. N(0, (weight_std * sqrt(d_model))^2): the
    scale a projection of a unit-RMS vector has under these weights.  Keyed by logical
    position, so the values do not depend on where the pages land.
    """
    std = shape.weight_std * math.sqrt(shape.d_model)
    per = shape.kv_dim
    out = []
    for which in (0, 1):
        key = rng.stream_key(seed, S_KV, layer, req, which)
        out.append(rng.normal_f32(key, pos0 * per, npos * per, std, device=device)
                   .to(torch.bfloat16).view(npos, shape.n_kv_heads, shape.head_dim))
    return out[0], out[1]


def gen_context_tokens(wl: Workload, req: int, n: int) -> torch.Tensor:
    """Uniform-random context token ids of one request (int32)."""
    return rng.randint(rng.stream_key(wl.seed, S_CTXTOK, req), 0, n, 0, wl.shape.vocab - 1).to(torch.int32)


def gen_anchor(wl: Workload, req: int) -> int:
    """The first chunk token (device-accepted, not a draft): uniform over the vocabulary."""
    return int(rng.randint(rng.stream_key(wl.seed, S_ANCHOR), req, 1, 0, wl.shape.vocab - 1)[0])


def gen_draft(wl: Workload, req: int, j: int, target_top1: int) -> int:
    """Draft number j (0-based) of a request: the supplied argmax with probability
    p_match, otherwise uniform over the vocabulary (which may coincide with it)."""
    u = float(rng.uniform01(rng.stream_key(wl.seed, S_DRAFT_U, req), j, 1)[0])
    if u < wl.p_match:
        return int(target_top1)
    return int(rng.randint(rng.stream_key(wl.seed, S_DRAFT_T, req), j, 1, 0, wl.shape.vocab - 1)[0])
