"""Device-side set-up of the seeded synthetic workloads: weights generated on the GPU,
the cached prefix written through syn_kv_import, the batch laid out by the shared generators.
Used by the benchmark, the smoke check and the full-size GPU tests.  No CPU fallback."""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import torch

from workloads import gen
from workloads.configs import ModelShape, Workload

from .binding import KVCache, Model, Plan


def load_model(shape: ModelShape, seed: int, via_host: bool = False) -> Model:
    """Generate every matrix on the GPU and hand it to syn_model_load.  `via_host` parks the
    generated layers in host memory first, so that the caller's copy and the library's packed
    copy never sit in HBM together (needed for the 32B shape)."""
    dev = "cpu" if via_host else "cuda"

    def place(d: Dict[str, torch.Tensor]):
        return {k: v.to(dev) for k, v in d.items()}

    glob = place(gen.gen_globals(shape, seed, device="cuda"))
    layers = [place(gen.gen_layer(shape, seed, l, device="cuda")) for l in range(shape.n_layers)]
    model = Model(shape, glob, layers)
    del glob, layers
    torch.cuda.empty_cache()
    return model


def fill_cache(kv: KVCache, shape: ModelShape, seed: int, batch: gen.Batch, reqs: Optional[Sequence[int]] = None) -> None:
    """Cached prefix of every request = seeded synthetic K/V keyed by logical position."""
    for r in (range(batch.n_req) if reqs is None else reqs):
        ctx = int(batch.ctx_lens[r])
        if ctx == 0:
            continue
        pt = batch.page_tables[r]
        for l in range(shape.n_layers):
            k, v = gen.gen_kv(shape, seed, l, r, 0, ctx, device="cuda")
            kv.import_kv(l, pt, 0, k, v)


def teacher_forced_chunks(kv: KVCache, wl: Workload, batch: gen.Batch, fixed: Optional[Dict[int, List[int]]] = None):
    """Chunk tokens of the whole batch by the sequential draft rule (u accepted tokens: the anchor,
    then uniform ids; then drafts), with the argmax supplied by the library itself (one pass per
    chunk index that precedes a draft).  Requests listed in `fixed` keep the given tokens (e.g.
    chunks whose drafts a test derived by other means)."""
    fixed = fixed or {}
    B = batch.n_req
    offs = batch.chunk_offsets.tolist()
    unc = batch.n_uncached.tolist()
    toks = torch.zeros(batch.n_tokens, dtype=torch.int32)
    for r in range(B):
        if r in fixed:
            toks[offs[r]:offs[r + 1]] = torch.tensor(fixed[r], dtype=torch.int32)
        else:
            toks[offs[r]] = gen.gen_anchor(wl, r)
            if unc[r] > 1:
                toks[offs[r] + 1:offs[r] + unc[r]] = gen.gen_context_tokens(wl, r, unc[r] - 1)
    acc = torch.empty(B, dtype=torch.int32, device="cuda")
    cor = torch.empty(B, dtype=torch.int32, device="cuda")
    top1 = torch.empty(batch.n_tokens, dtype=torch.int32, device="cuda")
    n_max = int(batch.chunk_lens.max())
    for j in range(n_max - 1):
        todo = [r for r in range(B) if r not in fixed and unc[r] <= j + 1 < offs[r + 1] - offs[r]]
        if not todo:
            continue
        plan = Plan(kv, toks, batch.chunk_offsets, batch.page_tables, batch.ctx_lens, batch.n_uncached)
        plan.run(acc, cor, top1)
        torch.cuda.synchronize()
        t1 = top1.cpu()
        plan.close()
        for r in todo:
            toks[offs[r] + j + 1] = gen.gen_draft(wl, r, j + 1 - unc[r], int(t1[offs[r] + j]))
    return toks
