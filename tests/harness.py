"""Shared machinery of the GPU parity tests: build the same seeded batch on both sides,
run the CPU oracle request by request, and judge the CUDA result by the stated rule.

Parity rule: accept_len and correction_token bit-exact, except that a chunk
position whose oracle top-2 logit gap is below 0.05 ("soft") may resolve to either of the
oracle's two best ids; logits within 3e-2 x the standard deviation of the oracle's logits.
"""
from __future__ import annotations

import itertools
from dataclasses import dataclass
from typing import Callable, Dict, List, Optional, Sequence

import numpy as np
import torch

from oracle import Oracle, verify_greedy
from workloads import gen
from workloads.configs import ModelShape, Workload

SOFT_GAP = 0.05
LOGIT_TOL = 3e-2


@dataclass
class OracleRequest:
    chunk: List[int]
    u: int
    top1: np.ndarray
    top2: np.ndarray
    gap: np.ndarray
    logits: Optional[np.ndarray]
    accept_len: int
    correction: int


def oracle_teacher_forced(orc: Oracle, glob, layer_w: Callable[[int], dict], pools, page_table, ctx: int, wl: Workload,
                          req: int, n: int, want_logits=True, u: int = 1,
                          head: Optional[Sequence[int]] = None) -> OracleRequest:
    """Build request `req`'s chunk by the sequential rule (u device-accepted tokens: the anchor, then
    uniform ids; draft j = the oracle's argmax after the actual earlier chunk tokens with
    probability p_match, else uniform) while running the oracle token by token, which is
    bit-identical to its one-shot chunk forward."""
    assert 1 <= u <= n
    if head is not None:   # the accepted tokens are given (a running draft-and-verify loop)
        assert len(head) == u
        chunk = [int(x) for x in head]
    else:
        chunk = [gen.gen_anchor(wl, req)] + [int(x) for x in gen.gen_context_tokens(wl, req, u - 1)]
    t1, t2, gp, lg = [], [], [], []
    for j in range(n):
        r = orc.forward_chunk(glob, layer_w, pools, page_table, ctx + j, [chunk[j]], u=1, want_logits=want_logits)
        t1.append(int(r.top1[0])); t2.append(int(r.top2[0])); gp.append(float(r.gap[0]))
        if want_logits:
            lg.append(r.logits[0])
        if u <= j + 1 < n:
            chunk.append(gen.gen_draft(wl, req, j + 1 - u, int(r.top1[0])))
    a, c = verify_greedy(t1, chunk, u)
    return OracleRequest(chunk, u, np.array(t1), np.array(t2), np.array(gp),
                         np.stack(lg) if want_logits else None, a, c)


def oracle_teacher_forced_many(orc: Oracle, glob, layer_w: Callable[[int], dict], wl: Workload, shape, seed: int,
                               batch: gen.Batch, picks: Sequence[int], want_logits=True) -> Dict[int, OracleRequest]:
    """oracle_teacher_forced for several requests at once, layer by layer, so that one layer's weights
    serve every request before the next layer's are fetched (the large shapes regenerate or page them).
    Token by token: step j forwards chunk token j of every listed request that has one (bit-identical to
    the one-shot chunk forward), then draws draft j + 1 from the oracle's argmax by the sequential rule.
    Each request gets its own contiguous page table and its seeded synthetic prefix."""
    st = {}
    for r in picks:
        ctx, n, u = int(batch.ctx_lens[r]), int(batch.chunk_lens[r]), int(batch.n_uncached[r])
        n_pages = -(-(ctx + n) // 16)
        pt = np.arange(n_pages, dtype=np.int32)
        pools = orc.new_pool(n_pages)
        for l in range(shape.n_layers):
            k, v = gen.gen_kv(shape, seed, l, r, 0, ctx)
            orc.load_kv(pools[l], pt, 0, k.float().numpy(), v.float().numpy())
        chunk = [gen.gen_anchor(wl, r)] + [int(x) for x in gen.gen_context_tokens(wl, r, u - 1)]
        st[r] = dict(ctx=ctx, n=n, u=u, pt=pt, pools=pools, chunk=chunk, t1=[], t2=[], gap=[], lg=[])
    for j in range(max(s["n"] for s in st.values())):
        live = [r for r in picks if j < st[r]["n"]]
        xs = {r: orc.embed(glob["embed"], [st[r]["chunk"][j]]) for r in live}
        for l in range(shape.n_layers):
            w = layer_w(l)
            for r in live:
                s = st[r]
                orc.layer(w, xs[r], s["pools"][l], s["pt"], s["ctx"] + j)
        for r in live:
            s = st[r]
            lg, t1, t2, gap = orc.logits(glob, xs[r], want_logits)
            s["t1"].append(int(t1[0])); s["t2"].append(int(t2[0])); s["gap"].append(float(gap[0]))
            if want_logits:
                s["lg"].append(lg[0].astype(np.float32))
            if s["u"] <= j + 1 < s["n"]:
                s["chunk"].append(gen.gen_draft(wl, r, j + 1 - s["u"], int(t1[0])))
    out = {}
    for r, s in st.items():
        a, c = verify_greedy(s["t1"], s["chunk"], s["u"])
        out[r] = OracleRequest(s["chunk"], s["u"], np.array(s["t1"]), np.array(s["t2"]), np.array(s["gap"]),
                               np.stack(s["lg"]) if want_logits else None, a, c)
    return out


def admissible_results(o: OracleRequest):
    """All (accept_len, correction) pairs reachable when every soft position may take either of the
    oracle's two best ids; and whether the request is strict (no soft position was consulted)."""
    n = len(o.chunk)
    soft = [j for j in range(n) if o.gap[j] < SOFT_GAP]
    consulted = range(o.u - 1, o.u - 1 + o.accept_len + 1)
    strict = not any(j in soft for j in consulted)
    out = set()
    for pick in itertools.product((0, 1), repeat=len(soft)):
        t = o.top1.copy()
        for j, b in zip(soft, pick):
            if b:
                t[j] = o.top2[j]
        out.add(verify_greedy(t, o.chunk, o.u))
    return out, strict


def judge(oracle_reqs: Sequence[OracleRequest], acc, cor, logits: Optional[torch.Tensor], offsets) -> Dict[str, float]:
    """Raises AssertionError on a parity violation; returns summary numbers."""
    n_strict = n_soft = 0
    for i, o in enumerate(oracle_reqs):
        ok, strict = admissible_results(o)
        got = (int(acc[i]), int(cor[i]))
        if strict:
            n_strict += 1
            assert got == (o.accept_len, o.correction), f"request {i}: got {got}, oracle {(o.accept_len, o.correction)}"
        else:
            n_soft += 1
            assert got in ok, f"request {i} (soft): got {got}, admissible {sorted(ok)}"
    worst = 0.0
    if logits is not None:
        ref = np.concatenate([o.logits for o in oracle_reqs])
        sigma = float(ref.std())
        g = logits.detach().to("cpu", torch.float64).numpy()
        for i, o in enumerate(oracle_reqs):
            b = int(offsets[i])
            worst = max(worst, float(np.abs(g[b:b + len(o.chunk)] - o.logits).max()) / sigma)
        assert worst <= LOGIT_TOL, f"max |dlogit| / sigma = {worst:.4f} > {LOGIT_TOL}"
    return {"strict": n_strict, "soft": n_soft, "max_dlogit_over_sigma": worst}


# ------------------------------------------------------------------------------------------ model / cache set-up

def cpu_model(shape: ModelShape, seed: int):
    glob = gen.gen_globals(shape, seed)
    layers = [gen.gen_layer(shape, seed, l) for l in range(shape.n_layers)]
    return glob, layers


def to_cuda(glob, layers):
    return ({k: v.cuda() for k, v in glob.items()}, [{k: v.cuda() for k, v in w.items()} for w in layers])


def fill_synthetic_kv(shape, seed, batch: gen.Batch, reqs: Sequence[int], kv=None, orc: Optional[Oracle] = None,
                      pools=None):
    """Cached prefix of the listed requests = seeded synthetic K/V (keyed by logical position).
    Fills the CUDA cache (values generated on the device) and/or the oracle pools (on the CPU)."""
    for r in reqs:
        ctx = int(batch.ctx_lens[r])
        if ctx == 0:
            continue
        pt = batch.page_tables[r]
        for l in range(shape.n_layers):
            if kv is not None:
                k, v = gen.gen_kv(shape, seed, l, r, 0, ctx, device="cuda")
                kv.import_kv(l, pt, 0, k, v)
            if orc is not None:
                k, v = gen.gen_kv(shape, seed, l, r, 0, ctx)
                orc.load_kv(pools[l], pt.numpy(), 0, k.float().numpy(), v.float().numpy())
