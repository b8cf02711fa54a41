"""Sampling-based verification, plain and slow (numpy, float64).

TEST INFRASTRUCTURE ONLY: imported by tests, never by the product package; shares no code with the
CUDA path.

What the paper fixes (Sec. 4.2, "Compression before transmission"): for verification the cloud LLM
needs the draft tokens and the SLM's distributions p(x | prefix), ..., and the device sends only the
most probable entries of each, as the sampling method in use (top-1, top-k or top-p) would keep
them.  The verification itself is the draft-and-verify procedure the paper builds on (Sec. 3.1,
speculative sampling of Leviathan et al. and Chen et al.): a draft x~ with SLM probability p(x~) is
kept with probability min(1, q(x~) / p(x~)) under the LLM's distribution q; at the first draft
that is not kept, the replacement is drawn from the normalised positive part of q - p; when every
draft is kept, one more token is drawn from q.  With top-1 on both sides this is the greedy rule.

Readings taken where the paper is silent:
  * q is the LLM's distribution as its sampling method keeps it: softmax(logits / temperature)
    over the top_k largest logits (ties: lower token id first), then, ordered by decreasing
    probability (ties: lower id first), the shortest prefix whose mass reaches top_p of the kept
    mass; renormalised.
  * p is what was transmitted: (token id, probability) pairs per draft, zero elsewhere; it is
    used as sent (the device has renormalised it).
  * The uniform draws are inputs: one per draft for the keep test (kept iff r * p(x~) < q(x~),
    which is r < min(1, q/p) for r in [0, 1)), one per request for the replacement / extra token,
    taken by inverse CDF over the candidate tokens in increasing token id.
  * If the positive part of q - p is empty (only possible through rounding), the replacement is
    the most probable token of q.

`margin` reports how close any consulted decision came to flipping (see verify_sampled); tests use
it to decide where two implementations in different precision must agree exactly.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence, Tuple

import numpy as np


def llm_distribution(logits: np.ndarray, top_k: int, top_p: float, temperature: float):
    """(ids, probs, boundary_gap, p_margin): the kept tokens in decreasing probability (ties:
    lower id first), their renormalised probabilities, the logit distance between the last kept
    and the first dropped token at the top-k boundary (inf if nothing was dropped there), and
    the distance of the top-p cut from moving by one token, as a fraction of the kept mass."""
    x = np.asarray(logits, dtype=np.float64)
    V = x.shape[0]
    k = min(top_k, V)
    order = np.lexsort((np.arange(V), -x))          # by logit descending, then id ascending
    kept = order[:k]
    gap = float(x[kept[-1]] - x[order[k]]) if k < V else float("inf")
    w = np.exp((x[kept] - x[kept[0]]) / temperature)
    total = w.sum()
    p_margin = float("inf")
    if top_p < 1.0:
        c = np.cumsum(w)
        m = int(np.searchsorted(c, top_p * total, side="left")) + 1   # shortest prefix with mass >= top_p * total
        m = min(m, k)
        near = [abs(c[m - 1] - top_p * total)] + ([abs(c[m - 2] - top_p * total)] if m >= 2 else [])
        p_margin = float(min(near) / total)
        kept, w = kept[:m], w[:m]
    return kept.astype(np.int64), w / w.sum(), gap, p_margin


def _inverse_cdf(ids: np.ndarray, weights: np.ndarray, r: float) -> Tuple[int, float]:
    """Token drawn by inverse CDF over `ids` in increasing id; and the relative distance of the
    draw from the nearest boundary between two candidates."""
    o = np.argsort(ids, kind="stable")
    ids, w = ids[o], weights[o]
    live = w > 0
    ids, w = ids[live], w[live]
    c = np.cumsum(w)
    t = r * c[-1]
    i = int(np.searchsorted(c, t, side="right"))
    i = min(i, len(ids) - 1)
    edges = c[:-1]
    dist = float(np.abs(edges - t).min() / c[-1]) if len(edges) else float("inf")
    return int(ids[i]), dist


@dataclass
class SampledResult:
    accept_len: int
    correction: int
    margin: float      # smallest relative distance of a consulted keep test / draw from flipping
    topk_gap: float    # smallest logit gap at a consulted top-k boundary


def verify_sampled(logits: np.ndarray, chunk: Sequence[int], u: int, slm_ids: np.ndarray, slm_probs: np.ndarray,
                   rand_accept: Sequence[float], rand_sample: float, top_k: int, top_p: float,
                   temperature: float) -> SampledResult:
    """One request.  logits [n, V] at the chunk's positions; chunk = u accepted tokens then drafts;
    slm_ids / slm_probs [n, K]: row t = the transmitted distribution the token at chunk index t
    was drawn from (rows of the accepted tokens are not read; id < 0 = unused entry);
    rand_accept [n]: the keep draw of the token at chunk index t."""
    n = len(chunk)
    margin, gap = float("inf"), float("inf")
    a = 0
    for j in range(n - u):
        t = u + j                                     # chunk index of the draft
        ids, q, g, pm = llm_distribution(logits[t - 1], top_k, top_p, temperature)
        gap, margin = min(gap, g), min(margin, pm)
        x = int(chunk[t])
        qx = float(q[ids == x].sum())
        sel = slm_ids[t] == x
        px = float(np.asarray(slm_probs[t], dtype=np.float64)[sel].sum())
        lhs = float(rand_accept[t]) * px
        margin = min(margin, abs(lhs - qx) / max(lhs, qx, 1e-300))
        if lhs < qx:
            a += 1
            continue
        # replacement from the positive part of q - p over the LLM's kept tokens
        p_on = np.zeros(len(ids))
        for i, tok in enumerate(ids):
            m = slm_ids[t] == tok
            if m.any():
                p_on[i] = float(np.asarray(slm_probs[t], dtype=np.float64)[m].sum())
        res = np.maximum(q - p_on, 0.0)
        if res.sum() <= 0.0:
            return SampledResult(a, int(ids[0]), margin, gap)
        tok, d = _inverse_cdf(ids, res, float(rand_sample))
        return SampledResult(a, tok, min(margin, d), gap)
    ids, q, g, pm = llm_distribution(logits[n - 1], top_k, top_p, temperature)
    tok, d = _inverse_cdf(ids, q, float(rand_sample))
    return SampledResult(a, tok, min(margin, d, pm), min(gap, g))
