"""Pins of the sampling-verification oracle (oracle/sampling.py): hand-worked cases, the greedy
special case, the identity case p = q, and the property that defines the method: the first token
a verification emits is distributed exactly as the LLM's distribution q, whatever the SLM's p."""
import os

import numpy as np
import pytest

from oracle import verify_greedy
from oracle.sampling import llm_distribution, verify_sampled

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "sampling_cases.txt")
LOGITS4 = np.log(np.array([4.0, 2.0, 1.0, 1.0]))


def _rows(kind):
    for raw in open(GOLDEN):
        line = raw.split("#")[0].strip()
        if line.startswith(kind + " "):
            yield line[len(kind) + 1:]


@pytest.mark.parametrize("row", list(_rows("dist")))
def test_llm_distribution_hand_worked(row):
    lhs, rhs = row.split("->")
    k, p, temp = lhs.split()
    ids_s, probs_s = rhs.split("|")
    ids, probs, _, _ = llm_distribution(LOGITS4, int(k), float(p), float(temp))
    assert ids.tolist() == [int(x) for x in ids_s.split()]
    assert np.allclose(probs, [float(x) for x in probs_s.split()], rtol=0, atol=1e-15)


@pytest.mark.parametrize("row", list(_rows("verify")))
def test_verify_sampled_hand_worked(row):
    lhs, rhs = row.split("->")
    drafts_s, keep_s, samp_s = lhs.split("|")
    drafts = [int(x) for x in drafts_s.split()]
    chunk = [3] + drafts
    n = len(chunk)
    slm_ids = np.tile(np.array([0, 1, 2]), (n, 1))
    slm_probs = np.tile(np.array([0.1, 0.8, 0.1]), (n, 1))
    ra = [0.0] + [float(x) for x in keep_s.split()]
    res = verify_sampled(np.tile(LOGITS4, (n, 1)), chunk, 1, slm_ids, slm_probs, ra, float(samp_s), 4, 1.0, 1.0)
    want = [int(x) for x in rhs.split()]
    assert [res.accept_len, res.correction] == want


def test_top1_on_both_sides_is_the_greedy_rule():
    rng = np.random.default_rng(0)
    V = 50
    for _ in range(200):
        n = int(rng.integers(1, 9))
        u = int(rng.integers(1, n + 1))
        logits = rng.normal(size=(n, V))
        top1 = logits.argmax(-1)
        chunk = [int(rng.integers(V)) for _ in range(n)]
        for t in range(u, n):          # drafts agree with the argmax about two times in three
            if rng.random() < 0.66:
                chunk[t] = int(top1[t - 1])
        slm_ids = np.array(chunk)[:, None]          # the device sends its top-1: the draft itself, probability 1
        slm_probs = np.ones((n, 1))
        res = verify_sampled(logits, chunk, u, slm_ids, slm_probs, rng.random(n), float(rng.random()), 1, 1.0, 1.0)
        assert (res.accept_len, res.correction) == verify_greedy(top1, chunk, u)


def test_identical_distributions_keep_every_draft():
    rng = np.random.default_rng(1)
    V, n = 12, 6
    logits = rng.normal(size=(n, V))
    chunk = [0] + [int(rng.integers(V)) for _ in range(n - 1)]
    slm_ids = np.tile(np.arange(V), (n, 1))
    slm_probs = np.zeros((n, V))
    for t in range(1, n):   # row t: what draft t was drawn from = the LLM's own distribution at t - 1
        ids, q, _, _ = llm_distribution(logits[t - 1], V, 1.0, 0.8)
        slm_probs[t, ids] = q
    for trial in range(50):
        res = verify_sampled(logits, chunk, 1, slm_ids, slm_probs, rng.random(n), float(rng.random()), V, 1.0, 0.8)
        assert res.accept_len == n - 1


@pytest.mark.parametrize("top_k,top_p,slm_k", [(6, 1.0, 6), (4, 0.9, 3)])
def test_first_emitted_token_follows_the_llm_distribution(top_k, top_p, slm_k):
    """Speculative sampling preserves the target distribution: with the draft drawn from p, the
    token that comes out at the first position (the draft if kept, else the replacement) has
    exactly the distribution q.  Monte Carlo with 60 000 trials; p is truncated to slm_k entries
    and renormalised, q to top_k / top_p."""
    rng = np.random.default_rng(5)
    V, N = 6, 60000
    logits = rng.normal(size=(2, V)) * 1.5
    ids_q, q, _, _ = llm_distribution(logits[0], top_k, top_p, 1.0)
    q_full = np.zeros(V)
    q_full[ids_q] = q
    p_raw = rng.dirichlet(np.ones(V))
    p_ids = np.argsort(-p_raw)[:slm_k]
    p = p_raw[p_ids] / p_raw[p_ids].sum()
    slm_ids = np.tile(p_ids, (2, 1))
    slm_probs = np.tile(p, (2, 1))
    counts = np.zeros(V)
    drafts = rng.choice(p_ids, size=N, p=p)
    keep, samp = rng.random(N), rng.random(N)
    for i in range(N):
        res = verify_sampled(logits, [0, int(drafts[i])], 1, slm_ids, slm_probs, [0.0, keep[i]], samp[i], top_k, top_p, 1.0)
        counts[int(drafts[i]) if res.accept_len == 1 else res.correction] += 1
    freq = counts / N
    sigma = np.sqrt(np.maximum(q_full * (1 - q_full), 1e-12) / N)
    assert (np.abs(freq - q_full) <= 4.5 * sigma + 1e-9).all(), (freq, q_full)
    assert (counts[q_full == 0] == 0).all()


def test_margins_report_the_nearest_decision():
    n = 2
    slm_ids = np.tile(np.array([0, 1, 2]), (n, 1))
    slm_probs = np.tile(np.array([0.1, 0.8, 0.1]), (n, 1))
    lg = np.tile(LOGITS4, (n, 1))
    # keep test .3125 * .8 = .25 = q exactly on the edge -> tiny margin; far from it -> large
    near = verify_sampled(lg, [3, 1], 1, slm_ids, slm_probs, [0, 0.3125 + 1e-9], 0.5, 4, 1.0, 1.0)
    far = verify_sampled(lg, [3, 1], 1, slm_ids, slm_probs, [0, 0.9], 0.2, 4, 1.0, 1.0)
    assert near.margin < 1e-6 and far.margin > 0.2
    # top-k boundary: k = 2 drops token 2 whose logit is ln 2 below token 1's
    assert abs(verify_sampled(lg, [3, 1], 1, slm_ids, slm_probs, [0, 0.9], 0.2, 2, 1.0, 1.0).topk_gap - np.log(2)) < 1e-12
