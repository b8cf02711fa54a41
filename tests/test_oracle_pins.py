"""Pins of the CPU oracle against things other than itself: a dense full-matrix numpy
forward, invariants of paging and chunking, hand-worked integer cases, closed forms,
and the capped-geometric acceptance expectation (paper Sec. 5)."""
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import Oracle, verify_greedy
from workloads import gen, rng
from workloads.configs import CONFIGS, TINY, ModelShape

from dense_ref import dense_forward, f64
from orc_util import PIN, PIN1, model, prefill, tokens_for

P = 4  # small page size so that short sequences span many pages


def _run(shape, glob, layers, toks, ctx, page_table, n_pages, u=1, f32=False, page_size=P, bf16_operands=False):
    orc = Oracle(shape, page_size=page_size, f32=f32, bf16_operands=bf16_operands)
    pools = orc.new_pool(n_pages)
    if ctx:
        prefill(orc, glob, layers, pools, page_table, toks[:ctx], step=5)
    res = orc.forward_chunk(glob, lambda l: layers[l], pools, page_table, ctx, list(toks[ctx:]), u=u)
    return res, pools


# ---------------------------------------------------------------- P-1 dense full-matrix attention
@pytest.mark.parametrize("shape,ctx,n", [(PIN, 13, 5), (PIN, 0, 7), (PIN1, 9, 1), (TINY, 21, 4)])
def test_chunk_logits_equal_dense_full_matrix_forward(shape, ctx, n):
    glob, layers = model(shape)
    toks = tokens_for(shape, ctx + n)
    n_pages = -(-(ctx + n) // P) + 3
    pt = np.random.default_rng(1).permutation(n_pages).astype(np.int32)
    res, pools = _run(shape, glob, layers, toks, ctx, pt, n_pages)
    ref, kvs = dense_forward(shape, glob, layers, toks)
    scale = np.abs(ref).max()
    assert np.abs(res.logits - ref[ctx:]).max() <= 1e-11 * scale
    assert (res.top1 == ref[ctx:].argmax(-1)).all()
    # the cache holds exactly the dense forward's post-RoPE K and V, at the paged slots
    for l, (k, v) in enumerate(kvs):
        for p in range(ctx + n):
            page, row = pt[p // P], p % P
            assert np.abs(pools[l][page, 0, :, row, :] - k[p]).max() <= 1e-11 * max(1.0, np.abs(k).max())
            assert np.abs(pools[l][page, 1, :, row, :] - v[p]).max() <= 1e-11 * max(1.0, np.abs(v).max())


# ---------------------------------------------------------------- the bf16-operand mode
def test_bf16_rounding_is_round_to_nearest_even():
    orc = Oracle(PIN)
    g = np.random.default_rng(3)
    vals = np.concatenate([g.standard_normal(4000) * 10.0 ** g.integers(-6, 6, 4000),
                           # exact ties between two bf16 neighbours, and values one float ulp off a tie
                           np.array([1.00390625, 1.01171875, -2.0078125, 3.0e-39, 0.0, -0.0, 65280.0 * 2.0 ** 100]),
                           np.nextafter(np.float32(1.00390625), np.float32(2.0)).astype(np.float64).reshape(1),
                           np.nextafter(np.float32(1.00390625), np.float32(0.0)).astype(np.float64).reshape(1)])
    vals = vals.astype(np.float32).astype(np.float64)
    ref = torch.from_numpy(vals).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(orc.bf16_round(vals), ref)
    assert orc.bf16_round([1.00390625])[0] == 1.0 and orc.bf16_round([1.01171875])[0] == 1.015625   # ties to even


@pytest.mark.parametrize("shape,ctx,n", [(PIN, 13, 5), (TINY, 21, 4)])
def test_bf16_operand_mode_equals_dense_forward_with_the_same_roundings(shape, ctx, n):
    """The bf16 model: activations entering a matrix product or the cache are bf16, sums are wide.
    The dense full-matrix forward rounds at the same places with torch's conversion."""
    glob, layers = model(shape)
    toks = tokens_for(shape, ctx + n)
    n_pages = -(-(ctx + n) // P) + 2
    pt = np.random.default_rng(2).permutation(n_pages).astype(np.int32)
    res, pools = _run(shape, glob, layers, toks, ctx, pt, n_pages, bf16_operands=True)
    ref, kvs = dense_forward(shape, glob, layers, toks, bf16_operands=True)
    sigma = ref.std()
    # a value that sits on a rounding boundary may round differently after a different summation order:
    # allow a handful of one-ulp flips, nothing systematic
    assert np.abs(res.logits - ref[ctx:]).max() <= 2e-3 * sigma
    assert np.sqrt(((res.logits - ref[ctx:]) ** 2).mean()) <= 1e-4 * sigma
    exact, _ = _run(shape, glob, layers, toks, ctx, pt, n_pages)
    d = np.sqrt(((res.logits - exact.logits) ** 2).mean()) / sigma
    assert 1e-4 < d < 2e-2          # the roundings are there, and are small
    # cached K and V are bf16 values
    k = pools[0][pt[0], 0, :, 0, :]
    assert np.array_equal(k, Oracle(shape).bf16_round(k).reshape(k.shape))


def test_bf16_operand_mode_keeps_the_chunking_and_paging_invariants():
    shape = PIN
    glob, layers = model(shape)
    toks = tokens_for(shape, 19)
    pt = np.arange(6, dtype=np.int32)
    a, _ = _run(shape, glob, layers, toks, 12, pt, 6, bf16_operands=True)
    orc = Oracle(shape, page_size=P, bf16_operands=True)
    pools = orc.new_pool(6)
    pt2 = np.array([4, 0, 5, 2, 1, 3], dtype=np.int32)
    prefill(orc, glob, layers, pools, pt2, toks[:12], step=3)
    rows = [orc.forward_chunk(glob, lambda l: layers[l], pools, pt2, 12 + j, [int(toks[12 + j])]).logits[0] for j in range(7)]
    assert np.array_equal(np.stack(rows), a.logits)


def test_runner_up_and_gap_match_sorted_logits():
    glob, layers = model(PIN)
    toks = tokens_for(PIN, 12)
    res, _ = _run(PIN, glob, layers, toks, 8, np.arange(6, dtype=np.int32), 6)
    srt = np.sort(res.logits, axis=-1)
    assert np.allclose(res.gap, srt[:, -1] - srt[:, -2], rtol=0, atol=0)
    assert (np.take_along_axis(res.logits, res.top2[:, None].astype(np.int64), -1)[:, 0] == srt[:, -2]).all()


# ---------------------------------------------------------------- P-2 paging invariance
def test_paged_equals_contiguous_and_any_page_permutation_bitwise():
    glob, layers = model(PIN)
    toks = tokens_for(PIN, 23)
    n_pages = 9
    ident = np.arange(n_pages, dtype=np.int32)
    base, _ = _run(PIN, glob, layers, toks, 17, ident, n_pages)
    for s in range(3):
        pt = np.random.default_rng(s).permutation(n_pages).astype(np.int32)
        r, _ = _run(PIN, glob, layers, toks, 17, pt, n_pages)
        assert np.array_equal(r.logits, base.logits)
    # one big page == contiguous cache
    r, _ = _run(PIN, glob, layers, toks, 17, np.zeros(1, dtype=np.int32), 1, page_size=32)
    assert np.array_equal(r.logits, base.logits)


# ---------------------------------------------------------------- P-3 chunking invariance
@pytest.mark.parametrize("total,ctx,splits", [
    (20, 11, ([1] * 9, [4, 5], [2, 3, 4], [8, 1])),
    (43, 11, ([16, 16], [5, 27], [31, 1], [1] * 32)),   # a 32-token chunk (chunked partial prefill, Sec. 4.5)
])
def test_chunk_equals_token_by_token_and_any_split(total, ctx, splits):
    glob, layers = model(PIN)
    toks = tokens_for(PIN, total)
    n_pages = -(-total // P) + 2
    pt = np.random.default_rng(5).permutation(n_pages).astype(np.int32)
    whole, _ = _run(PIN, glob, layers, toks, ctx, pt, n_pages)
    orc = Oracle(PIN, page_size=P)
    for split in splits:
        pools = orc.new_pool(n_pages)
        prefill(orc, glob, layers, pools, pt, toks[:ctx], step=3)
        p, rows = ctx, []
        for s in split:
            r = orc.forward_chunk(glob, lambda l: layers[l], pools, pt, p, list(toks[p:p + s]), u=s)
            rows.append(r.logits)
            p += s
        assert np.array_equal(np.concatenate(rows), whole.logits)


# ---------------------------------------------------------------- P-4 batch composition
def test_request_result_independent_of_batch_mates_and_order():
    glob, layers = model(PIN)
    wl = CONFIGS[1]
    orc = Oracle(PIN, page_size=P)
    lens = [(6, 3), (9, 2), (0, 4)]
    toks = [tokens_for(PIN, c + n, seed=i) for i, (c, n) in enumerate(lens)]
    n_pages = 12
    perm = np.random.default_rng(9).permutation(n_pages).astype(np.int32)
    tables = [perm[0:4], perm[4:8], perm[8:12]]
    alone = []
    for i, (c, n) in enumerate(lens):
        r, _ = _run(PIN, glob, layers, toks[i], c, tables[i], n_pages)
        alone.append(r.logits)
    for order in ([0, 1, 2], [2, 0, 1]):
        pools = orc.new_pool(n_pages)            # one shared pool, interleaved pages
        for i in order:
            prefill(orc, glob, layers, pools, tables[i], toks[i][:lens[i][0]], step=4)
        for i in order:
            c, n = lens[i]
            r = orc.forward_chunk(glob, lambda l: layers[l], pools, tables[i], c, list(toks[i][c:]))
            assert np.array_equal(r.logits, alone[i])


# ---------------------------------------------------------------- P-5 hand-worked accept cases
def _golden(name):
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", name)
    rows = []
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            rows.append([c.strip() for c in line.split(";")])
    return rows


@pytest.mark.parametrize("row", _golden("verify_cases.txt"))
def test_greedy_verify_hand_worked(row):
    top1, chunk = [int(x) for x in row[0].split()], [int(x) for x in row[1].split()]
    assert verify_greedy(top1, chunk, int(row[2])) == (int(row[3]), int(row[4]))


def test_argmax_tie_takes_lowest_id():
    shape = PIN1
    glob, layers = model(shape)
    lm = glob["lm_head"].clone()
    lm[30] = lm[11]                      # two identical vocabulary rows -> exactly equal logits
    lm[11] *= 64
    lm[30] *= 64                         # and by far the largest ones for some direction
    glob = dict(glob, lm_head=lm)
    orc = Oracle(shape, page_size=P)
    x = f64(lm[11:12]) * 3.0
    _, t1, t2, gap = orc.logits(glob, x.astype(np.float64))
    assert t1[0] == 11 and t2[0] == 30 and gap[0] == 0.0


# ---------------------------------------------------------------- P-6 losslessness (Sec. 4.2: lossless verification)
def test_draft_verify_loop_reproduces_greedy_continuation():
    shape = PIN
    glob, layers = model(shape, seed=3)
    orc = Oracle(shape, page_size=P)
    prompt = list(tokens_for(shape, 7, seed=4))
    n_new, n_pages = 14, 12
    pt = np.random.default_rng(2).permutation(n_pages).astype(np.int32)
    lw = lambda l: layers[l]
    # plain greedy decoding
    pools = orc.new_pool(n_pages)
    r = prefill(orc, glob, layers, pools, pt, prompt, step=16)
    greedy, nxt = [], int(r.top1[-1])
    for i in range(n_new):
        greedy.append(nxt)
        r = orc.forward_chunk(glob, lw, pools, pt, len(prompt) + i, [nxt])
        nxt = int(r.top1[0])
    # draft & verify with arbitrary (mostly wrong, sometimes right) drafts
    g = np.random.default_rng(11)
    pools = orc.new_pool(n_pages)
    r = prefill(orc, glob, layers, pools, pt, prompt, step=16)
    out, anchor, ctx = [int(r.top1[-1])], int(r.top1[-1]), len(prompt)
    while len(out) < n_new:
        gamma = int(g.integers(0, 5))
        drafts = [greedy[len(out) + j] if (len(out) + j < n_new and g.random() < 0.6) else int(g.integers(0, shape.vocab))
                  for j in range(gamma)]
        res = orc.forward_chunk(glob, lw, pools, pt, ctx, [anchor] + drafts)
        out += drafts[:res.accept_len] + [res.correction]
        ctx += 1 + res.accept_len        # rejected drafts' slots are simply overwritten later
        anchor = res.correction
    assert out[:n_new] == greedy


# ---------------------------------------------------------------- P-7 closed forms
def test_zero_output_projections_reduce_logits_to_normed_embedding():
    shape = PIN
    glob, layers = model(shape)
    layers = [dict(w, wo=torch.zeros_like(w["wo"]), wd=torch.zeros_like(w["wd"])) for w in layers]
    toks = tokens_for(shape, 6)
    res, _ = _run(shape, glob, layers, toks, 2, np.arange(2, dtype=np.int32), 2)
    e = f64(glob["embed"])[toks[2:]]
    ref = e / np.sqrt((e * e).mean(-1, keepdims=True) + shape.rms_eps) * f64(glob["final_norm"]) @ f64(glob["lm_head"]).T
    assert np.abs(res.logits - ref).max() <= 1e-12 * np.abs(ref).max()


def _rand_pool(orc, n_pages, seed):
    g = np.random.default_rng(seed)
    return g.standard_normal(orc.new_pool(n_pages)[0].shape)


def test_attention_zero_query_is_mean_of_visible_values():
    orc = Oracle(PIN, page_size=P)
    pool = _rand_pool(orc, 5, 0)
    pt = np.array([3, 0, 4, 1, 2], dtype=np.int32)
    ctx, n = 10, 3
    out = orc.attention(np.zeros((n, PIN.q_dim)), pool, pt, ctx)
    G = PIN.group
    for j in range(n):
        vis = np.stack([pool[pt[t // P], 1, :, t % P, :] for t in range(ctx + j + 1)])   # [len, Hkv, hd]
        for h in range(PIN.n_q_heads):
            assert np.allclose(out[j].reshape(PIN.n_q_heads, -1)[h], vis[:, h // G].mean(0), rtol=1e-12, atol=1e-13)


def test_attention_equal_value_rows_return_that_row():
    orc = Oracle(PIN, page_size=P)
    pool = _rand_pool(orc, 4, 1)
    row = np.random.default_rng(2).standard_normal((PIN.n_kv_heads, PIN.head_dim))
    pool[:, 1] = row[None, :, None, :]
    q = np.random.default_rng(3).standard_normal((2, PIN.q_dim))
    out = orc.attention(q, pool, np.arange(4, dtype=np.int32), 9).reshape(2, PIN.n_q_heads, PIN.head_dim)
    for h in range(PIN.n_q_heads):
        assert np.allclose(out[:, h], row[h // PIN.group], rtol=1e-12)


def test_attention_brute_force_single_head_and_causal_edge():
    """softmax(q K^T / sqrt(d_k)) V over exactly positions 0..ctx+j (paper Sec. 3.2)."""
    orc = Oracle(PIN1, page_size=P)
    pool = _rand_pool(orc, 3, 4)
    pt = np.array([2, 0, 1], dtype=np.int32)
    q = np.random.default_rng(5).standard_normal((3, PIN1.q_dim))
    ctx = 6
    out = orc.attention(q, pool, pt, ctx).reshape(3, PIN1.n_q_heads, PIN1.head_dim)
    for j in range(3):
        K = np.stack([pool[pt[t // P], 0, 0, t % P] for t in range(ctx + j + 1)])
        V = np.stack([pool[pt[t // P], 1, 0, t % P] for t in range(ctx + j + 1)])
        for h in range(PIN1.n_q_heads):
            s = K @ q[j].reshape(PIN1.n_q_heads, -1)[h] / math.sqrt(PIN1.head_dim)
            w = np.exp(s - s.max())
            w /= w.sum()
            assert np.allclose(out[j, h], w @ V, rtol=1e-12)
    # changing a key/value beyond the causal horizon of row 0 must not change row 0
    pool2 = pool.copy()
    pool2[pt[(ctx + 1) // P], :, :, (ctx + 1) % P] += 7.0
    out2 = orc.attention(q, pool2, pt, ctx).reshape(3, PIN1.n_q_heads, PIN1.head_dim)
    assert np.array_equal(out2[0], out[0]) and not np.array_equal(out2[1], out[1])


def test_rope_identity_at_zero_norm_preserving_and_relative():
    orc = Oracle(PIN, page_size=P)
    g = np.random.default_rng(0)
    hd = PIN.head_dim
    a, b = g.standard_normal(hd), g.standard_normal(hd)
    assert np.array_equal(orc.rope(a, 1, 0), a)
    assert np.isclose(np.linalg.norm(orc.rope(a, 1, 777)), np.linalg.norm(a), rtol=1e-12)
    d0 = orc.rope(a, 1, 5) @ orc.rope(b, 1, 2)
    for s in (1, 40, 8000):
        assert np.isclose(orc.rope(a, 1, 5 + s) @ orc.rope(b, 1, 2 + s), d0, rtol=1e-9, atol=1e-9)
    # explicit 2-D rotation of the pair (i, i + hd/2) by pos * base^(-2i/hd)
    pos, i = 3, 2
    ang = pos * PIN.rope_base ** (-2.0 * i / hd)
    r = orc.rope(a, 1, pos)
    assert np.isclose(r[i], a[i] * math.cos(ang) - a[i + hd // 2] * math.sin(ang), rtol=1e-12)
    assert np.isclose(r[i + hd // 2], a[i + hd // 2] * math.cos(ang) + a[i] * math.sin(ang), rtol=1e-12)


def test_rmsnorm_and_linear_against_numpy():
    orc = Oracle(PIN, page_size=P)
    g = np.random.default_rng(1)
    x = g.standard_normal((3, PIN.d_model))
    w = gen.gen_weight(PIN, 0, "wg", 0)
    gain = gen.gen_gain(PIN, 0, "norm1", 0)
    assert np.allclose(orc.linear(x, w), x @ f64(w).T, rtol=1e-12, atol=1e-14)
    ref = x / np.sqrt((x * x).mean(-1, keepdims=True) + PIN.rms_eps) * f64(gain)
    assert np.allclose(orc.rmsnorm(x, gain), ref, rtol=1e-13)
    # a transposed weight must be caught: non-square matrix, distinct rows
    assert orc.linear(x, w).shape == (3, PIN.d_ffn)


# ---------------------------------------------------------------- P-8 slot map, hand-written
def test_slot_map_hand_written_page_tables():
    orc = Oracle(PIN, page_size=16)
    pt = [7, 2, 9, 4, 0]
    # ctx 48, chunk 4: starts exactly on a page boundary -> logical page 3 -> physical 4
    assert [orc.slot(pt, 48 + j) for j in range(4)] == [(4, 0), (4, 1), (4, 2), (4, 3)]
    # ctx 60, chunk 8: crosses from logical page 3 (rows 12..15) into logical page 4 (rows 0..3)
    assert [orc.slot(pt, 60 + j) for j in range(8)] == [(4, 12), (4, 13), (4, 14), (4, 15),
                                                        (0, 0), (0, 1), (0, 2), (0, 3)]
    # ctx 0
    assert [orc.slot(pt, j) for j in range(3)] == [(7, 0), (7, 1), (7, 2)]


# ---------------------------------------------------------------- P-9 acceptance statistics (Sec. 5)
def test_mean_accept_len_follows_capped_geometric():
    """With i.i.d. match probability p' per draft, E[accepted + 1] = (1 - p'^(gamma+1)) / (1 - p')."""
    wl = CONFIGS[1]
    V, gamma, p = wl.shape.vocab, 3, wl.p_match
    n_req = 6000
    total = 0
    for r in range(n_req):
        top1 = [(r * 31 + 7 * j) % V for j in range(gamma + 1)]
        chunk = [0] + [gen.gen_draft(wl, r, j, top1[j]) for j in range(gamma)]
        total += verify_greedy(top1, chunk, 1)[0]
    pp = p + (1 - p) / V
    expect = (1 - pp ** (gamma + 1)) / (1 - pp) - 1          # = sum_{k=1..gamma} p'^k  (1.5337 here)
    se = 1.2 / math.sqrt(n_req)
    assert abs(total / n_req - expect) < 4 * se


@pytest.mark.parametrize("row", _golden("expected_generated_tokens.txt"))
def test_generated_tokens_per_verification_match_the_papers_expectation(row):
    """Drafts that match the argmax independently with probability alpha: accepted drafts + the
    correction/bonus token per verification have the stored closed-form expectation (Sec. 5).
    Exact: every one of the 2^gamma hit patterns goes through the verification routine and is
    weighted with its probability, so a wrong fourth decimal in the stored value fails."""
    alpha, gamma, expect = float(row[0]), int(row[1]), float(row[2])
    top1 = [11 + 3 * j for j in range(gamma + 1)]
    total = 0.0
    for pattern in itertools.product((False, True), repeat=gamma):
        prob = 1.0
        for hit in pattern:
            prob *= alpha if hit else 1.0 - alpha
        chunk = [0] + [top1[j] if pattern[j] else top1[j] + 1000 for j in range(gamma)]
        total += prob * (verify_greedy(top1, chunk, 1)[0] + 1)
    assert abs(total - expect) < 1e-12


# ---------------------------------------------------------------- SwiGLU: hand values, not the formula again
def test_swiglu_product_against_hand_values_of_silu():
    """One layer whose attention contributes nothing (zero q/k/v/o projections), unit gains and
    eps = 0, fed rows of mean square 1, so the normalised hidden state h equals the row itself.
    With W_g = I, W_d = I and every row of W_u picking h[1], the layer adds silu(h_i) * h[1] to
    x_i.  The expected numbers are tabulated values of the logistic function, typed in, not the
    expression under test evaluated again: silu(0) = 0, silu(1) = 0.7310585786,
    silu(-1) = -0.2689414214, silu(2) = 1.7615941560."""
    shape = ModelShape("swiglu-pin", 1, 4, 1, 1, 4, 4, 8, rms_eps=0.0)
    orc = Oracle(shape, page_size=16)

    def bf(a):
        return torch.tensor(a, dtype=torch.float32).to(torch.bfloat16)

    eye = [[1.0 if i == j else 0.0 for j in range(4)] for i in range(4)]
    zero = [[0.0] * 4 for _ in range(4)]
    w = {"wq": bf(zero), "wk": bf(zero), "wv": bf(zero), "wo": bf(zero), "wg": bf(eye),
         "wu": bf([[0.0, 1.0, 0.0, 0.0]] * 4), "wd": bf(eye), "norm1": bf([1.0] * 4), "norm2": bf([1.0] * 4)}
    pt = np.array([0], dtype=np.int32)
    pool = orc.new_pool(1)
    # h = (0, 1, -1, sqrt 2): up = h[1] = 1;  h = (1, -1, 1, 1): up = -1 (the product's second factor and its sign)
    x = np.array([[0.0, 1.0, -1.0, math.sqrt(2.0)], [1.0, -1.0, 1.0, 1.0]], dtype=np.float64)
    before = x.copy()
    orc.layer(w, x, pool[0], pt, 0)
    upd = x - before
    assert np.allclose(upd[0][:3], [0.0, 0.7310585786, -0.2689414214], atol=1e-9)
    assert np.allclose(upd[1], [-0.7310585786, 0.2689414214, -0.7310585786, -0.7310585786], atol=1e-9)
    # gate and up from different inputs and with weights other than 0 / 1: g = 2 h[0], u = -2 h[1]
    w2 = dict(w)
    w2["wg"] = bf([[2.0, 0, 0, 0]] + [[0.0] * 4] * 3)
    w2["wu"] = bf([[0, -2.0, 0, 0]] + [[0.0] * 4] * 3)
    x2 = np.ones((1, 4), dtype=np.float64)
    orc.layer(w2, x2, pool[0], pt, 0)
    assert abs((x2[0][0] - 1.0) - 1.7615941560 * -2.0) < 1e-8
    assert np.allclose(x2[0][1:], 1.0, atol=1e-12)


# ---------------------------------------------------------------- the single-precision build agrees
def test_f32_build_agrees_with_f64_far_inside_parity_tolerance():
    shape = TINY
    glob, layers = model(shape)
    toks = tokens_for(shape, 40)
    pt = np.random.default_rng(0).permutation(4).astype(np.int32)
    a, _ = _run(shape, glob, layers, toks, 36, pt, 4, page_size=16)
    b, _ = _run(shape, glob, layers, toks, 36, pt, 4, page_size=16, f32=True)
    sigma = a.logits.std()
    assert np.abs(a.logits - b.logits).max() < 1e-4 * sigma


# ---------------------------------------------------------------- generator sanity (shared input module)
def test_counter_rng_matches_big_int_reference_and_is_sliceable():
    k = rng.stream_key(5, 3, 2)
    for i in (0, 1, 7, 123456789):
        z = (k + i * rng._GOLDEN) & rng._MASK64
        assert (int(rng.bits64(k, i, 1)[0]) & rng._MASK64) == rng._mix_py(z)
    a = rng.normal_f32(k, 0, 1000, 0.02)
    b = rng.normal_f32(k, 400, 100, 0.02)
    assert torch.equal(a[400:500], b)
    big = rng.normal_f32(k, 0, 400000, 1.0)
    assert abs(float(big.mean())) < 0.01 and abs(float(big.std()) - 1.0) < 0.01
