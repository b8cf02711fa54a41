"""The host planner (syn_plan_host: validation, positions, KV slots, attention work list) on the CPU.
No device is involved; the same code runs inside syn_plan_create / syn_verify_batch."""
import numpy as np
import pytest
import torch

import paper_2511_07423_b200 as syn
from workloads import gen
from workloads.configs import CONFIGS, MINI_8B, TINY, ModelShape, Workload


def _plan(shape, batch, toks=None, **kw):
    toks = torch.zeros(batch.n_tokens, dtype=torch.int32) if toks is None else toks
    args = dict(chunk_tokens=toks, chunk_offsets=batch.chunk_offsets, page_tables=batch.page_tables,
                ctx_lens=batch.ctx_lens)
    args.update(kw)
    return syn.plan_host(shape, batch.n_pages, **args)


def test_positions_and_slots_follow_the_page_table():
    """Hand-written table (paper Sec. 3.4: the chunk is appended after the cached prefix)."""
    shape = TINY
    pt = torch.tensor([[7, 2, 9, 4, 0], [1, 3, 5, 6, 8]], dtype=torch.int32)
    # request 0: ctx 60, chunk 8 -> positions 60..67: page 4 rows 12..15, then page 0 rows 0..3
    # request 1: ctx 0, chunk 3 -> page 1 rows 0..2
    r = syn.plan_host(shape, 10, torch.zeros(11, dtype=torch.int32), [0, 8, 11], pt, [60, 0])
    assert r["pos"].tolist() == list(range(60, 68)) + [0, 1, 2]
    assert r["slot"].tolist() == [4 * 16 + 12, 4 * 16 + 13, 4 * 16 + 14, 4 * 16 + 15, 0, 1, 2, 3, 16, 17, 18]


@pytest.mark.parametrize("attention", [0, 1, 2], ids=["auto", "warp_mma", "tcgen05"])
@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 6])
def test_work_list_covers_every_key_of_every_row_group_exactly_once(cfg, attention):
    wl = CONFIGS[cfg]
    shape = wl.shape
    batch = gen.gen_batch(wl)
    syn.debug_set_attention(attention)
    try:
        r = _plan(shape, batch)
    finally:
        syn.debug_set_attention(0)
    rows = r["stats"].attn_rows
    # the planner's own choice: 128-row tiles where a chunk would otherwise be several items per kv head
    assert rows == {0: 128 if cfg == 6 else 64, 1: 64, 2: 128}[attention]
    items = r["items"].numpy()
    cb = r["cta_begin"].numpy()
    G, Hkv = shape.group, shape.n_kv_heads
    assert cb[0] == 0 and cb[-1] == len(items) and (np.diff(cb) >= 1).all() and r["n_cta"] <= 148
    offs = batch.chunk_offsets.numpy()
    cover = {}
    for q_tok, nj, kvh, req, kb, ke, qp0, part, grp in items:
        assert offs[req] <= q_tok and q_tok + nj <= offs[req + 1] and 1 <= nj and nj * G <= rows
        assert 0 <= kvh < Hkv and kb % 64 == 0 and kb < ke
        assert qp0 == batch.ctx_lens[req] + (q_tok - offs[req])
        assert ke <= qp0 + nj                       # never past the last key the group's last row may see
        assert (part >= 0) == (grp >= 0)
        cover.setdefault((q_tok, nj, kvh), []).append((kb, ke, part))
    # every (token group, kv head) appears, its key ranges tile [0, ctx + j0 + nj) without gap or overlap
    n_groups = 0
    for i in range(batch.n_req):
        n = offs[i + 1] - offs[i]
        tpg = min(16, 64 // G) if rows == 64 else min(32, 128 // G)
        for j0 in range(0, n, tpg):
            nj = min(tpg, n - j0)
            for h in range(Hkv):
                rng_ = sorted(cover.pop((offs[i] + j0, nj, h)))
                assert rng_[0][0] == 0 and rng_[-1][1] == batch.ctx_lens[i] + j0 + nj
                for a, b in zip(rng_, rng_[1:]):
                    assert a[1] == b[0]
                assert (len(rng_) == 1) == (rng_[0][2] < 0)
                n_groups += 1
    assert not cover
    st = r["stats"]
    assert st.n_tokens == batch.n_tokens and st.attn_items == len(items)
    assert st.kv_read_bytes == int((batch.ctx_lens + batch.chunk_lens).sum()) * shape.kv_bytes_per_token()
    assert st.weight_bytes == 2 * shape.dense_params()


def test_oversized_units_are_split_and_small_batches_fill_the_machine():
    shape = MINI_8B
    wl = Workload("t", shape, 1, 2, ("list", (5000, 100)), ("list", (16, 1)), 0.5)
    batch = gen.gen_batch(wl)
    r = _plan(shape, batch)
    assert r["stats"].attn_split_items > 0
    parts = r["items"][:, 7]
    assert sorted(parts[parts >= 0].tolist()) == list(range(r["stats"].attn_split_items))


def test_validation_codes_match_the_header():
    shape = TINY
    wl = CONFIGS[1]
    batch = gen.gen_batch(wl)
    toks = torch.zeros(batch.n_tokens, dtype=torch.int32)

    def code(**kw):
        with pytest.raises(syn.SynError) as e:
            _plan(shape, batch, **kw)
        return e.value.code

    assert code(chunk_offsets=torch.tensor([0, 4, 8, 12, 45])) == -2
    assert code(chunk_offsets=torch.tensor([0, 4, 4, 12, 16])) == -2
    assert code(chunk_offsets=torch.tensor([1, 4, 8, 12, 16])) == -1
    assert code(n_uncached=[1, 5, 1, 1]) == -3
    assert code(n_uncached=[0, 1, 1, 1]) == -3
    bad = batch.page_tables.clone(); bad[0, 0] = batch.n_pages
    assert code(page_tables=bad) == -4
    bad = batch.page_tables.clone(); bad[1, 0] = -1
    assert code(page_tables=bad) == -4
    assert code(ctx_lens=torch.tensor([48, 64, 96, 16 * batch.max_pages - 3])) == -5
    assert code(ctx_lens=torch.tensor([48, -1, 96, 128])) == -1
    t2 = toks.clone(); t2[3] = shape.vocab
    assert code(chunk_tokens=t2) == -6
    alias = batch.page_tables.clone(); alias[1] = alias[0]
    assert code(page_tables=alias, ctx_lens=torch.tensor([48, 48, 96, 128])) == -7
    assert _plan(shape, batch, n_uncached=[4, 1, 2, 3])["stats"].n_req == 4
