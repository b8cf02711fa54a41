"""Ragged paged attention kernel (C ABI: syn_op_attention) against the CPU oracle's attention,
element by element, on random queries over a seeded synthetic cache."""
import numpy as np
import pytest
import torch

from oracle import Oracle
from workloads import gen, rng
from workloads.configs import ModelShape, Workload

from harness import cpu_model, fill_synthetic_kv, to_cuda

pytestmark = pytest.mark.gpu


def _batch(ctx, chunk, P=16, seed=0):
    wl = Workload("t", None, seed, len(ctx), ("list", tuple(ctx)), ("list", tuple(chunk)), 0.5)
    return gen.gen_batch(wl)


CASES = [
    # head_dim, Hq, Hkv, ctx lens, chunk lens
    (64, 4, 2, [48, 64, 96, 128], [4, 4, 4, 4]),                     # config-1 geometry
    (128, 8, 2, [0, 5, 16, 100, 333], [1, 16, 7, 3, 12]),            # G=4: 1..4 row tiles, ctx 0, page-boundary starts
    (128, 10, 2, [20, 700], [16, 13]),                               # G=5: token groups of 12
    (64, 8, 8, [130, 31], [16, 2]),                                  # G=1
    (128, 8, 2, [1500, 900, 2300], [16, 1, 9]),                      # long contexts: key ranges split over items
    (64, 16, 2, [40], [8]),                                          # G=8
    (128, 8, 2, [100, 5, 0], [32, 19, 17]),                          # chunks beyond 16: two token groups per request
    (128, 10, 2, [50], [30]),                                        # G=5, three token groups
    (64, 16, 2, [200], [32]),                                        # G=8, four token groups
    (128, 8, 2, [3000, 40], [32, 32]),                               # 128-row tiles whose key ranges are split over items
    (128, 10, 2, [2500], [25]),                                      # G=5: 125 rows in one tile of the tcgen05 kernel, split keys
]


@pytest.mark.parametrize("kind", [1, 2], ids=["warp_mma", "tcgen05"])
@pytest.mark.parametrize("hd,Hq,Hkv,ctx,chunk", CASES)
def test_attention_matches_oracle(hd, Hq, Hkv, ctx, chunk, kind):
    import paper_2511_07423_b200 as syn
    syn.debug_set_attention(kind)
    try:
        _run(hd, Hq, Hkv, ctx, chunk)
    finally:
        syn.debug_set_attention(0)


def _run(hd, Hq, Hkv, ctx, chunk):
    import paper_2511_07423_b200 as syn
    shape = ModelShape("att", 2, 256, Hq, Hkv, hd, 256, 512)
    seed = 7
    batch = _batch(ctx, chunk, seed=seed)
    glob, layers = cpu_model(shape, seed)
    gg, gl = to_cuda(glob, layers)
    model = syn.Model(shape, gg, gl)
    kv = syn.KVCache(model, batch.n_pages)
    orc = Oracle(shape)
    pools = orc.new_pool(batch.n_pages)
    layer = 1
    T = batch.n_tokens
    q = rng.normal_f32(rng.stream_key(seed, 77), 0, T * shape.q_dim, 1.5).view(T, shape.q_dim).to(torch.float16)
    # cached prefix + the chunk's own keys/values: all positions < ctx + n come from the seeded stream
    for r in range(batch.n_req):
        tot = int(batch.ctx_lens[r] + batch.chunk_lens[r])
        pt = batch.page_tables[r]
        k, v = gen.gen_kv(shape, seed, layer, r, 0, tot)
        kv.import_kv(layer, pt, 0, k.cuda(), v.cuda())
        orc.load_kv(pools[layer], pt.numpy(), 0, k.float().numpy(), v.float().numpy())
        # stale rows after the chunk (rejected drafts of an earlier step) must be ignored
        if tot % 16:
            junk = torch.full((16 - tot % 16, Hkv, hd), 300.0, dtype=torch.bfloat16)
            kv.import_kv(layer, pt, tot, junk.cuda(), junk.cuda())
    toks = torch.zeros(T, dtype=torch.int32)
    plan = syn.Plan(kv, toks, batch.chunk_offsets, batch.page_tables, batch.ctx_lens)
    out = plan.attention(layer, q.cuda())
    torch.cuda.synchronize()
    assert model.status() == 0
    got = out.float().cpu().numpy()
    for r in range(batch.n_req):
        b, n = int(batch.chunk_offsets[r]), int(batch.chunk_lens[r])
        ref = orc.attention(q[b:b + n].double().numpy(), pools[layer], batch.page_tables[r].numpy(), int(batch.ctx_lens[r]))
        scale = np.abs(ref).max()
        err = np.abs(got[b:b + n] - ref).max()
        assert err <= 2e-3 * scale, (r, err, scale)   # half-precision softmax weights and output (11 significant bits)
    st = plan.stats()
    if max(ctx) > 1000:
        assert st.attn_split_items > 0


@pytest.mark.parametrize("kind", [1, 2], ids=["warp_mma", "tcgen05"])
@pytest.mark.parametrize("hd,Hq,Hkv", [(128, 8, 2), (64, 8, 2)])
def test_scores_that_keep_growing_along_the_keys(hd, Hq, Hkv, kind):
    """Keys whose scores rise steadily with the position (about 13 in log2 units per 64 keys, in one half of the
    query heads; falling in the other half): the running maximum moves in every stage, so the tcgen05 kernel
    rescales its accumulator in tensor memory every time instead of about once in a thousand stages, and the last
    keys carry almost all the weight."""
    import paper_2511_07423_b200 as syn
    syn.debug_set_attention(kind)
    try:
        shape = ModelShape("att-grow", 1, 256, Hq, Hkv, hd, 256, 512)
        seed = 9
        ctx, chunk = [700, 130, 1400], [16, 5, 32]
        batch = _batch(ctx, chunk, seed=seed)
        glob, layers = cpu_model(shape, seed)
        gg, gl = to_cuda(glob, layers)
        model = syn.Model(shape, gg, gl)
        kv = syn.KVCache(model, batch.n_pages)
        orc = Oracle(shape)
        pools = orc.new_pool(batch.n_pages)
        T = batch.n_tokens
        # q: a large component along dimension 0 (sign by head), small noise elsewhere; k: component 0 grows with the position
        q = 0.05 * rng.normal_f32(rng.stream_key(seed, 77), 0, T * shape.q_dim, 1.0).view(T, Hq, hd)
        q[:, :, 0] = torch.tensor([31.0 if h % 2 == 0 else -31.0 for h in range(Hq)])
        q = q.reshape(T, shape.q_dim).to(torch.float16)
        slope = 0.2 * (hd ** 0.5) / (31.0 * 1.4426950408889634)      # 0.2 log2 units per key
        for r in range(batch.n_req):
            tot = int(batch.ctx_lens[r] + batch.chunk_lens[r])
            pt = batch.page_tables[r]
            k, v = gen.gen_kv(shape, seed, 0, r, 0, tot)
            k = (0.05 * k.float())
            k[:, :, 0] = (slope * torch.arange(1, tot + 1, dtype=torch.float32))[:, None]
            k = k.to(torch.bfloat16)
            kv.import_kv(0, pt, 0, k.cuda(), v.cuda())
            orc.load_kv(pools[0], pt.numpy(), 0, k.float().numpy(), v.float().numpy())
        plan = syn.Plan(kv, torch.zeros(T, dtype=torch.int32), batch.chunk_offsets, batch.page_tables, batch.ctx_lens)
        out = plan.attention(0, q.cuda())
        torch.cuda.synchronize()
        assert model.status() == 0
        got = out.float().cpu().numpy()
        assert np.isfinite(got).all()
        for r in range(batch.n_req):
            b, n = int(batch.chunk_offsets[r]), int(batch.chunk_lens[r])
            ref = orc.attention(q[b:b + n].double().numpy(), pools[0], batch.page_tables[r].numpy(), int(batch.ctx_lens[r]))
            scale = np.abs(ref).max()
            err = np.abs(got[b:b + n] - ref).max()
            assert err <= 2e-3 * scale, (r, err, scale)
    finally:
        syn.debug_set_attention(0)
