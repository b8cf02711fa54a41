"""End-to-end parity of syn_verify_batch with the CPU oracle on seeded batches, the KV slots
it writes, and its host-side error behaviour."""
import numpy as np
import pytest
import torch

from oracle import Oracle
from workloads import gen
from workloads.configs import CONFIGS, MINI_1B, MINI_8B, TINY, ModelShape, Workload

from harness import (cpu_model, fill_synthetic_kv, judge, oracle_teacher_forced, to_cuda)

pytestmark = pytest.mark.gpu


def _setup(shape, seed, batch):
    import paper_2511_07423_b200 as syn
    glob, layers = cpu_model(shape, seed)
    gg, gl = to_cuda(glob, layers)
    model = syn.Model(shape, gg, gl)
    kv = syn.KVCache(model, batch.n_pages)
    orc = Oracle(shape)
    pools = orc.new_pool(batch.n_pages)
    return glob, layers, model, kv, orc, pools


def _run_and_judge(wl, shape, batch, glob, layers, kv, orc, pools, check_kv=True, uncached=None):
    reqs = []
    for r in range(batch.n_req):
        reqs.append(oracle_teacher_forced(orc, glob, lambda l: layers[l], pools, batch.page_tables[r].numpy(),
                                          int(batch.ctx_lens[r]), wl, r, int(batch.chunk_lens[r]),
                                          u=1 if uncached is None else uncached[r]))
    tokens = torch.tensor([t for o in reqs for t in o.chunk], dtype=torch.int32)
    acc, cor, logits = kv.verify_batch(tokens, batch.chunk_offsets, batch.page_tables, batch.ctx_lens,
                                       n_uncached=uncached, want_logits=True)
    assert kv.model.status() == 0
    res = judge(reqs, acc, cor, logits, batch.chunk_offsets)
    if check_kv:   # the chunk's K/V landed in exactly the slots the page table names
        for r in range(batch.n_req):
            ctx, n = int(batch.ctx_lens[r]), int(batch.chunk_lens[r])
            pt = batch.page_tables[r]
            for l in range(shape.n_layers):
                k, v = kv.export_kv(l, pt, ctx, n)
                for j in range(n):
                    page, row = int(pt[(ctx + j) // 16]), (ctx + j) % 16
                    for which, t in ((0, k), (1, v)):
                        ref = pools[l][page, which, :, row, :]
                        err = np.abs(t[j].float().cpu().numpy() - ref).max()
                        assert err <= 0.02 * max(1.0, np.abs(ref).max()), (r, l, j, which, err)
    return res


def test_config1_tiny_real_prefill():
    """Configuration 1: 2-layer decoder, real prefill of uniform-random context tokens on both sides
    (the CUDA side prefills through its own u = n calls), 4-token chunks = 1 anchor + 3 drafts."""
    wl = CONFIGS[1]
    shape = wl.shape
    batch = gen.gen_batch(wl)
    glob, layers, model, kv, orc, pools = _setup(shape, wl.seed, batch)
    ctx_tokens = [gen.gen_context_tokens(wl, r, int(batch.ctx_lens[r])) for r in range(batch.n_req)]
    # oracle prefill, request by request
    for r in range(batch.n_req):
        p = 0
        while p < len(ctx_tokens[r]):
            c = ctx_tokens[r][p:p + 16].tolist()
            orc.forward_chunk(glob, lambda l: layers[l], pools, batch.page_tables[r].numpy(), p, c, u=len(c),
                              want_logits=False)
            p += len(c)
    # CUDA prefill: rounds of <= 16 tokens per request, batched over the requests that still have tokens
    done = [0] * batch.n_req
    while True:
        live = [r for r in range(batch.n_req) if done[r] < len(ctx_tokens[r])]
        if not live:
            break
        toks, offs, ctxs = [], [0], []
        for r in live:
            c = ctx_tokens[r][done[r]:done[r] + 16].tolist()
            toks += c
            offs.append(offs[-1] + len(c))
            ctxs.append(done[r])
        unc = [offs[i + 1] - offs[i] for i in range(len(live))]
        kv.verify_batch(toks, offs, batch.page_tables[live], ctxs, n_uncached=unc)
        for i, r in enumerate(live):
            done[r] += unc[i]
    res = _run_and_judge(wl, shape, batch, glob, layers, kv, orc, pools)
    print("config 1:", res)


@pytest.mark.parametrize("shape,ctx,chunk", [
    (MINI_1B, [0, 33, 48, 200, 515, 1030], [1, 8, 16, 5, 3, 11]),     # head_dim 64, G = 4
    (MINI_8B, [17, 64, 300, 1200], [16, 2, 9, 13]),                    # head_dim 128, G = 4
    (ModelShape("g5", 2, 640, 10, 2, 128, 1376, 3000), [100, 40], [16, 13]),   # G = 5, ffn and vocab with ragged tails
])
def test_mini_shapes_synthetic_cache(shape, ctx, chunk, attention_kind):
    wl = Workload("mini", shape, 11, len(ctx), ("list", tuple(ctx)), ("list", tuple(chunk)), 0.7)
    batch = gen.gen_batch(wl)
    glob, layers, model, kv, orc, pools = _setup(shape, wl.seed, batch)
    fill_synthetic_kv(shape, wl.seed, batch, range(batch.n_req), kv=kv, orc=orc, pools=pools)
    res = _run_and_judge(wl, shape, batch, glob, layers, kv, orc, pools)
    print(shape.name, res)


@pytest.mark.parametrize("shape,ctx,chunk,unc", [
    # chunked partial prefill (paper Sec. 4.5: fixed chunks of 32) and long uncached runs before the drafts
    (MINI_8B, [0, 40, 300, 1000, 15], [32, 17, 31, 25, 32], [32, 1, 20, 9, 28]),        # G = 4: two token groups
    (MINI_1B, [7, 260], [32, 29], [1, 29]),                                             # head_dim 64
    (ModelShape("g5c", 2, 640, 10, 2, 128, 1376, 3000), [100, 33], [32, 27], [16, 3]),  # G = 5: groups of 12
])
def test_chunks_up_to_32_and_long_uncached_runs(shape, ctx, chunk, unc, attention_kind):
    wl = Workload("chunk32", shape, 13, len(ctx), ("list", tuple(ctx)), ("list", tuple(chunk)), 0.7)
    batch = gen.gen_batch(wl)
    glob, layers, model, kv, orc, pools = _setup(shape, wl.seed, batch)
    fill_synthetic_kv(shape, wl.seed, batch, range(batch.n_req), kv=kv, orc=orc, pools=pools)
    res = _run_and_judge(wl, shape, batch, glob, layers, kv, orc, pools, uncached=unc)
    print(shape.name, res)


def test_uncached_prefix_longer_than_one_and_rerun_is_idempotent():
    shape = MINI_1B
    wl = Workload("u", shape, 5, 3, ("list", (20, 64, 7)), ("list", (6, 16, 1)), 0.7)
    batch = gen.gen_batch(wl)
    glob, layers, model, kv, orc, pools = _setup(shape, wl.seed, batch)
    fill_synthetic_kv(shape, wl.seed, batch, range(3), kv=kv, orc=orc, pools=pools)
    reqs = [oracle_teacher_forced(orc, glob, lambda l: layers[l], pools, batch.page_tables[r].numpy(),
                                  int(batch.ctx_lens[r]), wl, r, int(batch.chunk_lens[r])) for r in range(3)]
    tokens = torch.tensor([t for o in reqs for t in o.chunk], dtype=torch.int32)
    from oracle import verify_greedy
    for u in ([1, 1, 1], [3, 16, 1], [6, 5, 1]):
        acc, cor = kv.verify_batch(tokens, batch.chunk_offsets, batch.page_tables, batch.ctx_lens, n_uncached=u)
        for r, o in enumerate(reqs):
            if o.gap.min() >= 0.05:
                assert (int(acc[r]), int(cor[r])) == verify_greedy(o.top1, o.chunk, u[r])


def test_host_resident_weights_give_the_same_results():
    """syn_model_load copies from host memory (location 0) as well as from device memory."""
    import paper_2511_07423_b200 as syn
    shape = MINI_1B
    wl = Workload("h", shape, 9, 3, ("list", (30, 0, 77)), ("list", (5, 16, 2)), 0.7)
    batch = gen.gen_batch(wl)
    glob, layers = cpu_model(shape, wl.seed)
    toks = gen.gen_context_tokens(wl, 0, batch.n_tokens)
    outs = []
    for on_device in (True, False):
        g2, l2 = to_cuda(glob, layers) if on_device else (glob, layers)
        model = syn.Model(shape, g2, l2)
        kv = syn.KVCache(model, batch.n_pages)
        fill_synthetic_kv(shape, wl.seed, batch, range(3), kv=kv)
        outs.append(kv.verify_batch(toks, batch.chunk_offsets, batch.page_tables, batch.ctx_lens, want_logits=True))
        assert model.status() == 0
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1]) and torch.equal(outs[0][2], outs[1][2])


def test_plan_run_device_outputs_match_blocking_call():
    import paper_2511_07423_b200 as syn
    shape = MINI_8B
    wl = Workload("p", shape, 3, 4, ("list", (10, 200, 64, 90)), ("list", (4, 16, 1, 8)), 0.7)
    batch = gen.gen_batch(wl)
    glob, layers, model, kv, orc, pools = _setup(shape, wl.seed, batch)
    fill_synthetic_kv(shape, wl.seed, batch, range(4), kv=kv)
    toks = gen.gen_context_tokens(wl, 0, batch.n_tokens)
    acc, cor, lg = kv.verify_batch(toks, batch.chunk_offsets, batch.page_tables, batch.ctx_lens, want_logits=True)
    plan = syn.Plan(kv, toks, batch.chunk_offsets, batch.page_tables, batch.ctx_lens)
    a = torch.empty(4, dtype=torch.int32, device="cuda")
    c = torch.empty(4, dtype=torch.int32, device="cuda")
    t1 = torch.empty(batch.n_tokens, dtype=torch.int32, device="cuda")
    plan.run(a, c, t1)
    torch.cuda.synchronize()
    assert model.status() == 0
    assert torch.equal(a.cpu(), acc) and torch.equal(c.cpu(), cor)
    assert torch.equal(t1.cpu().long(), lg.argmax(-1).cpu())
    st = plan.stats()
    assert st.n_tokens == batch.n_tokens and st.n_req == 4 and st.kernel_launches > 0


def test_host_validation_errors_leave_outputs_untouched():
    """Every refused call returns its error code before any launch: the result arrays keep their
    sentinel values and the KV slots the chunks would have written keep their contents, bit for bit."""
    import paper_2511_07423_b200 as syn
    shape = TINY
    wl = CONFIGS[1]
    batch = gen.gen_batch(wl)
    glob, layers, model, kv, orc, pools = _setup(shape, wl.seed, batch)
    fill_synthetic_kv(shape, wl.seed, batch, range(batch.n_req), kv=kv)
    toks = torch.zeros(batch.n_tokens, dtype=torch.int32)
    # a good call first, so that the chunks' slots hold something a refused call could destroy
    kv.verify_batch(toks, batch.chunk_offsets, batch.page_tables, batch.ctx_lens)

    def slots():
        out = []
        for r in range(batch.n_req):
            for l in range(shape.n_layers):
                k, v = kv.export_kv(l, batch.page_tables[r], int(batch.ctx_lens[r]), int(batch.chunk_lens[r]))
                out += [k.cpu(), v.cpu()]
        return out

    before = slots()
    acc = torch.full((batch.n_req,), -77, dtype=torch.int32)
    cor = torch.full((batch.n_req,), -78, dtype=torch.int32)

    def code(**kw):
        args = dict(chunk_tokens=toks, chunk_offsets=batch.chunk_offsets, page_tables=batch.page_tables,
                    ctx_lens=batch.ctx_lens, n_uncached=None)
        args.update(kw)
        with pytest.raises(syn.SynError) as e:
            kv.verify_batch(out=(acc, cor), **args)
        torch.cuda.synchronize()
        assert (acc == -77).all() and (cor == -78).all()
        after = slots()
        assert all(torch.equal(a.view(torch.int16), b.view(torch.int16)) for a, b in zip(before, after))
        return e.value.code

    assert code(chunk_offsets=torch.tensor([0, 4, 8, 12, 45])) == -2                      # chunk of 33
    assert code(chunk_offsets=torch.tensor([0, 4, 4, 12, 16])) == -2                      # empty chunk
    assert code(n_uncached=[1, 5, 1, 1]) == -3
    assert code(n_uncached=[0, 1, 1, 1]) == -3
    bad = batch.page_tables.clone(); bad[0, 0] = batch.n_pages
    assert code(page_tables=bad) == -4
    bad = batch.page_tables.clone(); bad[1, 0] = -1
    assert code(page_tables=bad) == -4
    assert code(ctx_lens=torch.tensor([48, 64, 96, 16 * batch.max_pages - 3])) == -5
    t2 = toks.clone(); t2[3] = shape.vocab
    assert code(chunk_tokens=t2) == -6
    alias = batch.page_tables.clone(); alias[1] = alias[0]
    assert code(page_tables=alias, ctx_lens=torch.tensor([48, 48, 96, 128])) == -7
    with pytest.raises(syn.SynError):
        syn.KVCache(model, 8, page_size=32)


def test_a_plan_runs_only_on_the_cache_it_was_made_for():
    """A plan's page ids and slots were checked against one cache.  Handing it, with another cache of the
    same model (here a smaller one, where those slots would lie past the end of the pool), to the calls
    that launch kernels is refused with SYN_E_INVALID_ARG before anything is launched."""
    import paper_2511_07423_b200 as syn
    shape = TINY
    wl = CONFIGS[1]
    batch = gen.gen_batch(wl)
    glob, layers, model, kv, orc, pools = _setup(shape, wl.seed, batch)
    small = syn.KVCache(model, 2)
    toks = torch.zeros(batch.n_tokens, dtype=torch.int32)
    plan = syn.Plan(kv, toks, batch.chunk_offsets, batch.page_tables, batch.ctx_lens)
    a = torch.full((batch.n_req,), -5, dtype=torch.int32, device="cuda")
    c = torch.full((batch.n_req,), -6, dtype=torch.int32, device="cuda")
    plan.kv = small                      # the binding passes plan.kv's handle
    with pytest.raises(syn.SynError) as e:
        plan.run(a, c)
    assert e.value.code == -1
    q = torch.zeros(batch.n_tokens, shape.q_dim, dtype=torch.float16, device="cuda")
    for call in (plan.attention, plan.attention_static):
        with pytest.raises(syn.SynError) as e:
            call(0, q)
        assert e.value.code == -1
    torch.cuda.synchronize()
    assert (a == -5).all() and (c == -6).all() and model.status() == 0
    plan.kv = kv
    plan.run(a, c)                       # and on its own cache it runs
    torch.cuda.synchronize()
    assert model.status() == 0 and (a >= 0).all()


def test_last_step_stats_belong_to_the_model():
    """syn_last_step_stats(model): the counters of the last step whichever call launched it, and with
    profiling on its device time and the wall time of the blocking call."""
    import paper_2511_07423_b200 as syn
    shape = TINY
    wl = CONFIGS[1]
    batch = gen.gen_batch(wl)
    glob, layers, model, kv, orc, pools = _setup(shape, wl.seed, batch)
    with pytest.raises(syn.SynError):
        model.last_step_stats()          # no step yet
    toks = torch.zeros(batch.n_tokens, dtype=torch.int32)
    kv.verify_batch(toks, batch.chunk_offsets, batch.page_tables, batch.ctx_lens)
    st = model.last_step_stats()
    assert st.n_req == batch.n_req and st.n_tokens == batch.n_tokens and st.t_gpu_ms == 0.0 and st.h2d_bytes > 0
    assert st.kernel_launches == 1 + 5 * shape.n_layers + 2
    model.set_profile(True)
    kv.verify_batch(toks[:8], batch.chunk_offsets[:3], batch.page_tables[:2], batch.ctx_lens[:2])
    st = model.last_step_stats()
    model.set_profile(False)
    assert st.n_req == 2 and st.n_tokens == 8 and 0.0 < st.t_gpu_ms <= st.t_wall_ms
