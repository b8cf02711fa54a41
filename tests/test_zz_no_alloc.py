"""syn_op_attention_static, the attention entry point for callers that cannot allocate device
memory while they run (inside a stream capture, or in a server whose memory was handed out up
front), against the ordinary syn_op_attention on the same plan.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from workloads import gen, rng
from workloads.configs import ModelShape, Workload

from harness import cpu_model, to_cuda

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("hd", [128, 64])
def test_static_scratch_attention_equals_the_allocating_one_twice_in_a_row(hd, attention_kind):
    import paper_2511_07423_b200 as syn
    shape = ModelShape("att-static", 1, 256, 8, 2, hd, 256, 512)
    seed = 21
    # long contexts, so that key ranges are split over work items and the partial-result array is used
    wl = Workload("t", None, seed, 4, ("list", (1500, 40, 2300, 900)), ("list", (16, 3, 9, 1)), 0.5)
    batch = gen.gen_batch(wl)
    glob, layers = cpu_model(shape, seed)
    gg, gl = to_cuda(glob, layers)
    model = syn.Model(shape, gg, gl)
    kv = syn.KVCache(model, batch.n_pages)
    T = batch.n_tokens
    for r in range(batch.n_req):
        tot = int(batch.ctx_lens[r] + batch.chunk_lens[r])
        k, v = gen.gen_kv(shape, seed, 0, r, 0, tot, device="cuda")
        kv.import_kv(0, batch.page_tables[r], 0, k, v)
    plan = syn.Plan(kv, torch.zeros(T, dtype=torch.int32), batch.chunk_offsets, batch.page_tables, batch.ctx_lens)
    assert plan.stats().attn_split_items > 0
    out_static = torch.empty(T, shape.q_dim, dtype=torch.float16, device="cuda")
    for call in range(2):   # the second call finds the first call's partials in the shared array
        q = rng.normal_f32(rng.stream_key(seed, 77 + call), 0, T * shape.q_dim, 1.5, device="cuda") \
            .view(T, shape.q_dim).to(torch.float16)
        ref = plan.attention(0, q)
        torch.cuda.synchronize()
        out_static.fill_(float("nan"))
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        plan.attention_static(0, q, out=out_static)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        # what the entry point is for: the device's free memory is the same before and after the call
        # (from the second call on: the first one on a device looks the array's address up)
        if call > 0:
            assert free_after == free_before
        assert model.status() == 0
        a, b = out_static.float().cpu().numpy(), ref.float().cpu().numpy()
        assert np.isfinite(a).all()
        assert np.abs(a - b).max() <= 0.02 * np.abs(b).max()   # the tolerance of the attention parity test


def test_static_scratch_attention_refuses_more_partials_than_it_holds():
    import paper_2511_07423_b200 as syn
    # 147 equal (request, kv head) units on 148 SMs: each is a little more than one CTA's share,
    # so the planner splits every one in two -> 294 partial items, more than the fixed array holds
    shape = ModelShape("att-static", 1, 256, 21, 21, 128, 256, 512)
    seed = 22
    wl = Workload("t", None, seed, 7, ("const", 2000), ("const", 1), 0.5)
    batch = gen.gen_batch(wl)
    glob, layers = cpu_model(shape, seed)
    gg, gl = to_cuda(glob, layers)
    model = syn.Model(shape, gg, gl)
    kv = syn.KVCache(model, batch.n_pages)
    T = batch.n_tokens
    plan = syn.Plan(kv, torch.zeros(T, dtype=torch.int32), batch.chunk_offsets, batch.page_tables, batch.ctx_lens)
    assert plan.stats().attn_split_items > 256
    q = torch.zeros(T, shape.q_dim, dtype=torch.float16, device="cuda")
    with pytest.raises(syn.SynError) as e:
        plan.attention_static(0, q)
    assert e.value.code == -5
