"""The full-width code paths held to a TIGHT logit tolerance: 2-layer models at the FULL width of the
8B and 32B shapes (d_model, d_ffn, vocabulary, head geometry) with the FULL batches of configurations 3
and 5, once on the kernels their shapes call for (CTA pairs: 512- and 256-feature items, K shared
between clusters, leftover items cut along K) and once with every projection on the one-CTA kernel
(pair tiles in full waves with leftover tiles cut along K under the SwiGLU and lm_head epilogues, K
shared between CTAs under the qkv and residual epilogues, mixed waves of pair and single tiles); four
row tiles and split key ranges in the attention.  At two layers the half-precision operands leave about
0.001 sigma rms, so a slip in any epilogue, schedule or exchange shows: the bound asserted is a third of
the stated 0.03 sigma.  The oracle judges a seeded choice of requests; their drafts come from the
ORACLE's argmax (sequential rule), the other requests' from the library's."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import Oracle
from workloads import gen, rng
from workloads.configs import CONFIGS

from harness import LOGIT_TOL, admissible_results, oracle_teacher_forced

pytestmark = pytest.mark.gpu


def judged_requests(wl, batch, count):
    """Seeded choice: the request with the longest chunk, the one with the longest context, and
    `count - 2` more drawn without replacement from the configuration's own stream."""
    n, ctx = batch.chunk_lens.tolist(), batch.ctx_lens.tolist()
    picks = [max(range(batch.n_req), key=lambda r: (n[r], ctx[r])), max(range(batch.n_req), key=lambda r: ctx[r])]
    order = rng.permutation(rng.stream_key(wl.seed, 901), batch.n_req).tolist()
    for r in order:
        if len(picks) >= count:
            break
        if r not in picks:
            picks.append(r)
    return sorted(set(picks))


@pytest.mark.parametrize("cfg,n_judged,schedule", [(3, 6, 0), (3, 6, 1), (5, 4, 0), (5, 4, 1)])
def test_two_layers_at_full_width_meet_a_third_of_the_stated_tolerance(cfg, n_judged, schedule):
    import paper_2511_07423_b200 as syn
    from paper_2511_07423_b200 import synthetic
    syn.debug_set_schedule(schedule)
    try:
        _run(cfg, n_judged)
    finally:
        syn.debug_set_schedule(0)


def test_wide_batch_at_the_1b_width_puts_64_wide_heads_through_the_pair_kernels():
    """Configuration 2's own batch (129 tokens) stays on the one-CTA kernel.  A wider mix at the same width
    (64 requests, chunks of 9-16 tokens: about 800 tokens) sends the qkv projection (64-wide heads, two per
    128-feature tile), gate/up, down (K shared between clusters) and the lm_head through the CTA-pair kernel."""
    import paper_2511_07423_b200 as syn
    base = CONFIGS[2]
    wl = dataclasses.replace(base, name="1b-wide", n_req=64, ctx=("uniform", 64, 768), chunk=("uniform", 9, 16))
    T = int(gen.gen_batch(dataclasses.replace(wl, shape=dataclasses.replace(base.shape, n_layers=2))).chunk_offsets[-1])
    s = base.shape
    assert syn.gemm2_plan_host(T, s.q_dim + 2 * s.kv_dim, s.d_model, "qkv")["kind"] != 0
    assert syn.gemm2_plan_host(T, s.d_model, s.d_ffn, "resid")["splits"] > 1
    _run(2, 4, wl)


def _run(cfg, n_judged, base=None):
    import paper_2511_07423_b200 as syn
    from paper_2511_07423_b200 import synthetic
    base = base or CONFIGS[cfg]
    shape = dataclasses.replace(base.shape, n_layers=2, name=base.shape.name + "-2l")
    wl = dataclasses.replace(base, shape=shape, fit_to_pool=False)
    model = synthetic.load_model(shape, wl.seed)
    batch = gen.gen_batch(wl)
    kv = syn.KVCache(model, batch.n_pages)
    synthetic.fill_cache(kv, shape, wl.seed, batch)
    offs, unc = batch.chunk_offsets.tolist(), batch.n_uncached.tolist()

    orc = Oracle(shape)
    glob = {k: v.cpu() for k, v in gen.gen_globals(shape, wl.seed, device="cuda").items()}
    layers = [{k: v.cpu() for k, v in gen.gen_layer(shape, wl.seed, l, device="cuda").items()} for l in range(shape.n_layers)]
    picks = judged_requests(wl, batch, n_judged)
    oracle_reqs = {}
    for r in picks:
        ctx, n = int(batch.ctx_lens[r]), int(batch.chunk_lens[r])
        n_pages = -(-(ctx + n) // 16)
        pt = np.arange(n_pages, dtype=np.int32)          # the oracle's own contiguous placement
        pools = orc.new_pool(n_pages)
        for l in range(shape.n_layers):
            k, v = gen.gen_kv(shape, wl.seed, l, r, 0, ctx)
            orc.load_kv(pools[l], pt, 0, k.float().numpy(), v.float().numpy())
        oracle_reqs[r] = oracle_teacher_forced(orc, glob, lambda l: layers[l], pools, pt, ctx, wl, r, n, u=unc[r])
    toks = synthetic.teacher_forced_chunks(kv, wl, batch, fixed={r: o.chunk for r, o in oracle_reqs.items()})
    acc, cor, logits = kv.verify_batch(toks, batch.chunk_offsets, batch.page_tables, batch.ctx_lens,
                                       n_uncached=batch.n_uncached, want_logits=True)
    assert model.status() == 0
    n_strict, worst, worst_rms = 0, 0.0, 0.0
    for r, o in oracle_reqs.items():
        ok, strict = admissible_results(o)
        got = (int(acc[r]), int(cor[r]))
        sigma = float(o.logits.std())
        g = logits[offs[r]:offs[r + 1]].to("cpu", torch.float64).numpy()
        dl = g - o.logits
        worst = max(worst, float(np.abs(dl).max()) / sigma)
        worst_rms = max(worst_rms, float(np.sqrt((dl ** 2).mean())) / sigma)
        print(f"request {r}: n {len(o.chunk)} ctx {int(batch.ctx_lens[r])} max|d|/sigma {np.abs(dl).max() / sigma:.4f} "
              f"rms {np.sqrt((dl ** 2).mean()) / sigma:.5f} strict {strict} got {got} oracle {(o.accept_len, o.correction)}")
        if strict:
            n_strict += 1
            assert got == (o.accept_len, o.correction), (cfg, r, got, (o.accept_len, o.correction))
        else:
            assert got in ok, (cfg, r, got, sorted(ok))
    print(f"config {cfg} width, 2 layers: judged {picks}, strict {n_strict}/{len(picks)}, "
          f"max |dlogit|/sigma {worst:.4f} (rms {worst_rms:.5f}), bound {LOGIT_TOL / 3:.3f}")
    assert worst <= LOGIT_TOL / 3, f"max |dlogit| / sigma = {worst:.4f} > {LOGIT_TOL / 3}"
    kv.close()
    model.close()
    torch.cuda.empty_cache()


def test_logit_error_grows_like_the_square_root_of_the_depth():
    """Depth study behind the tolerance: the 1B width (configuration 2's batch and geometry) at 1, 2, 4, 8 and 16
    layers.  The rms difference to the oracle follows c x sqrt(layers) with c about 0.0008 sigma (the rounding of
    the half-precision operands, added in quadrature layer by layer); the bound asserted is 0.0012 sqrt(L), and
    the maximum over all judged logits stays below 0.03 sigma at every depth."""
    import paper_2511_07423_b200 as syn
    from paper_2511_07423_b200 import synthetic
    base = CONFIGS[2]
    rows = []
    for n_layers in (1, 2, 4, 8, 16):
        shape = dataclasses.replace(base.shape, n_layers=n_layers, name=f"1b-{n_layers}l")
        wl = dataclasses.replace(base, shape=shape)
        model = synthetic.load_model(shape, wl.seed)
        batch = gen.gen_batch(wl)
        kv = syn.KVCache(model, batch.n_pages)
        try:
            synthetic.fill_cache(kv, shape, wl.seed, batch)
            offs, unc = batch.chunk_offsets.tolist(), batch.n_uncached.tolist()
            orc = Oracle(shape)
            glob = {k: v.cpu() for k, v in gen.gen_globals(shape, wl.seed, device="cuda").items()}
            layers = [{k: v.cpu() for k, v in gen.gen_layer(shape, wl.seed, l, device="cuda").items()} for l in range(n_layers)]
            picks = judged_requests(wl, batch, 3)
            reqs = {}
            for r in picks:
                ctx, n = int(batch.ctx_lens[r]), int(batch.chunk_lens[r])
                n_pages = -(-(ctx + n) // 16)
                pt = np.arange(n_pages, dtype=np.int32)
                pools = orc.new_pool(n_pages)
                for l in range(n_layers):
                    k, v = gen.gen_kv(shape, wl.seed, l, r, 0, ctx)
                    orc.load_kv(pools[l], pt, 0, k.float().numpy(), v.float().numpy())
                reqs[r] = oracle_teacher_forced(orc, glob, lambda l: layers[l], pools, pt, ctx, wl, r, n, u=unc[r])
            toks = synthetic.teacher_forced_chunks(kv, wl, batch, fixed={r: o.chunk for r, o in reqs.items()})
            _, _, logits = kv.verify_batch(toks, batch.chunk_offsets, batch.page_tables, batch.ctx_lens,
                                           n_uncached=batch.n_uncached, want_logits=True)
            assert model.status() == 0
            ref = np.concatenate([o.logits for o in reqs.values()])
            got = np.concatenate([logits[offs[r]:offs[r + 1]].to("cpu", torch.float64).numpy() for r in reqs])
            sigma = float(ref.std())
            rows.append((n_layers, float(np.sqrt(((got - ref) ** 2).mean())) / sigma, float(np.abs(got - ref).max()) / sigma))
        finally:
            kv.close()
            model.close()
            torch.cuda.empty_cache()
    print("layers  rms/sigma  max/sigma  rms / sqrt(layers)")
    for n_layers, rms, mx in rows:
        print(f"{n_layers:6d}  {rms:9.5f}  {mx:9.5f}  {rms / np.sqrt(n_layers):9.5f}")
        assert rms <= 0.0012 * np.sqrt(n_layers) and mx <= LOGIT_TOL
    assert 2.0 <= rows[-1][1] / rows[0][1] <= 8.0      # sixteen times the depth: about four times the error
