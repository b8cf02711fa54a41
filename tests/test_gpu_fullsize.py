"""Parity at the full sizes of configurations 2..6, in the launch configuration bench.py times: the
whole batch goes through syn_verify_batch on the GPU (seeded synthetic cache), and the CPU oracle (all
intermediates in double) judges EVERY request of configurations 2 and 3, 32 requests of configuration 4
and 8 of configuration 5 (a seeded choice that always holds the longest chunk and the longest context).
The judged requests' drafts come from the ORACLE's argmax by the sequential rule, the other requests'
from the library's.  For every judged request accept_len / correction_token must follow the stated
rule (bit-exact unless a consulted position's top-2 gap is below 0.05, where either of the oracle's two
best ids may be taken), and the logits must agree within 3e-2 x the standard deviation of the oracle's
logits, at every depth up to 32 layers.  At the 64 layers of configuration 5 the rounding of 16-bit
operands does not allow that: the error of half-precision operands (11 significant bits) grows like
0.0008 x sqrt(layers) rms (measured 0.0011 / 0.0023 / 0.0043 / 0.0064 at 2 / 16 / 32 / 64 layers) and its
maximum over ten million logits sits six standard deviations out, 0.038 measured; the bound asserted
there is 0.045.  Strict / soft counts are printed; if fewer than half of the judged requests are strict
the test says so."""
import numpy as np
import pytest
import torch

from oracle import Oracle, verify_greedy
from workloads import gen, rng
from workloads.configs import CONFIGS

from harness import LOGIT_TOL, admissible_results, oracle_teacher_forced_many

pytestmark = pytest.mark.gpu

# requests the oracle judges per configuration (None: all), and how many it walks through together
JUDGED = {2: (None, 32), 3: (None, 16), 4: (32, 16), 5: (8, 4), 6: (3, 3)}


def judged_requests(wl, batch, count):
    if count is None or count >= batch.n_req:
        return list(range(batch.n_req))
    n, ctx = batch.chunk_lens.tolist(), batch.ctx_lens.tolist()
    picks = [max(range(batch.n_req), key=lambda r: (n[r], ctx[r])), max(range(batch.n_req), key=lambda r: ctx[r]),
             min(range(batch.n_req), key=lambda r: (n[r], -ctx[r]))]
    for r in rng.permutation(rng.stream_key(wl.seed, 901), batch.n_req).tolist():
        if len(set(picks)) >= count:
            break
        picks.append(r)
    return sorted(set(picks))


def weight_source(shape, seed):
    """layer -> weights on the CPU.  Held in host memory when they fit beside everything else, else
    regenerated on the GPU and copied per use (the 32B shape is 64 GB)."""
    import psutil
    per_layer = 2 * (shape.d_model * (shape.q_dim + 2 * shape.kv_dim) + shape.q_dim * shape.d_model + 3 * shape.d_model * shape.d_ffn)
    cache = {}
    keep_all = per_layer * shape.n_layers < 0.4 * psutil.virtual_memory().available

    def layer_w(l):
        if l not in cache:
            if not keep_all:
                cache.clear()
            cache[l] = {k: v.cpu() for k, v in gen.gen_layer(shape, seed, l, device="cuda").items()}
        return cache[l]
    return layer_w


def logit_tolerance(n_layers: int) -> float:
    return LOGIT_TOL if n_layers <= 32 else 0.045


@pytest.mark.parametrize("cfg", [2, 3, 4, 5, 6])
def test_judged_requests_match_the_oracle_at_full_size(cfg):
    import paper_2511_07423_b200 as syn
    from paper_2511_07423_b200 import synthetic
    wl = CONFIGS[cfg]
    shape = wl.shape
    model = synthetic.load_model(shape, wl.seed, via_host=shape.dense_params() * 2 > 40e9)
    kv = None
    try:
        kv = _judge(syn, synthetic, cfg, wl, shape, model)
    finally:   # a failure must not leave 100+ GB behind for the next configuration
        if kv is not None:
            kv.close()
        model.close()
        torch.cuda.empty_cache()


def _judge(syn, synthetic, cfg, wl, shape, model):
    pool_tokens = None
    if wl.fit_to_pool:
        free, _ = torch.cuda.mem_get_info()
        pool_tokens = int((free - 6e9) // shape.kv_bytes_per_token()) // 16 * 16
    batch = gen.gen_batch(wl, pool_tokens=pool_tokens)
    kv = syn.KVCache(model, batch.n_pages)
    try:
        _judge_batch(syn, synthetic, cfg, wl, shape, model, kv, batch)
    except BaseException:
        kv.close()
        raise
    return kv


def _judge_batch(syn, synthetic, cfg, wl, shape, model, kv, batch):
    synthetic.fill_cache(kv, shape, wl.seed, batch)
    offs, unc = batch.chunk_offsets.tolist(), batch.n_uncached.tolist()

    orc = Oracle(shape)
    glob = {k: v.cpu() for k, v in gen.gen_globals(shape, wl.seed, device="cuda").items()}
    layer_w = weight_source(shape, wl.seed)
    count, together = JUDGED[cfg]
    picks = judged_requests(wl, batch, count)
    oracle_reqs = {}
    for g in range(0, len(picks), together):
        oracle_reqs.update(oracle_teacher_forced_many(orc, glob, layer_w, wl, shape, wl.seed, batch, picks[g:g + together]))
    toks = synthetic.teacher_forced_chunks(kv, wl, batch, fixed={r: o.chunk for r, o in oracle_reqs.items()})
    acc, cor, logits = kv.verify_batch(toks, batch.chunk_offsets, batch.page_tables, batch.ctx_lens,
                                       n_uncached=batch.n_uncached, want_logits=True)
    assert model.status() == 0
    # which attention kernel the planner took: the tcgen05 one where a chunk is more than one 64-row tile
    assert model.last_step_stats().attn_rows == (128 if cfg in (5, 6) else 64)
    # the same step again: bit-identical (static schedules, fixed summation orders, counters back at zero)
    acc2, cor2, logits2 = kv.verify_batch(toks, batch.chunk_offsets, batch.page_tables, batch.ctx_lens,
                                          n_uncached=batch.n_uncached, want_logits=True)
    assert torch.equal(acc, acc2) and torch.equal(cor, cor2) and torch.equal(logits, logits2)
    del logits2
    # every request: results are in range and consistent with the returned logits' argmax
    top1_gpu = logits.argmax(-1).cpu()
    for r in range(batch.n_req):
        chunk = toks[offs[r]:offs[r + 1]].tolist()
        assert (int(acc[r]), int(cor[r])) == verify_greedy(top1_gpu[offs[r]:offs[r + 1]].tolist(), chunk, unc[r])

    n_strict = n_equal = 0
    worst = worst_rms = 0.0
    sigma = float(np.concatenate([o.logits.ravel() for o in oracle_reqs.values()]).std())
    bad = []
    for r, o in oracle_reqs.items():
        ok, strict = admissible_results(o)
        got = (int(acc[r]), int(cor[r]))
        n_equal += got == (o.accept_len, o.correction)
        if strict:
            n_strict += 1
            if got != (o.accept_len, o.correction):
                bad.append((r, "strict", got, (o.accept_len, o.correction), float(o.gap.min())))
        elif got not in ok:
            bad.append((r, "soft", got, sorted(ok), float(o.gap.min())))
        dl = logits[offs[r]:offs[r + 1]].to("cpu", torch.float64).numpy() - o.logits
        worst = max(worst, float(np.abs(dl).max()) / sigma)
        worst_rms = max(worst_rms, float(np.sqrt((dl ** 2).mean())) / sigma)
    n = len(oracle_reqs)
    print(f"config {cfg}: judged {n} of {batch.n_req} requests ({sum(len(o.chunk) for o in oracle_reqs.values())} tokens), "
          f"strict {n_strict}, soft {n - n_strict}, equal to the oracle {n_equal}; max |dlogit|/sigma {worst:.4f}, "
          f"largest per-request rms {worst_rms:.5f} (tolerance {logit_tolerance(shape.n_layers)}); ctx scale {batch.scale:.3f}")
    if 2 * n_strict < n:
        print(f"config {cfg}: FEWER THAN HALF of the judged requests are strict ({n_strict} of {n}): most results rest on the "
              f"top-2-gap exemption")
    assert not bad, bad
    assert worst <= logit_tolerance(shape.n_layers), f"config {cfg}: max |dlogit| / sigma = {worst:.4f}"
