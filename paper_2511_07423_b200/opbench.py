"""Time single kernels of the step through the C ABI (CUDA events on the launching stream).

    python -m paper_2511_07423_b200.opbench linear --T 544 --N 28672 --K 4096
    python -m paper_2511_07423_b200.opbench attention --config 3
    python -m paper_2511_07423_b200.opbench sched --config 2 --rounds 8
    python -m paper_2511_07423_b200.opbench sample --config 3
    python -m paper_2511_07423_b200.opbench scale --config 2 --budgets 0.3,0.6,0.9 --rates 2,4,8,16,32

`attention` builds a one-layer model with the attention geometry of the chosen configuration
and that configuration's request mix (seeded synthetic cache), so one launch reads one layer's
worth of the configuration's KV.  `sched` drives the verification-aware scheduler with the
configuration's request mix: every request's context arrives as a prompt (prefilled in 32-token
chunks, prompts first), then each request offloads `--rounds` chunks drawn from the mix; it
reports the iterations by kind and the share of the wall time spent in the scheduler's own code.
`sample` times the sampling-verification stage (top-k of the logits rows + the per-request kernel)
behind a one-layer model with the configuration's vocabulary and request mix.
`scale` is the scalability experiment of the paper's Sec. 6.4 in shape: the arrival-driven workload
of workloads/arrivals.py (sessions arrive at a given rate, every device drafts chunks of gamma tokens
at a fixed pace and offloads a chunk with probability = the offloading budget) with the scheduler over
the real model on this GPU as its cloud.  Device and network time are simulated, cloud time is the
measured wall time of every iteration; the output is the verification latency per request against the
arrival rate.
"""
from __future__ import annotations

import argparse
import dataclasses
import json

import torch

from workloads import gen, rng
from workloads.configs import CONFIGS, ModelShape

from . import binding as syn
from . import synthetic


def _time(fn, iters: int, warmup: int = 3):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for a, b in ev:
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    ts = sorted(a.elapsed_time(b) for a, b in ev)
    return ts[len(ts) // 2], ts[0]


def bench_linear(a):
    syn.debug_set_schedule(1 if a.one_cta else 0)
    key = rng.stream_key(0, 1234)
    x = rng.normal_f32(key, 0, a.T * a.K, 1.0, device="cuda").view(a.T, a.K).to(torch.float16)
    w = rng.normal_f32(key, a.T * a.K, a.N * a.K, 0.02, device="cuda").view(a.N, a.K).to(torch.bfloat16)
    syn.syn_op_linear(x, w, schedule_as=a.sched)
    med, best = _time(lambda: syn.syn_op_linear(x, w, schedule_as=a.sched, reuse_pack=True), a.iters)
    fl = 2.0 * a.T * a.N * a.K
    print(json.dumps({"op": "linear", "sched": a.sched, "one_cta": bool(a.one_cta), "T": a.T, "N": a.N, "K": a.K, "ms_median": med, "ms_best": best,
                      "tflops": fl / med / 1e9, "weight_gbs": 2.0 * a.N * a.K / med / 1e6,
                      "note": "includes the fp32 [T][N] store of the test epilogue and a stream sync per call"}))


def bench_attention(a):
    syn.debug_set_attention(a.kind)
    wl = CONFIGS[a.config]
    s = wl.shape
    shape = ModelShape(f"attn-{s.name}", 1, s.d_model, s.n_q_heads, s.n_kv_heads, s.head_dim, 1024, 1024)
    model = synthetic.load_model(shape, wl.seed)
    batch = gen.gen_batch(wl, pool_tokens=a.pool_tokens)
    kv = syn.KVCache(model, batch.n_pages)
    for r in range(batch.n_req):
        tot = int(batch.ctx_lens[r] + batch.chunk_lens[r])
        k, v = gen.gen_kv(shape, wl.seed, 0, r, 0, tot, device="cuda")
        kv.import_kv(0, batch.page_tables[r], 0, k, v)
    T = batch.n_tokens
    q = rng.normal_f32(rng.stream_key(wl.seed, 77), 0, T * shape.q_dim, 1.5, device="cuda").view(T, shape.q_dim).to(torch.float16)
    plan = syn.Plan(kv, torch.zeros(T, dtype=torch.int32), batch.chunk_offsets, batch.page_tables, batch.ctx_lens)
    out = torch.empty_like(q)
    model.set_profile(True)
    for _ in range(3):
        plan.attention(0, q, out)
    model.get_profile()
    for _ in range(a.iters):
        plan.attention(0, q, out)
    prof = model.get_profile()
    st = plan.stats()
    kvb = st.kv_read_bytes  # one layer
    ms_att = prof["attention"][0] / prof["attention"][1]
    ms_mrg = prof["attention_merge"][0] / max(1, prof["attention_merge"][1])
    print(json.dumps({"op": "attention", "kind": a.kind, "config": wl.name, "n_req": batch.n_req, "T": T, "kv_bytes": kvb,
                      "items": st.attn_items, "split_items": st.attn_split_items, "ms_attention": ms_att,
                      "ms_merge": ms_mrg, "kv_gbs": kvb / ms_att / 1e6, "kv_gbs_with_merge": kvb / (ms_att + ms_mrg) / 1e6,
                      "attn_tflops": st.attn_flops / ms_att / 1e9}))


def bench_sched(a):
    import time
    wl = CONFIGS[a.config]
    shape = wl.shape
    model = synthetic.load_model(shape, wl.seed)
    batch = gen.gen_batch(wl)
    B = batch.n_req
    n_pages = int(batch.n_pages + B * (a.rounds * 2 + 2))
    kv = syn.KVCache(model, n_pages)
    sched = syn.Scheduler(kv, max_batch_tokens=a.budget)
    t_start = time.perf_counter()
    for r in range(B):
        sched.add_request(r, gen.gen_context_tokens(wl, r, int(batch.ctx_lens[r])))
    rounds = [0] * B
    per_kind = {"prefill": [0, 0.0, 0], "verify": [0, 0.0, 0]}
    while True:
        t0 = time.perf_counter()
        kind, results = sched.step()
        dt = time.perf_counter() - t0
        if kind == "idle":
            break
        e = per_kind[kind]
        e[0] += 1
        e[1] += dt
        e[2] += sum(x["n_tokens"] for x in results)
        for x in results:
            r = x["req_id"]
            if not x["prompt_done"]:
                continue
            if rounds[r] >= a.rounds:
                sched.finish(r)
                continue
            # the device's next chunk: the correction token, then drafts (uniform ids: the timing does
            # not depend on how many are accepted)
            n = int(batch.chunk_lens[r])
            chunk = [x["correction_token"]] + gen.gen_context_tokens(wl, 1000 + r, rounds[r] + n)[rounds[r]:rounds[r] + n - 1].tolist()
            sched.add_verify(r, chunk, 1)
            rounds[r] += 1
    wall = time.perf_counter() - t_start
    assert model.status() == 0
    st = sched.stats()
    out = {"op": "sched", "config": wl.name, "n_req": B, "rounds": a.rounds, "max_batch_tokens": a.budget,
           "wall_s": wall, "scheduler_host_s": st.host_seconds, "execute_s": st.execute_seconds,
           "scheduler_share_of_library_time": st.host_seconds / (st.host_seconds + st.execute_seconds),
           "deferred": st.deferred}
    for k, (n, t, tok) in per_kind.items():
        out[k] = {"iterations": n, "tokens": tok, "ms_per_iteration": 1e3 * t / max(1, n), "tokens_per_s": tok / max(t, 1e-9)}
    out["scheduler_us_per_iteration"] = 1e6 * st.host_seconds / max(1, st.iterations[1] + st.iterations[2])
    print(json.dumps(out))


def bench_sample(a):
    wl = CONFIGS[a.config]
    s = wl.shape
    shape = ModelShape(f"sample-{s.name}", 1, s.d_model, s.n_q_heads, s.n_kv_heads, s.head_dim, 1024, s.vocab)
    model = synthetic.load_model(shape, wl.seed)
    batch = gen.gen_batch(wl)
    kv = syn.KVCache(model, batch.n_pages)
    T, B = batch.n_tokens, batch.n_req
    toks = gen.gen_context_tokens(wl, 0, T)
    key = rng.stream_key(wl.seed, 4242)
    slm_k = a.slm_k
    # transmitted rows: the draft itself with probability 0.5, the rest spread over random ids
    slm_ids = rng.randint(key, 0, T * slm_k, 0, s.vocab - 1).to(torch.int32).view(T, slm_k)
    slm_ids[:, 0] = toks
    slm_probs = torch.full((T, slm_k), 0.5 / max(1, slm_k - 1))
    slm_probs[:, 0] = 0.5 if slm_k > 1 else 1.0
    ra = rng.uniform01(key, 1 << 20, T).float().clamp_(0, 0.999999)
    rs = rng.uniform01(key, 2 << 20, B).float().clamp_(0, 0.999999)
    cfg = syn.Sampling(a.top_k, a.top_p, 1.0, slm_k)
    args = (kv, toks, batch.chunk_offsets, batch.page_tables, batch.ctx_lens, batch.n_uncached, cfg, slm_ids, slm_probs, ra, rs)
    for _ in range(3):
        syn.verify_batch_sampled(*args)
    model.set_profile(True)
    model.get_profile()
    for _ in range(a.iters):
        syn.verify_batch_sampled(*args)
    prof = model.get_profile()
    ms = prof["verify"][0] / a.iters          # greedy compare + top-k rows + sampling kernel, per step
    rows = int((batch.chunk_lens - batch.n_uncached + 1).sum())
    by = rows * s.vocab * 4
    print(json.dumps({"op": "sample", "config": wl.name, "T": T, "rows_with_a_distribution": rows, "vocab": s.vocab,
                      "top_k": a.top_k, "top_p": a.top_p, "slm_k": slm_k, "ms_sampling_stage": ms, "logit_bytes_read_once": by,
                      "gbs": by / ms / 1e6}))


def bench_scale(a):
    import time
    from workloads import arrivals
    wl = CONFIGS[a.config]
    shape = wl.shape
    model = synthetic.load_model(shape, wl.seed)
    lo, hi = wl.ctx[1], wl.ctx[2]                      # prompt lengths: the configuration's context range
    n_pages = int(a.max_sessions * ((hi + a.out_tokens + 64) // 16 + 1))
    kv = syn.KVCache(model, n_pages)

    def execute(b):                                    # one real iteration on this GPU, wall time
        t0 = time.perf_counter()
        _, cor = kv.verify_batch(b["chunk_tokens"], b["chunk_offsets"], b["page_tables"], b["ctx_lens"],
                                 n_uncached=b["n_uncached"])
        return time.perf_counter() - t0, cor

    for budget in [float(x) for x in a.budgets.split(",")]:
        for rate in [float(x) for x in a.rates.split(",")]:
            seed = int(1000 * budget) * 7919 + int(100 * rate)
            cfg = arrivals.ArrivalConfig(budget=budget, gamma=a.gamma, device_s=a.device_ms * 1e-3, rtt=a.rtt_ms * 1e-3,
                                         out_tokens=a.out_tokens, p_match=wl.p_match, prompt_lo=lo, prompt_hi=hi,
                                         vocab=shape.vocab, max_sessions=a.max_sessions, seed=seed)
            sched = syn.Scheduler(kv, max_batch_tokens=a.budget_tokens)
            res = arrivals.simulate(sched, execute, cfg, arrivals.poisson_arrivals(rate, a.horizon, seed), stop_after=3 * a.horizon)
            sched.close()
            print(json.dumps(dict({"op": "scale", "config": wl.name, "offload_budget": budget, "arrival_rate_per_s": rate},
                                  **res.summary())), flush=True)
    assert model.status() == 0


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="op", required=True)
    l = sub.add_parser("linear")
    l.add_argument("--T", type=int, default=544)
    l.add_argument("--N", type=int, default=28672)
    l.add_argument("--K", type=int, default=4096)
    l.add_argument("--iters", type=int, default=10)
    l.add_argument("--sched", default="plain", help="schedule: plain, qkv, resid, swiglu, lmhead, pair_quad, pair_duo, pair_quad_resid, pair_duo_resid")
    l.add_argument("--one-cta", action="store_true", help="keep the projection on the one-CTA kernel whatever its shape")
    t = sub.add_parser("attention")
    t.add_argument("--config", type=int, default=3)
    t.add_argument("--pool-tokens", type=int, default=None)
    t.add_argument("--kind", type=int, default=0, help="attention kernel: 0 default, 1 warp-level MMAs, 2 tcgen05")
    t.add_argument("--iters", type=int, default=10)
    m = sub.add_parser("sample")
    m.add_argument("--config", type=int, default=3)
    m.add_argument("--top-k", type=int, default=50)
    m.add_argument("--top-p", type=float, default=0.9)
    m.add_argument("--slm-k", type=int, default=20)
    m.add_argument("--iters", type=int, default=10)
    z = sub.add_parser("scale")
    z.add_argument("--config", type=int, default=2)
    z.add_argument("--budgets", default="0.3,0.6,0.9")
    z.add_argument("--rates", default="2,4,8,16,32", help="session arrivals per second")
    z.add_argument("--horizon", type=float, default=10.0, help="seconds of arrivals (virtual time)")
    z.add_argument("--out-tokens", type=int, default=128)
    z.add_argument("--gamma", type=int, default=4)
    z.add_argument("--device-ms", type=float, default=25.0, help="device time per drafted token")
    z.add_argument("--rtt-ms", type=float, default=10.0, help="one-way network delay")
    z.add_argument("--max-sessions", type=int, default=512)
    z.add_argument("--budget-tokens", type=int, default=2048, help="chunk tokens per iteration")
    c = sub.add_parser("sched")
    c.add_argument("--config", type=int, default=2)
    c.add_argument("--rounds", type=int, default=8)
    c.add_argument("--budget", type=int, default=2048, help="chunk tokens per iteration")
    a = ap.parse_args()
    {"linear": bench_linear, "attention": bench_attention, "sched": bench_sched, "sample": bench_sample, "scale": bench_scale}[a.op](a)


if __name__ == "__main__":
    main()
