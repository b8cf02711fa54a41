"""The arrival-driven workload of the scalability experiment (paper Sec. 6.4) on the CPU: the event
simulation of workloads/arrivals.py over the scheduler's policy (no device), with an injected,
constant service time per iteration, checked against a hand-worked three-session trace."""
import pytest

import paper_2511_07423_b200 as syn
from workloads import arrivals


def _run(arr, prompts, cfg, service=0.005):
    sched = syn.Scheduler(None, n_pages=256, page_size=16, max_batch_tokens=2048)
    batches = []

    def execute(b):
        batches.append((b["kind"], list(b["req_ids"]), int(b["n_tokens"])))
        return service, [7] * b["n_req"]

    res = arrivals.simulate(sched, execute, cfg, arr, prompt_lens=prompts)
    sched.close()
    return res, batches


def test_hand_worked_three_session_trace():
    """Service 5 ms per iteration, 10 ms each way on the network, 4 drafts of 1 ms each, every chunk
    offloaded, every draft accepted, 5 tokens per session (one verification each).
      t = 0       A arrives (32-token prompt): prefill 0 -> 5 ms; A's chunk reaches the cloud at 5 + 20 + 4 = 29 ms
      t = 27      B arrives (64 tokens): prefill of its first 32 tokens 27 -> 32 ms; A's request (29 ms) waits:
                  prompts go first (Algorithm 1), B's second chunk 32 -> 37 ms; then A is verified 37 -> 42 ms:
                  latency 42 - 29 + 20 = 33 ms.  B's chunk reaches the cloud at 37 + 24 = 61 ms
      t = 60.5    C arrives (32 tokens): prefill 60.5 -> 65.5 ms; B (61 ms) is verified 65.5 -> 70.5 ms:
                  latency 70.5 - 61 + 20 = 29.5 ms.  C's chunk at 65.5 + 24 = 89.5 ms, verified -> 94.5: 25 ms."""
    cfg = arrivals.ArrivalConfig(budget=1.0, gamma=4, device_s=0.001, rtt=0.010, out_tokens=5, p_match=1.0,
                                 vocab=1000, max_sessions=8, seed=3)
    res, batches = _run([0.0, 0.027, 0.0605], [32, 64, 32], cfg)
    assert [b[0] for b in batches] == ["prefill", "prefill", "prefill", "verify", "prefill", "verify", "verify"]
    assert [b[1] for b in batches] == [[0], [1], [1], [0], [2], [1], [2]]
    assert [b[2] for b in batches] == [32, 32, 32, 5, 32, 5, 5]
    assert res.latencies == pytest.approx([0.033, 0.0295, 0.025], abs=1e-9)
    assert res.sessions_done == 3 and res.sessions_dropped == 0
    assert res.iterations == {"prefill": 4, "verify": 3}
    assert res.busy == pytest.approx(0.035) and res.end == pytest.approx(0.0945)


def test_runs_are_a_function_of_the_seed_and_budget_zero_never_offloads_early():
    cfg = arrivals.ArrivalConfig(budget=0.0, gamma=4, device_s=0.001, rtt=0.002, out_tokens=40, p_match=0.7,
                                 prompt_lo=16, prompt_hi=80, vocab=1000, max_sessions=4, seed=11)
    arr = arrivals.poisson_arrivals(200.0, 0.05, seed=11)
    assert arr == arrivals.poisson_arrivals(200.0, 0.05, seed=11) and all(0 < a < 0.05 for a in arr) and sorted(arr) == arr
    r1, b1 = _run(arr, None, cfg)
    r2, b2 = _run(arr, None, cfg)
    assert r1.latencies == r2.latencies and b1 == b2
    # budget 0: a chunk is offloaded only when the kept tokens would no longer fit a 32-token chunk with the next
    # drafts, i.e. with 1 + 24 kept tokens + 4 drafts = 29 tokens
    assert all(n == 29 for kind, _, n in b1 if kind == "verify" for n in [n // max(1, len(_))] if len(_) == 1)
    assert r1.sessions_done + r1.sessions_dropped == len(arr)
    # more load, longer waits: the same arrivals against a slower cloud
    slow, _ = _run(arr, None, cfg, service=0.02)
    assert sum(slow.latencies) / len(slow.latencies) > sum(r1.latencies) / len(r1.latencies)
