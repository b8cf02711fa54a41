"""Arrival-driven workload in the shape of the paper's scalability experiment (Sec. 6.4): sessions
arrive over time, every session's device drafts chunks of gamma tokens at a fixed pace and offloads
a chunk to the cloud with probability = the offloading budget; the cloud is the verification-aware
scheduler (Algorithm 1) over some executor.  Reported: the verification latency per request against
the arrival rate.

This module holds the EVENT SIMULATION only.  It draws every random number from ``workloads.rng``
(arrival gaps, prompt lengths, offload decisions, accepted drafts), so a run is a pure function of its
seed; it knows nothing of the verification step's arithmetic.  The cloud is handed in:
``sched`` (anything with ``add_request / add_verify / finish / peek / commit`` like the library's
scheduler) and ``execute(batch) -> (seconds, correction_tokens)``: the measured wall time of a real
iteration on a GPU, or an injected service time in a CPU test.

Model of one session (times in seconds):
  - it arrives with a prompt; the cloud prefills it in the scheduler's 32-token chunks;
  - when the prompt is done the result travels to the device (one-way delay ``rtt``), the device
    drafts gamma tokens (``device_s`` each) and its next message reaches the cloud after another
    ``rtt``: the "chunk" event, at completion + 2 rtt + gamma device_s;
  - at a chunk event the device offloads (probability ``budget``; always once 32 tokens would not
    hold another chunk): the request = [tokens kept on the device since the last offload, the first
    being the cloud's last correction | gamma drafts]; otherwise it keeps the drafts (they count as
    generated and ride along as uncached tokens of the next offload) and drafts again;
  - a verification accepts a leading run of the drafts, each with probability ``p_match`` (capped
    geometric, Sec. 5), plus the correction token; latency of the request = cloud completion time -
    chunk event time + 2 rtt;
  - the session ends after ``out_tokens`` generated tokens.
"""
from __future__ import annotations

import heapq
import math
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence

from . import rng

S_ARRIVE, S_PROMPT, S_OFFLOAD, S_ACCEPT, S_TOKENS = 101, 102, 103, 104, 105


@dataclass
class ArrivalConfig:
    budget: float                 # probability that a drafted chunk is offloaded
    gamma: int = 4                # drafts per chunk (the paper's default draft length)
    device_s: float = 0.025       # device time per drafted token
    rtt: float = 0.010            # one-way network delay
    out_tokens: int = 128         # tokens a session generates
    p_match: float = 0.7          # probability that a draft is accepted
    prompt_lo: int = 256
    prompt_hi: int = 2048
    vocab: int = 32000
    max_sessions: int = 64        # arrivals beyond this many live sessions are dropped
    max_chunk: int = 32
    seed: int = 0


def poisson_arrivals(rate: float, horizon: float, seed: int) -> List[float]:
    """Arrival times of a Poisson stream of `rate` per second on [0, horizon)."""
    out, t, i = [], 0.0, 0
    key = rng.stream_key(seed, S_ARRIVE)
    while True:
        u = float(rng.uniform01(key, i, 1)[0])
        t += -math.log(1.0 - u) / rate
        i += 1
        if t >= horizon:
            return out
        out.append(t)


@dataclass
class ArrivalResult:
    latencies: List[float] = field(default_factory=list)      # one per verification request, in completion order
    sessions_done: int = 0
    sessions_dropped: int = 0
    iterations: Dict[str, int] = field(default_factory=lambda: {"prefill": 0, "verify": 0})
    busy: float = 0.0
    end: float = 0.0

    def summary(self) -> Dict[str, float]:
        lat = sorted(self.latencies)
        return {"verify_requests": len(lat), "sessions_done": self.sessions_done, "sessions_dropped": self.sessions_dropped,
                "verify_latency_ms_mean": 1e3 * sum(lat) / max(1, len(lat)),
                "verify_latency_ms_p95": 1e3 * lat[int(0.95 * (len(lat) - 1))] if lat else None,
                "gpu_busy_fraction": self.busy / max(self.end, 1e-9), "virtual_seconds": self.end,
                "iterations": dict(self.iterations)}


def simulate(sched, execute: Callable[[dict], tuple], cfg: ArrivalConfig, arrivals: Sequence[float],
             prompt_lens: Optional[Sequence[int]] = None, stop_after: Optional[float] = None) -> ArrivalResult:
    """Run the sessions that arrive at `arrivals` to completion (or until virtual time `stop_after`)."""
    res = ArrivalResult()
    ev: list = []                                   # (time, seq, kind, session)
    seq = 0
    for sid, t in enumerate(arrivals):
        heapq.heappush(ev, (float(t), seq, "arrive", sid)); seq += 1
    sess: Dict[int, dict] = {}
    submitted: Dict[int, float] = {}
    now = 0.0
    k_prompt, k_tok = rng.stream_key(cfg.seed, S_PROMPT), rng.stream_key(cfg.seed, S_TOKENS)

    def draw(stream: int, sid: int, n: int) -> float:
        return float(rng.uniform01(rng.stream_key(cfg.seed, stream, sid), n, 1)[0])

    def tokens(sid: int, start: int, n: int) -> List[int]:
        return rng.randint(rng.stream_key(cfg.seed, S_TOKENS, sid), start, n, 0, cfg.vocab - 1).tolist() if n > 0 else []

    def next_chunk(sid: int, at: float) -> None:
        nonlocal seq
        heapq.heappush(ev, (at, seq, "chunk", sid)); seq += 1

    while True:
        while ev and ev[0][0] <= now:
            t_ev, _, kind, sid = heapq.heappop(ev)
            if kind == "arrive":
                if len(sess) >= cfg.max_sessions:
                    res.sessions_dropped += 1
                    continue
                n = int(prompt_lens[sid]) if prompt_lens is not None else \
                    int(rng.randint(k_prompt, sid, 1, cfg.prompt_lo, cfg.prompt_hi)[0])
                sess[sid] = {"gen": 0, "pend": [], "chunks": 0, "used": n}
                sched.add_request(sid, tokens(sid, 0, n))
            elif sid in sess:                       # the device's next chunk has reached the cloud
                s = sess[sid]
                drafts = tokens(sid, s["used"], cfg.gamma)
                s["used"] += cfg.gamma
                s["chunks"] += 1
                must = len(s["pend"]) + 2 * cfg.gamma > cfg.max_chunk
                if must or draw(S_OFFLOAD, sid, s["chunks"]) < cfg.budget:
                    sched.add_verify(sid, s["pend"] + drafts, len(s["pend"]))
                    submitted[sid] = t_ev
                else:                               # kept on the device: accepted locally, cached at the next offload
                    s["pend"] += drafts
                    s["gen"] += cfg.gamma
                    if s["gen"] >= cfg.out_tokens:
                        sched.finish(sid); del sess[sid]; res.sessions_done += 1
                    else:
                        next_chunk(sid, t_ev + cfg.gamma * cfg.device_s)
        b = sched.peek()
        if b["kind"] == "idle":
            sched.commit()
            if not ev:
                break
            now = max(now, ev[0][0])
            if stop_after is not None and now > stop_after:
                break
            continue
        dt, cor = execute(b)
        now += dt
        res.busy += dt
        res.iterations[b["kind"]] += 1
        offs = [int(x) for x in b["chunk_offsets"]]
        if b["kind"] == "verify":                   # accepted drafts: capped geometric
            acc = []
            for i in range(b["n_req"]):
                sid = int(b["req_ids"][i])
                g = offs[i + 1] - offs[i] - int(b["n_uncached"][i])
                k = 0
                while k < g and draw(S_ACCEPT, sid, sess[sid]["chunks"] * 64 + k) < cfg.p_match:
                    k += 1
                acc.append(k)
            out = sched.commit(acc, cor)
        else:
            out = sched.commit([0] * b["n_req"], cor)
        for x in out:
            sid = x["req_id"]
            if sid not in sess or not x["prompt_done"]:
                continue
            s = sess[sid]
            if x["kind"] == 2:
                res.latencies.append(now - submitted.pop(sid) + 2 * cfg.rtt)
                s["gen"] += x["accept_len"] + 1
            s["pend"] = [x["correction_token"]]
            if s["gen"] >= cfg.out_tokens:
                sched.finish(sid); del sess[sid]; res.sessions_done += 1
            else:
                next_chunk(sid, now + 2 * cfg.rtt + cfg.gamma * cfg.device_s)
        if stop_after is not None and now > stop_after:
            break
    for sid in list(sess):
        sched.finish(sid)
    sched.peek(); sched.commit()
    res.end = now
    return res
