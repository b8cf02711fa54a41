"""Plain restatement of the verification-aware scheduler (paper Sec. 4.5, Algorithm 1).

TEST INFRASTRUCTURE ONLY: imported by tests, never by the product package; shares no code with the
C++ scheduler.  It keeps the algorithm's own objects and order:

    every iteration:
        B_prefill <- all waiting prefill requests            (arrival order)
        if B_prefill is not empty: execute_prefill(B_prefill); end of the iteration
        otherwise B_verify <- all waiting verification requests, L_uncached <- their u
                  if B_verify is not empty: execute_partialprefill(B_verify, L_uncached)
        B <- remove_completed(B)

plus what the section's text adds: a prompt is fed in fixed chunks of 32 tokens ("chunked partial
prefill"), one chunk of every waiting prompt per prefill iteration, all of its tokens uncached.

Two things the paper leaves to its serving engine are stated here as the rules both sides follow:
a token budget per iteration (requests are taken in arrival order until the first one that does
not fit), and page availability (a request needs ceil((ctx + n) / page) pages in total; one that
cannot get them is passed over for this iteration; if prefill requests wait but none can be
served, the iteration falls through to verification).  After a verification the cached length
grows by u + accept_len (Sec. 3.4: accepted tokens stay, rejected drafts are overwritten).
A completion is an outside event here; it takes effect at the next iteration boundary
(remove_completed runs at the end of an iteration, as in Algorithm 1, and again before the next
one is formed, for completions reported in between).
Pages are only counted here, never numbered: which physical page a request gets is not part of
the algorithm.

Pins: tests/test_scheduler_host.py checks this module against a hand-worked trace
(tests/golden/scheduler_trace.txt) before it is used to judge the C++ scheduler.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

CHUNK = 32   # fixed chunk length of chunked partial prefill (Sec. 4.5)


@dataclass
class _Req:
    rid: int
    prompt: List[int]
    done_prompt: int = 0
    ctx: int = 0
    pages: int = 0
    chunk: Optional[List[int]] = None
    u: int = 0
    finished: bool = False

    @property
    def prefilling(self) -> bool:
        return self.done_prompt < len(self.prompt)


@dataclass
class Iteration:
    kind: str                                   # "idle" | "prefill" | "verify"
    entries: List[Tuple[int, List[int], int, int]] = field(default_factory=list)   # (id, tokens, u, ctx before)


class SchedulerOracle:
    def __init__(self, n_pages: int, page_size: int = 16, max_batch_tokens: int = 2048):
        self.free = n_pages
        self.P = page_size
        self.budget = max_batch_tokens
        self.reqs: Dict[int, _Req] = {}
        self.prefill_q: List[int] = []
        self.verify_q: List[int] = []
        self.current: Optional[Iteration] = None

    # ---- arrivals
    def add_request(self, rid: int, prompt: List[int]) -> None:
        assert rid not in self.reqs and len(prompt) >= 1
        self.reqs[rid] = _Req(rid, list(prompt))
        self.prefill_q.append(rid)

    def add_verify(self, rid: int, tokens: List[int], u: int = 1) -> None:
        r = self.reqs[rid]
        assert not r.finished and not r.prefilling and r.chunk is None and 1 <= u <= len(tokens) <= CHUNK
        r.chunk, r.u = list(tokens), u
        self.verify_q.append(rid)

    def finish(self, rid: int) -> None:
        self.reqs[rid].finished = True

    # ---- one iteration
    def _take(self, queue: List[int], prefill: bool) -> List[Tuple[int, List[int], int, int]]:
        out, total, full = [], 0, False
        for rid in queue:
            r = self.reqs.get(rid)
            if r is None or r.finished:
                continue
            toks = r.prompt[r.done_prompt:r.done_prompt + CHUNK] if prefill else r.chunk
            n = len(toks)
            if full or total + n > self.budget:
                full = True
                continue
            need = -(-(r.ctx + n) // self.P) - r.pages
            if need > self.free:
                continue
            if need > 0:
                self.free -= need
                r.pages += need
            out.append((rid, list(toks), n if prefill else r.u, r.ctx))
            total += n
        return out

    def _remove_completed(self) -> None:
        for rid in [rid for rid, r in self.reqs.items() if r.finished]:
            self.free += self.reqs[rid].pages
            del self.reqs[rid]
        self.prefill_q = [rid for rid in self.prefill_q if rid in self.reqs]
        self.verify_q = [rid for rid in self.verify_q if rid in self.reqs]

    def next_iteration(self) -> Iteration:
        assert self.current is None
        self._remove_completed()   # completions reported since the last iteration ended
        entries = self._take(self.prefill_q, True)
        kind = "prefill"
        if not entries:
            entries = self._take(self.verify_q, False)
            kind = "verify"
        self.current = Iteration(kind if entries else "idle", entries)
        return self.current

    def complete(self, accept_len: Optional[List[int]] = None) -> None:
        it = self.current
        assert it is not None
        for i, (rid, toks, u, _) in enumerate(it.entries):
            r = self.reqs[rid]
            if it.kind == "prefill":
                r.ctx += len(toks)
                r.done_prompt += len(toks)
            else:
                assert 0 <= accept_len[i] <= len(toks) - u
                r.ctx += u + accept_len[i]
                r.chunk = None
        self.prefill_q = [rid for rid in self.prefill_q if rid in self.reqs and self.reqs[rid].prefilling]
        self.verify_q = [rid for rid in self.verify_q if rid in self.reqs and self.reqs[rid].chunk is not None]
        self._remove_completed()
        self.current = None
