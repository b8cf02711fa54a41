"""The verification-aware scheduler (paper Sec. 4.5, Algorithm 1) on the CPU: the plain restatement
in oracle/scheduler.py is pinned to a hand-worked trace, then the C++ scheduler (policy only: peek /
commit, no device) is compared with both, on the trace and on seeded random arrival scripts."""
import os
import random

import pytest
import torch

import paper_2511_07423_b200 as syn
from oracle.scheduler import SchedulerOracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "scheduler_trace.txt")


class OracleSide:
    def __init__(self, n_pages, page, budget):
        self.s = SchedulerOracle(n_pages, page, budget)

    def add(self, rid, prompt): self.s.add_request(rid, prompt)
    def verify(self, rid, toks, u): self.s.add_verify(rid, toks, u)
    def finish(self, rid): self.s.finish(rid)

    def iterate(self):
        it = self.s.next_iteration()
        return it.kind, [(rid, tuple(t), u, ctx) for rid, t, u, ctx in it.entries]

    def complete(self, accept): self.s.complete(accept)
    def free(self): return self.s.free


class LibrarySide:
    def __init__(self, n_pages, page, budget):
        self.s = syn.Scheduler(None, n_pages=n_pages, page_size=page, max_batch_tokens=budget)
        self.n_pages, self.P = n_pages, page
        self.live_pages = {}

    def add(self, rid, prompt): self.s.add_request(rid, prompt)
    def verify(self, rid, toks, u): self.s.add_verify(rid, toks, u)
    def finish(self, rid): self.s.finish(rid)

    def iterate(self):
        b = self.s.peek()
        self.batch = b
        if b["kind"] == "idle":
            return "idle", []
        offs = b["chunk_offsets"].tolist()
        out = []
        for i, rid in enumerate(b["req_ids"]):
            toks = tuple(b["chunk_tokens"][offs[i]:offs[i + 1]].tolist())
            ctx, u = int(b["ctx_lens"][i]), int(b["n_uncached"][i])
            out.append((rid, toks, u, ctx))
            # the page table covers every position of the request, with valid page ids
            used = -(-(ctx + len(toks)) // self.P)
            row = b["page_tables"][i].tolist()
            assert all(0 <= p < self.n_pages for p in row[:used]) and all(p == -1 for p in row[used:])
            # logical pages never move once assigned
            old = self.live_pages.get(rid, [])
            assert row[:min(len(old), used)] == old[:min(len(old), used)]
            self.live_pages[rid] = row[:used] + old[used:]
        return b["kind"], out

    def complete(self, accept):
        b = self.batch
        if b["kind"] == "idle":
            res = self.s.commit()
            assert res == []
        else:
            n = b["n_req"]
            cor = [1000 + i for i in range(n)]
            res = self.s.commit(accept if accept is not None else [0] * n, cor)
            offs = b["chunk_offsets"].tolist()
            for i, r in enumerate(res):
                nt = offs[i + 1] - offs[i]
                a = accept[i] if b["kind"] == "verify" else 0
                assert r["req_id"] == b["req_ids"][i] and r["n_tokens"] == nt and r["correction_token"] == cor[i]
                assert r["accept_len"] == a
                grow = nt if b["kind"] == "prefill" else int(b["n_uncached"][i]) + a
                assert r["ctx_len"] == int(b["ctx_lens"][i]) + grow
        st = self.s.stats()
        # no page belongs to two live requests; free + held = pool
        live = {rid: p for rid, p in self.live_pages.items() if rid not in self.finished_ids()}
        held = [p for pages in live.values() for p in pages]
        assert len(held) == len(set(held))
        assert st.free_pages + len(held) == self.n_pages
        self.live_pages = live

    def finished_ids(self):
        return getattr(self, "_finished", set())

    def mark_finished(self, rid):
        self._finished = self.finished_ids() | {rid}

    def free(self): return self.s.stats().free_pages


def _play_golden(side_cls):
    side = None
    for raw in open(GOLDEN):
        line = raw.split("#")[0].split()
        if not line:
            continue
        op = line[0]
        if op == "pool":
            side = side_cls(int(line[1]), int(line[2]), int(line[3]))
        elif op == "add":
            side.add(int(line[1]), list(range(int(line[2]))))
        elif op == "verify":
            side.verify(int(line[1]), [7] * int(line[2]), int(line[3]))
        elif op == "finish":
            side.finish(int(line[1]))
            if hasattr(side, "mark_finished"):
                side.mark_finished(int(line[1]))
        elif op == "free":
            assert side.free() == int(line[1]), raw
        elif op == "expect":
            kind, entries = side.iterate()
            assert kind == line[1], raw
            spec = line[2:]
            accept = None
            if "accept" in spec:
                k = spec.index("accept")
                accept = [int(x) for x in spec[k + 1:]]
                spec = spec[:k]
            want = [tuple(int(x) for x in e.split(":")) for e in spec]
            got = [(rid, len(t), u, ctx) for rid, t, u, ctx in entries]
            assert got == want, raw
            side.complete(accept)
        else:
            raise AssertionError(raw)


def test_oracle_follows_the_hand_worked_trace():
    _play_golden(OracleSide)


def test_library_follows_the_hand_worked_trace():
    _play_golden(LibrarySide)


def test_prefill_chunks_carry_the_prompt_in_order_and_are_all_uncached():
    for cls in (OracleSide, LibrarySide):
        side = cls(40, 16, 256)
        prompt = [(37 * i + 5) % 1000 for i in range(75)]
        side.add(3, prompt)
        seen = []
        while True:
            kind, entries = side.iterate()
            if kind == "idle":
                side.complete(None)
                break
            assert kind == "prefill" and len(entries) == 1
            rid, toks, u, ctx = entries[0]
            assert u == len(toks) <= 32 and ctx == len(seen)
            seen += list(toks)
            side.complete(None)
        assert seen == prompt


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_random_arrival_scripts_give_the_same_iterations_as_the_oracle(seed):
    rnd = random.Random(seed)
    n_pages, P, budget = rnd.choice([(60, 16, 64), (200, 16, 128), (35, 16, 96)])
    a, b = OracleSide(n_pages, P, budget), LibrarySide(n_pages, P, budget)
    next_id, active, waiting_chunk, prefilling = 0, set(), set(), set()
    n_iter = {"idle": 0, "prefill": 0, "verify": 0}
    for step in range(300):
        # arrivals before the iteration
        for _ in range(rnd.choice([0, 0, 1, 1, 2])):
            if len(active) + len(prefilling) < 8:
                prompt = [rnd.randrange(1000) for _ in range(rnd.randint(1, 90))]
                for s in (a, b):
                    s.add(next_id, prompt)
                prefilling.add(next_id)
                next_id += 1
        for rid in sorted(active - waiting_chunk):
            r = rnd.random()
            if r < 0.5:
                n = rnd.randint(1, 32)
                u = rnd.randint(1, n)
                toks = [rnd.randrange(1000) for _ in range(n)]
                for s in (a, b):
                    s.verify(rid, toks, u)
                waiting_chunk.add(rid)
            elif r < 0.58:
                for s in (a, b):
                    s.finish(rid)
                b.mark_finished(rid)
                active.discard(rid)
        ka, ea = a.iterate()
        try:
            kb, eb = b.iterate()
        except syn.SynError as e:
            # the library reports "work waits but nothing can be served"; the restatement calls it idle
            assert e.code == -5 and ka == "idle"
            a.complete(None)
            victim = sorted(active | prefilling)[0]   # make room
            for s in (a, b):
                s.finish(victim)
            b.mark_finished(victim)
            active.discard(victim); prefilling.discard(victim); waiting_chunk.discard(victim)
            continue
        assert (ka, ea) == (kb, eb), (seed, step)
        n_iter[ka] += 1
        accept = None
        if ka == "verify":
            accept = [rnd.randint(0, len(t) - u) for _, t, u, _ in ea]
            for rid, _, _, _ in ea:
                waiting_chunk.discard(rid)
        a.complete(accept)
        b.complete(accept)
        assert a.free() == b.free()
        # requests whose prompt is fully cached become active
        for rid in list(prefilling):
            r = a.s.reqs.get(rid)
            if r is not None and not r.prefilling:
                prefilling.discard(rid)
                active.add(rid)
    assert n_iter["prefill"] > 20 and n_iter["verify"] > 20


def test_error_codes_and_states():
    s = syn.Scheduler(None, n_pages=4, max_batch_tokens=64)
    with pytest.raises(syn.SynError) as e:
        syn.Scheduler(None, n_pages=4, max_batch_tokens=8)      # below one chunk
    assert e.value.code == -1
    s.add_request(1, [1, 2, 3])
    for fn, code in ((lambda: s.add_request(1, [4]), -21), (lambda: s.add_verify(2, [1]), -20),
                     (lambda: s.add_verify(1, [1]), -22),                      # still prefilling
                     (lambda: s.add_verify(1, [1] * 33), -2), (lambda: s.add_verify(1, [1, 2], 3), -3),
                     (lambda: s.finish(5), -20), (lambda: s.commit([0], [0]), -23)):
        with pytest.raises(syn.SynError) as e:
            fn()
        assert e.value.code == code
    b = s.peek()
    assert b["kind"] == "prefill" and s.peek()["chunk_tokens"].tolist() == [1, 2, 3]   # a second peek: same batch
    s.commit([0], [9])
    s.add_verify(1, [9, 4, 4], 1)
    with pytest.raises(syn.SynError) as e:
        s.add_verify(1, [9], 1)                                  # one chunk may wait
    assert e.value.code == -22
    s.peek()
    with pytest.raises(syn.SynError) as e:
        s.commit([3], [0])                                       # more accepted than drafts
    assert e.value.code == -1
    s.commit([2], [0])
    # a prompt the pool cannot hold: reported, and served once pages are free again
    s.add_request(2, list(range(60)))                            # 4 pages, 3 free
    s.peek(); s.commit([0], [0])                                 # first chunk of 32: 2 pages
    with pytest.raises(syn.SynError) as e:
        s.peek()                                                 # needs 2 more, 1 free
    assert e.value.code == -5
    s.finish(1)
    with pytest.raises(syn.SynError) as e:
        s.step()                                                 # no model behind this scheduler
    assert e.value.code == -1
    b = s.peek()
    assert b["kind"] == "prefill" and b["n_tokens"] == 28
    assert s.stats().live_requests == 1
