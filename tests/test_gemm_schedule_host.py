"""The projection kernel's static schedule, checked on the CPU through syn_gemm_plan_host /
syn_gemm_work_host (the code the kernel's three roles run to find their work): for the projections of
every configuration and for a sweep of awkward sizes, every (128-feature tile, token tile) of the output
is produced exactly once over the whole K, every token tile holds a token (an empty one would issue an
MMA of width 0), and the parts of a K-split leftover tile sit on different CTAs with the helpers first."""
import pytest

import paper_2511_07423_b200 as syn
from workloads import gen
from workloads.configs import CONFIGS, MINI_1B, MINI_8B


def _check(T, N, K, epilogue, n_sm=148):
    p = syn.gemm_plan_host(T, N, K, epilogue, n_sm)
    n_tt, TN, nkb = p["n_tt"], p["TN"], p["num_kb"]
    assert 16 <= TN <= 256 and TN % 16 == 0
    assert (n_tt - 1) * TN < T <= n_tt * TN                      # every token tile holds a token
    assert nkb == -(-K // 64) and p["n_pairs"] == -(-N // 256)
    assert 1 <= p["n_cta"] <= max(n_sm, p["n_pairs"] * n_tt * p["splits"])
    if p["splits"] == 1:
        assert p["n_cta"] <= n_sm
    cover = {}        # (pair, 128-feature tile, token tile) -> list of (kb0, kb1, split, role, cta, item index)
    for cta in range(p["n_cta"]):
        i = 0
        while True:
            w = syn.gemm_work_host(T, N, K, epilogue, cta, i, n_sm)
            if w is None:
                break
            assert 0 <= w["pair"] < p["n_pairs"] and 0 <= w["tt"] < n_tt
            assert 0 <= w["mt_lo"] < w["mt_hi"] <= 2 and 0 <= w["kb0"] < w["kb1"] <= nkb
            for mt in range(w["mt_lo"], w["mt_hi"]):
                cover.setdefault((w["pair"], mt, w["tt"]), []).append((w["kb0"], w["kb1"], w["split"], w["role"], cta, i))
            i += 1
            assert i < 5000
    assert len(cover) == p["n_pairs"] * 2 * n_tt
    for key, parts in cover.items():
        parts.sort()
        assert parts[0][0] == 0 and parts[-1][1] == nkb
        for a, b in zip(parts, parts[1:]):
            assert a[1] == b[0]                                     # the k ranges tile [0, nkb) without gap or overlap
        if p["splits"] > 1:                                         # K shared by neighbouring CTAs, parts numbered in order
            assert epilogue in ("resid", "qkv") and [x[2] for x in parts] == list(range(len(parts)))
            ctas = [x[4] for x in parts]
            assert ctas == list(range(ctas[0], ctas[0] + len(parts))) and ctas[0] % p["splits"] == 0
            assert p["n_cta"] <= n_sm                                   # all of them run at the same time
        elif len(parts) > 1:                                        # a leftover tile cut along K
            assert p["ksplit"] == len(parts) and epilogue != "resid"
            assert [x[3] for x in parts] == [1] * (len(parts) - 1) + [2]
            assert len({x[4] for x in parts}) == len(parts)         # helpers and the owner are different CTAs
            assert all(x[5] == 0 for x in parts[:-1])               # helper parts are their CTAs' first items
            assert parts[-1][1] - parts[-1][0] <= parts[0][1] - parts[0][0]   # the owner's k range is the shortest
        else:
            assert parts[0][3] == 0
    return p


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5, 6])
def test_projections_of_the_configurations(cfg):
    wl = CONFIGS[cfg]
    s = wl.shape
    T = gen.gen_batch(wl).n_tokens
    f_pad = -(-s.d_ffn // 64) * 64
    for N, K, epi in ((s.q_dim + 2 * s.kv_dim, s.d_model, "qkv"), (s.d_model, s.q_dim, "resid"),
                      (2 * f_pad, s.d_model, "swiglu"), (s.d_model, f_pad, "resid"), (s.vocab, s.d_model, "lmhead")):
        _check(T, N, K, epi)


def test_the_launch_rules_show_up_where_they_should():
    # gate/up of the 8B shape at 544 tokens: 336 pair tiles, 40 left after two waves, cut in three
    p = _check(544, 28672, 4096, "swiglu")
    assert (p["n_tt"], p["TN"], p["pair_mode"], p["ksplit"]) == (3, 192, 1, 3)
    # its QKV projection at 921 tokens: 96 pair tiles = 192 single tiles on 148 SMs -> one mixed wave
    assert _check(921, 6144, 4096, "qkv")["pair_mode"] == 2
    # the 1B shape's QKV projection at 129 tokens: narrow token tiles put 120 CTAs to work instead of 24
    p = _check(129, 3072, 2048, "qkv")
    assert p["TN"] == 32 and p["n_cta"] == 120
    # the 32B shape's down projection: 100 pair tiles cannot split K, seven token tiles fill the machine
    p = _check(1194, 5120, 27648, "resid")
    assert p["n_tt"] == 7 and p["splits"] == 1 and p["n_cta"] == 140
    # the 8B shape's o projection at 544 tokens: 48 pair tiles, K shared by three CTAs each
    assert _check(544, 4096, 4096, "resid")["splits"] == 3
    # its QKV projection at 544 tokens: 72 pair tiles, K shared by two CTAs each instead of 144 single tiles
    p = _check(544, 6144, 4096, "qkv")
    assert (p["splits"], p["n_cta"], p["TN"]) == (2, 144, 192)


@pytest.mark.parametrize("epilogue", ["plain", "qkv", "resid", "swiglu", "lmhead"])
def test_sweep_of_awkward_sizes(epilogue):
    sizes = [(1, 128, 64), (16, 128, 688), (17, 384, 2048), (33, 256, 128), (129, 3072, 2048), (137, 4096, 512),
             (255, 640, 320), (256, 25600, 256), (257, 128, 128), (300, 38144, 1024), (544, 640, 4096), (921, 6144, 512),
             (1194, 7168, 5120), (2048, 4096, 4096), (2049, 152064, 5120), (97, 18944, 1536)]
    for T, N, K in sizes:
        _check(T, N, K, epilogue)
    for n_sm in (1, 7, 132, 148, 160):
        _check(544, 28672, 4096, epilogue, n_sm)
        _check(129, 3072, 2048, epilogue, n_sm)


# ------------------------------------------------------------------------------------------ the CTA-pair kernel

def _check2(T, N, K, epilogue, force="auto", n_sm=148):
    p = syn.gemm2_plan_host(T, N, K, epilogue, force, n_sm)
    if p["kind"] == 0:
        return p
    n_tt, TN, nkb, n_cl = p["n_tt"], p["TN"], p["num_kb"], p["n_clusters"]
    per = 2 if p["kind"] == 1 else 1                       # feature pairs of 256 per group
    assert 16 <= TN <= 256 and TN % 16 == 0 and (n_tt - 1) * TN < T <= n_tt * TN
    assert p["n_groups"] == -(-(-(-N // 256)) // per) and 1 <= n_cl <= n_sm // 2
    cover = {}
    for cl in range(n_cl):
        i = 0
        while True:
            w = syn.gemm2_work_host(T, N, K, epilogue, cl, i, force, n_sm)
            if w is None:
                break
            assert 0 <= w["grp"] < p["n_groups"] and 0 <= w["tt"] < n_tt and 0 <= w["kb0"] < w["kb1"] <= nkb
            assert w["tile"] == w["grp"] * n_tt + w["tt"]
            cover.setdefault(w["tile"], []).append((w["kb0"], w["kb1"], w["split"], w["nsplit"], w["first_cl"], w["counter"], cl, i))
            i += 1
            assert i < 5000
    assert sorted(cover) == list(range(p["n_groups"] * n_tt))          # every tile, once over the whole K
    counters = {}
    for tile, parts in cover.items():
        parts.sort()
        assert parts[0][0] == 0 and parts[-1][1] == nkb
        assert all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
        if len(parts) > 1:                                              # K shared: neighbouring clusters, parts in order,
            S = len(parts)                                              # one counter per tile, all in the same round
            assert [x[2] for x in parts] == list(range(S)) and all(x[3] == S for x in parts)
            assert [x[6] for x in parts] == list(range(parts[0][4], parts[0][4] + S))
            assert len({x[5] for x in parts}) == 1 and len({x[7] for x in parts}) == 1 and 0 <= parts[0][5] < n_sm // 2
            assert min(x[1] - x[0] for x in parts) >= min(8, nkb // S)
            counters.setdefault(parts[0][7], []).append(parts[0][5])
        else:
            assert parts[0][3] == 1
    for rnd, cs in counters.items():
        assert len(set(cs)) == len(cs)                                  # tiles of one round meet on different counters
    return p


def test_pair_schedules_of_the_configurations():
    for cfg in (3, 4, 5, 6):
        wl = CONFIGS[cfg]
        s = wl.shape
        T = gen.gen_batch(wl).n_tokens
        f_pad = -(-s.d_ffn // 64) * 64
        for N, K, epi in ((s.q_dim + 2 * s.kv_dim, s.d_model, "qkv"), (s.d_model, s.q_dim, "resid"),
                          (2 * f_pad, s.d_model, "swiglu"), (s.d_model, f_pad, "resid"), (s.vocab, s.d_model, "lmhead")):
            _check2(T, N, K, epi)
    # fewer than 256 tokens: the one-CTA kernel keeps the projection
    assert syn.gemm2_plan_host(129, 3072, 2048, "qkv")["kind"] == 0
    # configuration 3: gate/up = 168 items of 512 features on 74 clusters, 2.27 waves: left to the one-CTA kernel; taken
    # all the same (forced), the 20 items left over are cut into 4 (14 of them) or 3 parts
    assert syn.gemm2_plan_host(544, 28672, 4096, "swiglu")["kind"] == 0
    p = _check2(544, 28672, 4096, "swiglu", "quad")
    assert (p["kind"], p["n_clusters"], p["rem_base"], p["rem_extra"]) == (1, 74, 3, 14)
    # configuration 4 (921 tokens): 224 items, three full waves and two items over, cut in eight
    p = _check2(921, 28672, 4096, "swiglu")
    assert (p["kind"], p["rem_base"], p["rem_extra"]) == (1, 8, 0)
    # its qkv and o projections: items of 256 features; its down projection: 24 items, K shared by three clusters each
    assert _check2(544, 6144, 4096, "qkv")["kind"] == 2 and _check2(544, 4096, 4096, "resid")["kind"] == 2
    p = _check2(544, 4096, 14336, "resid")
    assert (p["kind"], p["splits"], p["n_clusters"]) == (1, 3, 72)
    # one wave of 512-feature items at least three quarters full (five eighths without a residual epilogue):
    # o and down at 2 048 tokens (64 items), the 32B shape's qkv at 1 194 (70), qkv at 921 (48); the 32B shape's
    # o at 1 194 tokens (50 items, residual epilogue) stays on the one-CTA kernel
    for T, N, K, epi, want in ((2048, 4096, 4096, "resid", (1, 64)), (2048, 4096, 14336, "resid", (1, 64)),
                               (1194, 7168, 5120, "qkv", (1, 70)), (921, 6144, 4096, "qkv", (1, 48))):
        p = _check2(T, N, K, epi)
        assert (p["kind"], p["n_clusters"]) == want and p["splits"] == 1
    assert syn.gemm2_plan_host(1194, 5120, 5120, "resid")["kind"] == 0


@pytest.mark.parametrize("force", ["quad", "duo"])
def test_pair_schedule_sweep(force):
    for T, N, K in [(1, 128, 64), (40, 512, 256), (257, 640, 2048), (300, 1280, 1024), (544, 640, 4096), (921, 6144, 512),
                    (1194, 7168, 5120), (2048, 4096, 4096), (2049, 152064, 5120), (544, 128256, 4096), (300, 38144, 1024)]:
        for epi in ("plain", "resid"):
            _check2(T, N, K, epi, force)
    for n_sm in (2, 7, 132, 148, 160):
        _check2(544, 28672, 4096, "swiglu", force, n_sm)
