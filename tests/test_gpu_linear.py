"""tcgen05 GEMM (through the C ABI test hook) against the CPU oracle's linear map."""
import numpy as np
import pytest
import torch

from oracle import Oracle
from workloads import rng
from workloads.configs import TINY

pytestmark = pytest.mark.gpu


def _case(T, N, K, seed):
    key = rng.stream_key(seed, 99)
    x = rng.normal_f32(key, 0, T * K, 1.0).view(T, K).to(torch.float16)
    w = rng.normal_f32(key, T * K, N * K, 0.05).view(N, K).to(torch.bfloat16)
    return x, w


@pytest.mark.parametrize("T,N,K", [
    (16, 128, 64),        # one tile, one k-block
    (16, 128, 256),       # several k-blocks, fewer than the ring
    (32, 256, 1024),      # ring wraps (16 k-blocks)
    (50, 300, 192),       # ragged tokens and features
    (129, 384, 2048),     # few feature tiles: five token tiles of 32 columns, the last with one token
    (544, 640, 4096),     # seventeen token tiles of 32 columns, 64 k-blocks
    (544, 28672, 512),    # many feature tiles: three token tiles of 192 columns, pair items in full waves + single tiles
    (544, 28672, 4096),   # 336 pair tiles on 148 SMs: two full waves, the other 40 cut along K into 3 parts each
    (300, 38144, 1024),   # 298 pair tiles: two left over, each cut in two
    (921, 6144, 512),     # 96 pair tiles, 192 single tiles on 148 SMs: 44 whole pair tiles + 104 single tiles in one wave
    (200, 25600, 256),    # 100 pair tiles: 52 whole + 96 single tiles
    (137, 4096, 512),     # token tiles of 48 columns: 3 x 48 covers 137, no fourth tile
    (300, 1024, 320),     # ten token tiles of 32 columns, the last with 12 tokens
    (16, 128, 688),       # K tail: 688 = 10.75 k-blocks (zero-filled by TMA)
    (257, 128, 128),      # two token tiles, the second nearly empty
    (1, 128, 64),         # a single token
])
def test_linear_matches_oracle(T, N, K):
    import paper_2511_07423_b200 as syn
    x, w = _case(T, N, K, T + N + K)
    y = syn.syn_op_linear(x.cuda(), w.cuda()).cpu().double().numpy()
    ref = Oracle(TINY).linear(x.double().numpy(), w)
    scale = np.abs(ref).max()
    err = np.abs(y - ref).max()
    assert err <= 2e-5 * scale * max(1.0, (K / 256) ** 0.5), (err, scale)


@pytest.mark.parametrize("T,N,K,sched", [
    (544, 4096, 4096, "resid"),    # the 8B o projection: 48 pair tiles, K shared by three CTAs each (reduce-scatter)
    (544, 4096, 14336, "resid"),   # its down projection: 224 k-blocks in three parts of 75, 75, 74
    (544, 6144, 4096, "qkv"),      # its qkv projection: 72 pair tiles, K shared by two CTAs each
    (129, 2048, 2048, "resid"),    # the 1B o projection: 8 tiles, K shared by eight CTAs, nine chunks among them
    (144, 2048, 8192, "resid"),    # the 1B down projection
    (300, 5120, 1024, "resid"),    # 40 tiles of 160 tokens (the last with 140), three parts
    (50, 300, 1024, "resid"),      # ragged tokens and features, four parts of four k-blocks
    (17, 256, 2048, "resid"),      # two chunks among eight CTAs: most of them keep no column
    (1194, 5120, 1024, "resid"),   # 100 pair tiles: K not shared, seven narrower token tiles instead
    (544, 28672, 4096, "swiglu"),  # schedule of the gate/up projection
    (300, 38144, 1024, "lmhead"),
    # the CTA-pair kernel (clusters of two share a token tile)
    (544, 28672, 4096, "pair_quad"),       # 56 x 3 items of 512 features on 74 clusters: 2.3 waves
    (544, 6144, 4096, "pair_duo"),         # 24 x 3 items of 256 features, two k-interleaved accumulators per CTA
    (544, 4096, 4096, "pair_duo"),         # 48 clusters
    (544, 4096, 14336, "pair_quad_resid"), # 24 items, K shared by three clusters each: exchange between CTAs of equal rank
    (300, 1280, 1024, "pair_quad"),        # five feature pairs: the last cluster's second pair is all padding; 160-token tiles
    (1194, 7168, 5120, "pair_quad"),       # five token tiles of 240, the last with 234 tokens
    (921, 4096, 512, "pair_duo_resid"),    # 64 items, no room to share K
    (257, 640, 2048, "pair_duo_resid"),    # token tiles of 144 and 113; 6 items, K shared by four clusters each
    (40, 512, 256, "pair_quad"),           # one item, a 48-token tile: halves of 24 rows
])
def test_every_schedule_of_the_step_gives_the_plain_product(T, N, K, sched):
    """The work decompositions the step uses for its projections (K shared between CTAs with a
    reduce-scatter of the accumulators, leftover tiles cut along K, mixed waves), each run with the
    plain store epilogue and held to the same tolerance as the plain schedule."""
    import paper_2511_07423_b200 as syn
    x, w = _case(T, N, K, T + N + K + 1)
    xc, wc = x.cuda(), w.cuda()
    y = syn.syn_op_linear(xc, wc, schedule_as=sched)
    y2 = syn.syn_op_linear(xc, wc, schedule_as=sched, reuse_pack=True)
    assert torch.equal(y, y2)                      # fixed summation order, counters back at zero
    ref = Oracle(TINY).linear(x.double().numpy(), w)
    y = y.cpu().double().numpy()
    scale = np.abs(ref).max()
    err = np.abs(y - ref).max()
    assert err <= 2e-5 * scale * max(1.0, (K / 256) ** 0.5), (err, scale)


def test_a_new_matrix_at_an_old_address_is_packed_again():
    import paper_2511_07423_b200 as syn
    x, w = _case(32, 256, 256, 5)
    xc, wc = x.cuda(), w.cuda()
    y1 = syn.syn_op_linear(xc, wc)
    wc.mul_(2)                                     # same address, same shape, new contents
    y2 = syn.syn_op_linear(xc, wc)
    assert torch.allclose(y2, 2 * y1)


@pytest.mark.parametrize("T,N,K,sched", [
    (129, 2048, 2048, "resid"),              # one-CTA kernel: tile 0's eight CTAs wait for 128 arrivals
    (544, 4096, 14336, "pair_quad_resid"),   # CTA-pair kernel: the rank-0 CTAs of tile 0's three clusters wait for 48
])
def test_a_wait_that_cannot_end_runs_out_and_the_next_call_works(T, N, K, sched):
    """SYN_E_DEVICE_TIMEOUT end to end: an arrival counter of the reduce-scatter is set so far below
    zero that the count its readers wait for cannot be reached; with the waits' limit shortened to a
    fraction of a millisecond they give up, the kernel ends normally, the call reports the timeout and
    clears the counters, and the same call then succeeds with the right result."""
    import paper_2511_07423_b200 as syn
    x, w = _case(T, N, K, 77)
    xc, wc = x.cuda(), w.cuda()
    good = syn.syn_op_linear(xc, wc, schedule_as=sched)
    try:
        syn.debug_set_spin_limit(400_000)
        syn.debug_linear_counter(0, -1_000_000)
        with pytest.raises(syn.SynError) as ei:
            syn.syn_op_linear(xc, wc, schedule_as=sched, reuse_pack=True)
        assert ei.value.code == -11
    finally:
        syn.debug_set_spin_limit(0)
    again = syn.syn_op_linear(xc, wc, schedule_as=sched, reuse_pack=True)
    assert torch.equal(again, good)
