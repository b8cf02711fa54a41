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
    x = rng.normal_f32(key, 0, T * K, 1.0).view(T, K).to(torch.bfloat16)
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
