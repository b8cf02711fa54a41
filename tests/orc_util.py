"""Helpers that drive the CPU oracle in tests (prefill in chunks, small models)."""
from __future__ import annotations

import numpy as np
import torch

from oracle import Oracle
from workloads import gen
from workloads.configs import ModelShape

PIN = ModelShape("pin", 2, 64, 4, 2, 16, 96, 50)     # very small: brute force is instant
PIN1 = ModelShape("pin1", 1, 32, 2, 1, 8, 48, 37)


def model(shape, seed=0):
    glob = gen.gen_globals(shape, seed)
    layers = [gen.gen_layer(shape, seed, l) for l in range(shape.n_layers)]
    return glob, layers


def prefill(orc: Oracle, glob, layers, pools, page_table, tokens, start=0, step=16):
    """Feed tokens[start:] through the oracle in chunks of <= step with u = n (no drafts)."""
    p = start
    res = None
    while p < len(tokens):
        c = list(tokens[p:p + step])
        res = orc.forward_chunk(glob, lambda l: layers[l], pools, page_table, p, c, u=len(c))
        p += len(c)
    return res


def tokens_for(shape, n, seed=123):
    g = np.random.default_rng(seed)
    return g.integers(0, shape.vocab, size=n).astype(np.int32)
