"""The benchmark configurations as data: model shapes and request mixes (1-5: verification
batches; 6: chunked partial prefill with 32-token chunks).

Shapes and mixes only; seeds follow the rule "configuration k (1-based) uses seed k-1".
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Tuple


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_base: float = 10000.0
    rms_eps: float = 1e-5
    weight_std: float = 0.02
    gain_std: float = 0.1

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def dense_params(self) -> int:
        """Parameters of the projections streamed once per step (embedding excluded)."""
        per_layer = self.d_model * (self.q_dim + 2 * self.kv_dim) + self.q_dim * self.d_model \
            + 3 * self.d_model * self.d_ffn
        return self.n_layers * per_layer + self.d_model * self.vocab

    def kv_bytes_per_token(self) -> int:
        return 2 * self.kv_dim * 2 * self.n_layers


TINY = ModelShape("tiny", 2, 256, 4, 2, 64, 688, 1024)
SHAPE_1B = ModelShape("1b", 16, 2048, 32, 8, 64, 8192, 32000)
SHAPE_8B = ModelShape("8b", 32, 4096, 32, 8, 128, 14336, 128256)
SHAPE_32B = ModelShape("32b", 64, 5120, 40, 8, 128, 27648, 152064)


@dataclass(frozen=True)
class Workload:
    """One request mix.  ``ctx`` / ``chunk`` are (kind, params) recipes, see workloads.gen."""
    name: str
    shape: ModelShape
    seed: int
    n_req: int
    ctx: Tuple
    chunk: Tuple
    p_match: float
    page_size: int = 16
    real_prefill: bool = False      # context KV produced by prefilling real tokens
    fit_to_pool: bool = False       # scale contexts by a common factor to fit the pool
    n_drafts: Optional[int] = None  # drafts at the end of a chunk; the rest is uncached accepted tokens (None: all but one)


CONFIGS = {
    1: Workload("cfg1-tiny", TINY, 0, 4, ("list", (48, 64, 96, 128)), ("const", 4), 0.7,
                real_prefill=True),
    2: Workload("cfg2-1b", SHAPE_1B, 1, 32, ("uniform", 256, 2048), ("uniform", 1, 8), 0.7),
    3: Workload("cfg3-8b", SHAPE_8B, 2, 64, ("uniform", 512, 4096), ("uniform", 1, 16), 0.6),
    4: Workload("cfg4-8b-scalable", SHAPE_8B, 3, 256, ("loguniform", 128, 8192),
                ("mix", ((0.6, 1, 1), (0.3, 2, 8), (0.1, 9, 16))), 0.65),
    5: Workload("cfg5-32b", SHAPE_32B, 4, 128, ("uniform", 1024, 8192), ("uniform", 1, 16), 0.6,
                fit_to_pool=True),
    # chunked partial prefill: every request feeds a full 32-token chunk, 28 uncached tokens + 4 drafts
    6: Workload("cfg6-8b-chunk32", SHAPE_8B, 5, 64, ("uniform", 512, 4096), ("const", 32), 0.6, n_drafts=4),
}

# Reduced shapes used by tests that need the structure of a large configuration
# (several tiles, ragged tails, GQA packing) at a size a CPU finishes in seconds.
MINI_1B = ModelShape("mini1b", 2, 512, 8, 2, 64, 1408, 2048)
MINI_8B = ModelShape("mini8b", 2, 512, 8, 2, 128, 1280, 4096)
