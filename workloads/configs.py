"""The five workload shapes (tiny, GPT-J-like, MPT-like long context,
Cerebras-GPT-like batched decode, prefill sweep) and scaled-down copies of them."""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int          # L
    batch: int             # B
    n_heads: int           # H
    head_dim: int          # d
    prompt_len: int        # n
    budget_k: int          # k
    recent_w: int          # w
    gen_len_T: int         # T (decode steps)
    tau_init: float = 1.0
    tau_end: float = 2.0
    data_seed: int = 0     # seed of the Q/K/V draws
    noise_seed: int = 0    # seed of the Gumbel noise
    positional: str = "none"       # "none" | "rotary" | "alibi"
    rotary_dims: int = 0           # leading dims rotated when positional == "rotary"
    heavy_frac: float = 0.0        # fraction of key positions that are heavy hitters
    heavy_logit: float = 0.0       # logit shift those keys receive (in units of scaled logits)
    n_kv_heads: int = 0            # key/value heads shared by groups of query heads (0 = one per query head)
    rotary_in_library: bool = False  # positional == "rotary": leave Q/K unrotated, the consumer applies the embedding itself

    @property
    def kv_heads(self) -> int:
        return self.n_kv_heads if self.n_kv_heads > 0 else self.n_heads

    @property
    def group(self) -> int:
        """Query heads per key/value head."""
        return self.n_heads // self.kv_heads

    @property
    def units(self) -> int:
        """Caches of the workload: one per (layer, batch row, key/value head)."""
        return self.n_layers * self.batch * self.kv_heads

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


def alibi_slopes(n_heads: int) -> np.ndarray:
    """slope_h = 2^(-8 (h+1) / H) for the 0-based head index h (geometric ALiBi slopes)."""
    h = np.arange(1, n_heads + 1, dtype=np.float64)
    return np.exp2(-8.0 * h / n_heads)


CONFIGS = {
    "c1_tiny": Workload("c1_tiny", 1, 1, 4, 64, 512, 256, 64, 32, data_seed=1, noise_seed=0),
    "c2_gptj": Workload("c2_gptj", 1, 1, 16, 256, 2048, 1024, 256, 256, data_seed=2, noise_seed=2,
                        positional="rotary", rotary_dims=64),
    "c3_mpt": Workload("c3_mpt", 1, 1, 32, 128, 8192, 4096, 1024, 512, data_seed=3, noise_seed=3,
                       positional="alibi"),
    "c4_cerebras": Workload("c4_cerebras", 32, 32, 32, 128, 4096, 2048, 512, 256, data_seed=4, noise_seed=4,
                            heavy_frac=0.05, heavy_logit=3.0),
    # the same model with its 32 query heads sharing 8 key/value heads (grouped-query attention, 4 heads per group)
    "c4_cerebras_gqa8": Workload("c4_cerebras_gqa8", 32, 32, 32, 128, 4096, 2048, 512, 256, data_seed=4, noise_seed=4,
                                 heavy_frac=0.05, heavy_logit=3.0, n_kv_heads=8),
    # prefill sweep: one entry per prompt length; budgets are swept by the caller
    "c5_prefill_1k": Workload("c5_prefill_1k", 1, 8, 32, 128, 1024, 512, 128, 0, data_seed=5, noise_seed=5),
    "c5_prefill_2k": Workload("c5_prefill_2k", 1, 8, 32, 128, 2048, 1024, 256, 0, data_seed=5, noise_seed=5),
    "c5_prefill_4k": Workload("c5_prefill_4k", 1, 8, 32, 128, 4096, 2048, 512, 0, data_seed=5, noise_seed=5),
    "c5_prefill_8k": Workload("c5_prefill_8k", 1, 8, 32, 128, 8192, 4096, 1024, 0, data_seed=5, noise_seed=5),
}

C5_BUDGET_FRACTIONS = (0.1, 0.3, 0.5, 0.7, 0.9)


def c5_budget(n: int, frac: float) -> tuple[int, int]:
    """(k, w) of the prefill sweep: k = frac * n, w = k / 4."""
    k = int(round(n * frac))
    return k, k // 4


def get_config(name: str) -> Workload:
    return CONFIGS[name]
