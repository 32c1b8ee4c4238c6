"""The five benchmark workloads as plain data.

Shapes follow the layer geometries the paper evaluates on (Llama-3.1-8B and
Qwen2.5-7B style grouped-query attention, 4 sink tokens, pooling kernel 7 with
max pooling and mean group aggregation as in the experiments section); the
budgets (local window, top-k, rank) are the ones the benchmark definition
fixes.  `context` counts every prompt token including the sinks, and the last
row of the generated K/V is the current decode token, so the non-sink cache
length is L = context - sink_count.
"""
from __future__ import annotations

import dataclasses


@dataclasses.dataclass(frozen=True)
class LayerConfig:
    name: str
    dtype: str            # "f32" | "bf16"  (storage type of K, V, q, sinks, bases, coefficients)
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    context: int          # prompt tokens incl. sinks; last one is the current token
    sink_count: int
    rank_k: int
    rank_v: int
    window: int           # local window W (Eq. 13)
    top_k: int            # global budget k (Eq. 14)
    n_sampled: int        # rows sampled for basis construction
    alpha_k: float        # key latent spectrum sigma_i = i^-alpha
    alpha_v: float
    noise_std: float = 0.05
    sink_scale: float = 10.0
    outlier_frac: float = 0.0
    outlier_scale: float = 8.0
    rope_theta: float = 0.0
    query_scale: float = 4.0
    query_cos: float = 0.6
    n_planted: int = 16
    pool_kernel: int = 7
    pool_mode: str = "max"
    group_mode: str = "mean"
    n_layers: int = 1
    decode_steps: int = 1
    seed: int = 0

    @property
    def d_kv(self) -> int:           # D' = h_kv * d_h
        return self.n_kv_heads * self.head_dim

    @property
    def group(self) -> int:          # G
        return self.n_q_heads // self.n_kv_heads

    @property
    def cache_len(self) -> int:      # L, non-sink rows incl. the current token
        return self.context - self.sink_count

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2


CONFIGS = {
    0: LayerConfig("cfg0_tiny_f32_4k", "f32", 1, 8, 2, 128, 4096, 4, 64, 64, 64, 256, 512,
                   0.8, 0.8, rope_theta=1.0e4),
    1: LayerConfig("cfg1_llama8b_bf16_32k", "bf16", 1, 32, 8, 128, 32768, 4, 192, 192, 64, 1024, 1024,
                   0.8, 0.8, rope_theta=5.0e5),
    2: LayerConfig("cfg2_llama8b_bf16_128k_b8", "bf16", 8, 32, 8, 128, 131072, 4, 192, 192, 128, 2048, 1024,
                   0.8, 0.8, rope_theta=5.0e5),
    3: LayerConfig("cfg3_qwen7b_bf16_128k_b4", "bf16", 4, 28, 4, 128, 131072, 4, 128, 128, 64, 1024, 1024,
                   1.2, 0.8, outlier_frac=0.02, rope_theta=1.0e6),
    4: LayerConfig("cfg4_llama8b_bf16_64k_b16_e2e", "bf16", 16, 32, 8, 128, 65536, 4, 192, 192, 64, 1024, 1024,
                   0.8, 0.8, rope_theta=5.0e5, n_layers=32, decode_steps=64),
}


def get_config(i: int) -> LayerConfig:
    return CONFIGS[i]


def scaled_config(cfg: LayerConfig, **overrides) -> LayerConfig:
    """A copy of `cfg` with some fields replaced (smaller context, batch, ...)."""
    return dataclasses.replace(cfg, **overrides)
