"""The five benchmark configurations as data, plus shrunken variants for parity tests."""
from __future__ import annotations

from dataclasses import dataclass, field, replace

import numpy as np

from . import generators as gen

__all__ = ["StepConfig", "StepInputs", "config0", "config1", "config3", "config4",
           "TOPP_SIZES", "TOPP_PS", "TOPP_FAMILIES", "make_step_inputs"]

TOPP_SIZES = (1024, 8192, 65536, 131072)
TOPP_PS = (0.5, 0.9, 0.99)
TOPP_FAMILIES = ("uniform", "zipf", "quantised")


@dataclass(frozen=True)
class StepConfig:
    name: str
    n_target_layers: int
    n_draft_layers: int
    batch: int
    ctx: int                      # context length (max over the batch when ragged)
    n_draft_heads: int
    gamma: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int
    paged: bool                   # False: contiguous cache, no block table
    p: float
    seed: int = 0
    ragged: bool = False
    ctx_min: int = 0              # ragged only
    n_groups: int = 1

    @property
    def n_q(self) -> int:
        return self.gamma + 1

    def scaled(self, **kw) -> "StepConfig":
        return replace(self, **kw)


def config0() -> StepConfig:
    return StepConfig("cfg0_single_layer_ctx4096", 1, 1, 1, 4096, 12, 4, 32, 8, 128, 16, False, 0.9, 0)


def config1() -> StepConfig:
    return StepConfig("cfg1_llama3_8b_b8_ctx32768", 32, 4, 8, 32768, 12, 5, 32, 8, 128, 16, True, 0.95, 1)


def config3() -> StepConfig:
    return StepConfig("cfg3_ragged_b32", 1, 1, 32, 65536, 12, 4, 32, 8, 128, 16, True, 0.9, 3,
                      ragged=True, ctx_min=2048)


def config4(n_target_layers: int = 80, p: float = 0.9) -> StepConfig:
    return StepConfig("cfg4_70b_b4_ctx131072", n_target_layers, 4, 4, 131072, 16, 4, 64, 8, 128, 16,
                      True, p, 4)


@dataclass
class StepInputs:
    cfg: StepConfig
    kv_len: np.ndarray                 # int32 [B]
    L_stride: int
    layer_map: np.ndarray              # int32 [n_target_layers]
    draft_probs: list                  # per draft layer float32 [B, H_d, gamma, L_stride]
    block_table: np.ndarray | None     # int32 [B, pages_per_seq]
    pages_per_seq: int
    n_pages: int
    q: list = field(default_factory=list)   # per target layer uint16 [B, T, H_q, d]


def make_step_inputs(cfg: StepConfig, with_q: bool = True) -> StepInputs:
    """Host-side inputs of one verification step (everything except the K/V pools, which
    ``generators.kv_pool`` produces per target layer on the device that needs them)."""
    if cfg.ragged:
        kv_len, sink, slope = gen.ragged_lengths(cfg.seed, cfg.batch, cfg.ctx_min, cfg.ctx)
    else:
        kv_len = np.full(cfg.batch, cfg.ctx, dtype=np.int32)
        sink, slope = 8.0, 0.002
    L_stride = gen.round_up(int(kv_len.max()), 4)
    if cfg.n_target_layers == 1:
        lmap = np.zeros(1, dtype=np.int32)
    else:
        lmap = gen.layer_map(cfg.seed, cfg.n_target_layers, cfg.n_draft_layers)
    used = set(int(x) for x in lmap if x >= 0)
    probs = [gen.draft_probs(cfg.seed, u, kv_len, cfg.n_draft_heads, cfg.gamma, L_stride, sink, slope)
             if u in used else None for u in range(cfg.n_draft_layers)]
    pages_per_seq = (int(kv_len.max()) + cfg.page_size - 1) // cfg.page_size
    n_pages = cfg.batch * pages_per_seq
    bt = gen.block_table(cfg.seed, cfg.batch, pages_per_seq, n_pages) if cfg.paged else None
    q = [gen.queries(cfg.seed, j, cfg.batch, cfg.n_q, cfg.n_q_heads, cfg.head_dim)
         for j in range(cfg.n_target_layers)] if with_q else []
    return StepInputs(cfg, kv_len, L_stride, lmap, probs, bt, pages_per_seq, n_pages, q)
