"""Shapes and batch recipes of the five verification workloads.

The paper evaluates on reasoning traces (32K-37K token budgets, steps ending
at a blank line, k = 5 drafted steps per iteration; Section 5.1). None of that
data is available offline, so each workload is a seeded synthetic stand-in with
the same structure: a cached context of some thousand tokens per step, a short
span of new tokens (draft step + target step + a fixed verification suffix),
and a batch of several requests times k candidate steps.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Tuple


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
    rope_theta: float
    rms_eps: float = 1e-6
    init_std: float = 0.02
    # per-head RMSNorm of the query and key vectors before the rotary turn (the Qwen3-style second family)
    qk_norm: bool = False

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def params_per_layer(self) -> int:
        d, f = self.d_model, self.d_ffn
        return d * (self.q_dim + 2 * self.kv_dim) + self.q_dim * d + 3 * d * f


TINY = ModelShape("tiny", 2, 256, 4, 4, 64, 688, 4096, 1.0e4)
QWEN_1P5B = ModelShape("qwen2.5-1.5b-shaped", 28, 1536, 12, 2, 128, 8960, 151936, 1.0e6)
QWEN_7B = ModelShape("qwen2.5-7b-shaped", 28, 3584, 28, 4, 128, 18944, 152064, 1.0e6)
# the draft model of the paper's second family (per-head query/key normalisation, head_dim not d_model / heads)
QWEN3_1P7B = ModelShape("qwen3-1.7b-shaped", 28, 2048, 16, 8, 128, 6144, 151936, 1.0e6, qk_norm=True)
TINY_QKNORM = ModelShape("tiny-qknorm", 2, 256, 4, 2, 64, 688, 4096, 1.0e4, qk_norm=True)


@dataclass(frozen=True)
class VerifyConfig:
    name: str
    model: ModelShape
    batch: int
    # context length distribution: ("fixed", n) | ("uniform", lo, hi) | ("lognormal", median, sigma, lo, hi)
    ctx_dist: Tuple
    # step length distribution (before the verify suffix): ("fixed", n) | ("uniform", lo, hi)
    step_dist: Tuple
    suffix_len: int = 8
    page_size: int = 16
    tau: float = 0.9
    taus: Tuple[float, ...] = ()
    verdict_ids: Tuple[int, ...] = (1, 2)
    # "prefill": context K/V come from running the model over seeded context tokens;
    # "synthetic": context K/V are drawn i.i.d. N(0, kv_std^2), rounded to bf16, K taken as already rotated.
    ctx_kv: str = "synthetic"
    kv_std: float = 0.78
    # cache format: "bf16", or an 8-bit float, unscaled, synthetic contexts only: "e4m3" (4 exponent / 3 mantissa bits)
    # or "e5m2" (5 / 2: the upper byte of an fp16)
    kv_format: str = "bf16"
    seed: int = 20260218


CONFIGS = {
    "cfg1_tiny": VerifyConfig(
        "cfg1_tiny", TINY, 4, ("fixed", 128), ("fixed", 32), tau=0.8, ctx_kv="prefill", seed=101),
    "cfg2_1p5b_b16": VerifyConfig(
        "cfg2_1p5b_b16", QWEN_1P5B, 16, ("uniform", 512, 2048), ("uniform", 24, 96), tau=0.9, seed=202),
    "cfg3_1p5b_b64": VerifyConfig(
        "cfg3_1p5b_b64", QWEN_1P5B, 64, ("lognormal", 1500.0, 0.6, 128, 8192), ("uniform", 16, 128),
        tau=0.9, taus=(0.5, 0.7, 0.9, 0.95, 0.99), seed=303),
    "cfg4_1p5b_long": VerifyConfig(
        "cfg4_1p5b_long", QWEN_1P5B, 8, ("uniform", 8192, 32768), ("uniform", 32, 128), tau=0.9, seed=404),
    "cfg5_7b_b32": VerifyConfig(
        "cfg5_7b_b32", QWEN_7B, 32, ("uniform", 1024, 4096), ("uniform", 24, 96), tau=0.9, seed=505),
    # beyond the five: the second model family, with the first family's batch recipe ...
    "cfg6_q3_b16": VerifyConfig(
        "cfg6_q3_b16", QWEN3_1P7B, 16, ("uniform", 512, 2048), ("uniform", 24, 96), tau=0.9, seed=606),
    # ... and a decode-shaped batch: many steps of at most 8 new tokens on long contexts, where attention is
    # bound by reading the cache rather than by arithmetic
    "cfg7_q3_short": VerifyConfig(
        "cfg7_q3_short", QWEN3_1P7B, 64, ("uniform", 2048, 8192), ("uniform", 1, 4), suffix_len=4, tau=0.9, seed=707),
    "cfg9_q3_short_fp8": VerifyConfig(
        "cfg9_q3_short_fp8", QWEN3_1P7B, 64, ("uniform", 2048, 8192), ("uniform", 1, 4), suffix_len=4, tau=0.9, seed=707,
        kv_format="e4m3"),
    "cfg10_q3_short_e5m2": VerifyConfig(
        "cfg10_q3_short_e5m2", QWEN3_1P7B, 64, ("uniform", 2048, 8192), ("uniform", 1, 4), suffix_len=4, tau=0.9,
        seed=707, kv_format="e5m2"),
    "cfg8_tiny_qknorm": VerifyConfig(
        "cfg8_tiny_qknorm", TINY_QKNORM, 6, ("uniform", 20, 150), ("uniform", 1, 40), tau=0.8, ctx_kv="prefill",
        seed=808),
}


@dataclass(frozen=True)
class CascadeConfig:
    """Two-tier verification (Eq. 4): the batch recipe, threshold and draft verifier of `draft`, plus the shape
    and weight seed of the target verifier that re-verifies the escalated steps. Both models cache the same
    contexts; the batch (token ids, lengths) is the draft config's."""
    name: str
    draft: VerifyConfig
    target_model: ModelShape
    target_seed: int

    @property
    def target(self) -> VerifyConfig:
        """The draft's recipe with the target's shape and seed: for drawing the target's weights and its cached
        context K/V. Its batch is NOT drawn from this (the seeds differ); both tiers share the draft's batch."""
        return replace(self.draft, name=self.name + "_target", model=self.target_model, seed=self.target_seed)


TINY_TARGET = ModelShape("tiny-target", 3, 384, 6, 2, 64, 1024, 4096, 1.0e4)

CASCADES = {
    "cascade_tiny": CascadeConfig(
        "cascade_tiny", replace(CONFIGS["cfg1_tiny"], batch=12), TINY_TARGET, 111),
    "cascade_1p5b_7b": CascadeConfig(
        "cascade_1p5b_7b", CONFIGS["cfg2_1p5b_b16"], QWEN_7B, 606),
}


def get_cascade(name: str, *, target_layers: int | None = None) -> CascadeConfig:
    c = CASCADES[name]
    if target_layers is not None:
        tm = replace(c.target_model, n_layers=target_layers, name=f"{c.target_model.name}-L{target_layers}")
        c = replace(c, target_model=tm)
    return c


def get_config(name: str) -> VerifyConfig:
    return CONFIGS[name]


def scaled_config(name: str, *, n_layers: int | None = None, batch: int | None = None,
                  vocab: int | None = None) -> VerifyConfig:
    """A cheaper variant of a named workload (fewer layers / steps / vocab rows) with every
    other dimension kept, used where the CPU oracle has to finish in seconds."""
    cfg = CONFIGS[name]
    m = cfg.model
    if n_layers is not None:
        m = replace(m, n_layers=n_layers, name=f"{m.name}-L{n_layers}")
    if vocab is not None:
        m = replace(m, vocab=vocab, name=f"{m.name}-V{vocab}")
    cfg = replace(cfg, model=m)
    if batch is not None:
        cfg = replace(cfg, batch=batch)
    return cfg
