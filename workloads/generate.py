"""Seeded draws of every input of the verification pass.

Every tensor has its own seed sequence (config seed, tensor tag, indices), so
any single piece — one layer's weights, one step's context K/V for one layer —
can be regenerated alone and always comes out bit-identical, whatever the number
of worker threads. Values that the model stores in bf16 are returned as uint16
bit patterns (round-to-nearest-even of the fp32 draw); nothing here decodes them
or computes with them.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from .configs import ModelShape, VerifyConfig

_TAG_WEIGHT, _TAG_BATCH, _TAG_CTXKV, _TAG_PAGES, _TAG_PLANT = 1, 2, 3, 4, 5
_CHUNK_ELEMS = 1 << 23

_GLOBAL_TENSORS = ("embed", "lm_head")
_LAYER_TENSORS = ("wq", "wk", "wv", "wo", "wg", "wu", "wd")


def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(k) for k in key])))


def bf16_bits_from_f32(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (nearest, ties to even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def e4m3_codes_from_f32(x: np.ndarray) -> np.ndarray:
    """Round to the nearest value of the 8-bit float with 4 exponent bits (bias 7), 3 mantissa bits and no infinities
    (ties to the even code, magnitudes beyond 448 saturate) and return the codes as uint8. Storage conversion only.
    Below 2^-6 the format is a fixed-point grid of step 2^-9 (codes 0 .. 8, code 8 being the smallest normal);
    above, the fp32 mantissa is rounded to 3 bits in place and the exponent re-biased."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    sign = ((u >> np.uint32(24)) & np.uint32(0x80)).astype(np.uint8)
    au = u & np.uint32(0x7FFFFFFF)
    r = au + np.uint32(0x7FFFF)
    r += (au >> np.uint32(20)) & np.uint32(1)
    r >>= np.uint32(20)                                   # (fp32 exponent field << 3) | 3 mantissa bits
    np.minimum(r, np.uint32(((127 - 7) << 3) + 0x7E), out=r)
    code = r.astype(np.int32) - np.int32((127 - 7) << 3)
    a = au.view(np.float32)
    small = a < np.float32(2.0 ** -6)
    if small.any():
        code[small] = np.rint(a[small] * np.float32(512.0)).astype(np.int32)      # rint rounds ties to even
    return code.astype(np.uint8) | sign


def e5m2_codes_from_f32(x: np.ndarray) -> np.ndarray:
    """Round to the nearest value of the 8-bit float with 5 exponent bits (bias 15) and 2 mantissa bits (ties to the
    even code; magnitudes beyond the largest finite value 57344 saturate to it) and return the codes as uint8.
    Below 2^-14 the format is a fixed-point grid of step 2^-16 (codes 0 .. 4, code 4 being the smallest normal)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    sign = ((u >> np.uint32(24)) & np.uint32(0x80)).astype(np.uint8)
    au = u & np.uint32(0x7FFFFFFF)
    r = au + np.uint32(0xFFFFF)
    r += (au >> np.uint32(21)) & np.uint32(1)
    r >>= np.uint32(21)                                   # (fp32 exponent field << 2) | 2 mantissa bits
    np.minimum(r, np.uint32(((127 - 15) << 2) + 0x7B), out=r)
    code = r.astype(np.int32) - np.int32((127 - 15) << 2)
    a = au.view(np.float32)
    small = a < np.float32(2.0 ** -14)
    if small.any():
        code[small] = np.rint(a[small] * np.float32(65536.0)).astype(np.int32)
    return code.astype(np.uint8) | sign


def _normal_bf16(key: Tuple[int, ...], shape: Tuple[int, ...], std: float,
                 pool: Optional[ThreadPoolExecutor] = None) -> np.ndarray:
    """i.i.d. N(0, std^2) rounded to bf16; drawn in fixed row chunks with one stream per chunk."""
    rows = int(shape[0])
    row_elems = int(np.prod(shape[1:], dtype=np.int64)) if len(shape) > 1 else 1
    out = np.empty((rows, row_elems), dtype=np.uint16)
    rows_per_chunk = max(1, _CHUNK_ELEMS // max(1, row_elems))
    n_chunks = (rows + rows_per_chunk - 1) // rows_per_chunk

    def fill(ci: int) -> None:
        r0 = ci * rows_per_chunk
        r1 = min(rows, r0 + rows_per_chunk)
        g = _rng(*key, ci)
        z = g.standard_normal((r1 - r0, row_elems), dtype=np.float32)
        z *= np.float32(std)
        out[r0:r1] = bf16_bits_from_f32(z)

    if pool is None or n_chunks == 1:
        for ci in range(n_chunks):
            fill(ci)
    else:
        list(pool.map(fill, range(n_chunks)))
    return out.reshape(shape)


def _weight_shapes(m: ModelShape) -> Dict[str, Tuple[int, int]]:
    return {
        "embed": (m.vocab, m.d_model), "lm_head": (m.vocab, m.d_model),
        "wq": (m.q_dim, m.d_model), "wk": (m.kv_dim, m.d_model), "wv": (m.kv_dim, m.d_model),
        "wo": (m.d_model, m.q_dim), "wg": (m.d_ffn, m.d_model), "wu": (m.d_ffn, m.d_model),
        "wd": (m.d_model, m.d_ffn),
    }


def model_weights(m: ModelShape, seed: int, threads: Optional[int] = None) -> dict:
    """Random-init decoder weights: every matrix bf16(N(0, init_std^2)), stored [out_features, in_features]
    row-major as uint16 bit patterns; RMSNorm gains fp32 1.0; embedding and LM head are separate draws."""
    shapes = _weight_shapes(m)
    threads = threads or min(16, os.cpu_count() or 1)
    with ThreadPoolExecutor(max_workers=threads) as pool:
        w: dict = {"shape": m, "layers": []}
        for ti, name in enumerate(_GLOBAL_TENSORS):
            w[name] = _normal_bf16((seed, _TAG_WEIGHT, 0, ti), shapes[name], m.init_std, pool)
        w["final_norm"] = np.ones(m.d_model, dtype=np.float32)
        for li in range(m.n_layers):
            layer = {}
            for ti, name in enumerate(_LAYER_TENSORS):
                layer[name] = _normal_bf16((seed, _TAG_WEIGHT, li + 1, ti), shapes[name], m.init_std, pool)
            layer["norm1"] = np.ones(m.d_model, dtype=np.float32)
            layer["norm2"] = np.ones(m.d_model, dtype=np.float32)
            if m.qk_norm:
                # trained gains of this kind are far from 1 and differ per entry; draw them so that a swapped
                # or dropped gain shows
                g = _rng(seed, _TAG_WEIGHT, li + 1, 100)
                layer["q_norm"] = (1.0 + 0.25 * g.standard_normal(m.head_dim)).astype(np.float32)
                layer["k_norm"] = (1.0 + 0.25 * g.standard_normal(m.head_dim)).astype(np.float32)
            w["layers"].append(layer)
    return w


def plant_verdict_rows(w: dict, verdict_ids: Sequence[int], beta: float, seed: int) -> None:
    """Overwrite the LM-head rows of the first two verdict ids with +beta*u and -beta*u (u a seeded unit
    vector), in place. With random-init weights every vocabulary probability is about 1/V, so the
    confidence never comes near a realistic threshold; this spreads it over (0, 1) without changing any
    shape or cost. Pure input construction."""
    m: ModelShape = w["shape"]
    u = _rng(seed, _TAG_PLANT).standard_normal(m.d_model)
    u /= np.sqrt(np.sum(u * u))
    row = (beta * u).astype(np.float32)
    w["lm_head"][int(verdict_ids[0])] = bf16_bits_from_f32(row)
    w["lm_head"][int(verdict_ids[1])] = bf16_bits_from_f32(-row)


@dataclass
class Batch:
    ctx_lens: np.ndarray       # int32 [B]   cached context length of each step
    step_lens: np.ndarray      # int32 [B]   new tokens of each step, verify suffix included
    cu_new: np.ndarray         # int32 [B+1] exclusive prefix sum of step_lens
    step_tokens: np.ndarray    # int32 [T]   concatenated new tokens (step body then suffix)
    suffix: np.ndarray         # int32 [suffix_len] shared verify suffix
    ctx_tokens: Optional[List[np.ndarray]]  # per step context token ids when the context is a real prefill

    @property
    def n_steps(self) -> int:
        return int(self.ctx_lens.shape[0])

    @property
    def n_tokens(self) -> int:
        return int(self.cu_new[-1])


def _draw_lengths(g: np.random.Generator, dist: Tuple, n: int) -> np.ndarray:
    kind = dist[0]
    if kind == "fixed":
        return np.full(n, int(dist[1]), dtype=np.int32)
    if kind == "uniform":
        return g.integers(int(dist[1]), int(dist[2]) + 1, size=n, dtype=np.int64).astype(np.int32)
    if kind == "lognormal":
        median, sigma, lo, hi = dist[1:]
        x = g.lognormal(mean=float(np.log(median)), sigma=float(sigma), size=n)
        return np.clip(np.rint(x), lo, hi).astype(np.int32)
    raise ValueError(f"unknown length distribution {dist!r}")


def make_batch(cfg: VerifyConfig, seed: Optional[int] = None) -> Batch:
    """Context lengths, step lengths and token ids of one batch. Token ids are uniform over
    [first non-reserved id, vocab): ids 0..max(verdict_ids) are never drawn."""
    seed = cfg.seed if seed is None else seed
    g = _rng(seed, _TAG_BATCH)
    lo_id = max(cfg.verdict_ids) + 1
    ctx_lens = _draw_lengths(g, cfg.ctx_dist, cfg.batch)
    body = _draw_lengths(g, cfg.step_dist, cfg.batch)
    suffix = g.integers(lo_id, cfg.model.vocab, size=cfg.suffix_len, dtype=np.int64).astype(np.int32)
    step_lens = (body + cfg.suffix_len).astype(np.int32)
    cu = np.zeros(cfg.batch + 1, dtype=np.int32)
    np.cumsum(step_lens, out=cu[1:])
    toks = np.empty(int(cu[-1]), dtype=np.int32)
    for i in range(cfg.batch):
        t = g.integers(lo_id, cfg.model.vocab, size=int(body[i]), dtype=np.int64).astype(np.int32)
        toks[cu[i]:cu[i] + body[i]] = t
        toks[cu[i] + body[i]:cu[i + 1]] = suffix
    ctx_tokens = None
    if cfg.ctx_kv == "prefill":
        ctx_tokens = [g.integers(lo_id, cfg.model.vocab, size=int(c), dtype=np.int64).astype(np.int32)
                      for c in ctx_lens]
    return Batch(ctx_lens, step_lens, cu, toks, suffix, ctx_tokens)


def context_kv(cfg: VerifyConfig, step: int, layer: int, ctx_len: int,
               seed: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Synthetic cached K and V of one step for one layer: uint16 bf16 bits (uint8 codes of an 8-bit format when
    cfg.kv_format is "e4m3" or "e5m2": the same draws, rounded once more), each [ctx_len, n_kv_heads, head_dim],
    i.i.d. N(0, kv_std^2). K is taken as already rotated."""
    seed = cfg.seed if seed is None else seed
    m = cfg.model
    shape = (int(ctx_len), m.n_kv_heads, m.head_dim)
    k = _normal_bf16((seed, _TAG_CTXKV, step, layer, 0), shape, cfg.kv_std)
    v = _normal_bf16((seed, _TAG_CTXKV, step, layer, 1), shape, cfg.kv_std)
    if cfg.kv_format in ("e4m3", "e5m2"):
        widen = lambda b: (b.astype(np.uint32) << np.uint32(16)).view(np.float32)
        enc = e4m3_codes_from_f32 if cfg.kv_format == "e4m3" else e5m2_codes_from_f32
        return enc(widen(k)), enc(widen(v))
    return k, v


def page_assignment(cfg: VerifyConfig, ctx_lens: np.ndarray, seed: Optional[int] = None,
                    slack_pages: int = 3) -> Tuple[int, List[np.ndarray]]:
    """Pages of each step's context, taken from a seeded permutation of the pool so that a sequence's
    pages are neither contiguous nor ordered. Returns (pool size in pages, per-step page id arrays)."""
    seed = cfg.seed if seed is None else seed
    need = [(int(c) + cfg.page_size - 1) // cfg.page_size for c in ctx_lens]
    total = sum(need) + slack_pages
    perm = _rng(seed, _TAG_PAGES).permutation(total).astype(np.int32)
    out, o = [], 0
    for n in need:
        out.append(perm[o:o + n].copy())
        o += n
    return total, out
