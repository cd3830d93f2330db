"""Wires a seeded workload (model tensors, paged contexts, a batch of steps) to the C ABI.

Only plumbing: allocation of output tensors with torch, upload of inputs, and the calls. Used by the tests,
the smoke check and the benchmark so that all three drive the library the same way.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as B


class VerifySession:
    """One model, one paged context cache and one batch of steps resident on the GPU."""

    def __init__(self, cfg, weights: dict, batch, device: str = "cuda:0"):
        self.cfg, self.batch = cfg, batch
        self.shape = cfg.model
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        B.load_library()
        self.model = B.cs_model_load(self.shape, weights)
        self.kv = None
        self.n_steps = batch.n_steps
        self.seq_ids = np.arange(self.n_steps, dtype=np.int32)
        self.out_conf = torch.empty(self.n_steps, dtype=torch.float32, device=self.device)
        self.out_accept = torch.empty(self.n_steps, dtype=torch.uint8, device=self.device)
        self.out_verdict = torch.empty(self.n_steps, dtype=torch.int32, device=self.device)
        self.tokens_dev = torch.from_numpy(batch.step_tokens.astype(np.int32)).to(self.device)
        self.tokens_pinned = torch.from_numpy(batch.step_tokens.astype(np.int32)).pin_memory()

    # ---------------------------------------------------------------- context cache
    def alloc_cache(self, pages_per_step: List[np.ndarray], total_pages: int, ctx_lens: Sequence[int],
                    room_for_prefill: bool = False) -> None:
        ps = self.cfg.page_size
        max_pp = max(1, max(len(p) for p in pages_per_step))
        fmt = getattr(self.cfg, "kv_format", "bf16")
        if fmt in ("e4m3", "e5m2"):
            self.kv = B.cs_kv_alloc_8bit(self.model, total_pages, ps, self.n_steps, max_pp, fmt)
        else:
            self.kv = B.cs_kv_alloc(self.model, total_pages, ps, self.n_steps, max_pp)
        for i, pages in enumerate(pages_per_step):
            B.cs_kv_set_seq(self.kv, i, pages, 0 if room_for_prefill else int(ctx_lens[i]))

    def fill_synthetic_context(self, context_kv_fn, threads: Optional[int] = None) -> None:
        """context_kv_fn(step, layer) -> (K, V) uint16 arrays [ctx_len, n_kv_heads, head_dim]."""
        jobs = [(i, l) for i in range(self.n_steps) for l in range(self.shape.n_layers)]
        threads = threads or min(16, os.cpu_count() or 8)
        with ThreadPoolExecutor(max_workers=threads) as pool:
            chunk = 4 * threads
            for o in range(0, len(jobs), chunk):
                part = jobs[o:o + chunk]
                for (i, l), (k, v) in zip(part, pool.map(lambda j: context_kv_fn(*j), part)):
                    B.cs_kv_fill(self.kv, i, l, k, v)

    def prefill_context(self, ctx_tokens: List[np.ndarray]) -> None:
        lens = np.array([len(t) for t in ctx_tokens], dtype=np.int32)
        keep = lens > 0   # a sequence with an empty context has nothing to prefill
        if keep.any():
            toks = np.concatenate([t for t in ctx_tokens if len(t)]).astype(np.int32)
            B.cs_prefill(self.model, self.kv, self.seq_ids[keep], toks, lens[keep])
        torch.cuda.synchronize()

    # ---------------------------------------------------------------- the pass
    def verify(self, tau: Optional[float] = None, host_tokens: bool = False, stream=None) -> None:
        """Enqueue one verification pass over the whole batch; outputs land in out_conf/out_accept/out_verdict."""
        toks = self.tokens_pinned if host_tokens else self.tokens_dev
        B.cs_verify_steps(self.model, self.kv, self.seq_ids, toks, self.batch.step_lens, self.cfg.verdict_ids,
                          self.cfg.tau if tau is None else tau, self.out_conf, self.out_accept, self.out_verdict,
                          stream=stream)

    def results(self) -> dict:
        torch.cuda.synchronize()
        B.cs_last_status(self.model)
        return {"conf": self.out_conf.cpu().numpy(), "accept": self.out_accept.cpu().numpy(),
                "verdict": self.out_verdict.cpu().numpy()}

    def last_logits(self) -> np.ndarray:
        out = torch.empty(self.n_steps, self.shape.vocab, dtype=torch.float32, device=self.device)
        B.cs_get_last_logits(self.model, out, self.n_steps)
        torch.cuda.synchronize()
        return out.cpu().numpy()

    def last_lse(self) -> np.ndarray:
        out = torch.empty(self.n_steps, dtype=torch.float32, device=self.device)
        B.cs_get_last_lse(self.model, out, self.n_steps)
        torch.cuda.synchronize()
        return out.cpu().numpy()

    def close(self) -> None:
        if self.kv is not None:
            B.cs_kv_free(self.kv)
            self.kv = None
        if self.model is not None:
            B.cs_model_free(self.model)
            self.model = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()


class CascadeSession:
    """A draft and a target VerifySession over the same batch (each model caches the same contexts under the same
    sequence ids) and the outputs of the two-tier pass."""

    def __init__(self, draft: VerifySession, target: VerifySession):
        assert draft.n_steps == target.n_steps
        self.draft, self.target = draft, target
        n, dev = draft.n_steps, draft.device
        self.out_conf_t = torch.empty(n, dtype=torch.float32, device=dev)
        self.out_verdict_t = torch.empty(n, dtype=torch.int32, device=dev)
        self.out_conf = torch.empty(n, dtype=torch.float32, device=dev)
        self.out_verdict = torch.empty(n, dtype=torch.int32, device=dev)
        self.n_escalated = -1

    def verify(self, tau: Optional[float] = None, req_offsets=None, accept_index: int = 0, stream=None) -> int:
        d = self.draft
        self.n_escalated = B.cs_verify_cascade(
            d.model, d.kv, self.target.model, self.target.kv, d.seq_ids, d.tokens_pinned, d.batch.step_lens,
            d.cfg.verdict_ids, d.cfg.tau if tau is None else tau, d.out_conf, d.out_accept, d.out_verdict,
            self.out_conf_t, self.out_verdict_t, self.out_verdict, self.out_conf, req_offsets=req_offsets,
            accept_index=accept_index, stream=stream)
        return self.n_escalated

    def results(self) -> dict:
        torch.cuda.synchronize()
        B.cs_last_status(self.draft.model)
        B.cs_last_status(self.target.model)
        return {"conf_d": self.draft.out_conf.cpu().numpy(), "trusted": self.draft.out_accept.cpu().numpy(),
                "verdict_d": self.draft.out_verdict.cpu().numpy(), "conf_t": self.out_conf_t.cpu().numpy(),
                "verdict_t": self.out_verdict_t.cpu().numpy(), "conf": self.out_conf.cpu().numpy(),
                "verdict": self.out_verdict.cpu().numpy(), "n_escalated": self.n_escalated}

    def close(self) -> None:
        self.draft.close()
        self.target.close()
