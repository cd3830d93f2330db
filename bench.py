#!/usr/bin/env python
"""Throughput of the batched draft-verification pass.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]
    python bench.py --cascade cascade_1p5b_7b [--steps K] [--warmup W]     (two-tier pass, one GPU; see run_cascade)

One "step" is one cs_verify_steps call over the whole batch of the workload (every kernel of the pass).
Prints ONE JSON line. With --gpus N > 1 every rank runs an independent replica on its own seeded batch (launched by
torch.distributed.run, or by this script itself when it is started without a launcher): the pass has no exchange
step, so there is no collective on the data path.
`--impl reference` times the CPU oracle (oracle/) on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from workloads import (context_kv, get_cascade, get_config, make_batch, model_weights, page_assignment,  # noqa: E402
                       plant_verdict_rows, scaled_config)

METRIC = "verified_steps_per_s"
UNIT = "steps/s"
DEFAULT_WORKLOAD = "cfg2_1p5b_b16"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# DRAM counters of the dominant kernel (one gate/up GEMM launch of the default workload): read from the small JSON that
# sits beside the ncu summary they were taken for. It names the kernel source and its hash at capture time; a kernel
# that has changed since has no counters, and traffic is then reported as null.
COUNTERS_JSON = os.path.join(ROOT, "profiles", "gemm_gateup_cfg2_counters.json")


def gateup_traffic(workload: str):
    import hashlib
    try:
        with open(COUNTERS_JSON) as f:
            c = json.load(f)
        with open(os.path.join(ROOT, c["source"]), "rb") as f:
            h = hashlib.sha256(f.read()).hexdigest()[:16]
    except (OSError, KeyError, ValueError):
        return None
    if workload != c.get("workload") or h != c.get("sha256_16"):
        return None
    return float(c["dram_bytes_read"]) + float(c["dram_bytes_write"])


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------------------------
# algorithmic work of the pass (per call)
# ------------------------------------------------------------------------------------------------
def work_counts(cfg, batch) -> dict:
    m = cfg.model
    T = int(batch.n_tokens)
    n = batch.step_lens.astype(np.float64)
    c = batch.ctx_lens.astype(np.float64)
    attn_flops_layer = float(np.sum(4.0 * m.n_q_heads * m.head_dim * (n * c + n * (n + 1) / 2)))
    cell = 1 if getattr(cfg, "kv_format", "bf16") in ("e4m3", "e5m2") else 2
    kv_row = 2 * m.n_kv_heads * m.head_dim * cell                    # bytes of K+V per token per layer
    attn_bytes_layer = float(np.sum(c) * kv_row + T * (m.q_dim + 2 * m.kv_dim + m.q_dim) * 2)
    return {
        "T": T,
        "gemm_qkv_flops": 2.0 * T * (m.q_dim + 2 * m.kv_dim) * m.d_model,
        "gemm_o_flops": 2.0 * T * m.d_model * m.q_dim,
        "gemm_gateup_flops": 2.0 * T * (2 * m.d_ffn) * m.d_model,
        "gemm_down_flops": 2.0 * T * m.d_model * m.d_ffn,
        "attention_flops": attn_flops_layer,
        "attention_bytes": attn_bytes_layer,
        "lm_head_bytes": 2.0 * m.vocab * m.d_model + batch.n_steps * m.d_model * 2,
        "lm_head_flops": 2.0 * batch.n_steps * m.vocab * m.d_model,
    }


# ------------------------------------------------------------------------------------------------
# clock sampling during the timed region
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_uuid: str):
        self.rows = []
        self.proc = None
        self.uuid = gpu_uuid

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", self.uuid], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass

    def summary(self, t0: float, t1: float) -> dict:
        sm, mx, reasons = [], [], set()
        for ts, line in self.rows:
            if ts < t0 or ts > t1 + 0.2:
                continue
            p = [x.strip() for x in line.split(",")]
            if len(p) < 7:
                continue
            try:
                sm.append(float(p[0]))
                mx.append(float(p[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# CPU oracle leg (bounded sample)
# ------------------------------------------------------------------------------------------------
def oracle_sample_run(cfg, weights, batch, sample_steps):
    """One oracle pass over `sample_steps` of the batch; returns seconds."""
    from oracle import confspec_oracle as O
    toks = [batch.step_tokens[batch.cu_new[i]:batch.cu_new[i + 1]] for i in sample_steps]

    def fn(j, l):
        i = sample_steps[j]
        k, v = context_kv(cfg, i, l, int(batch.ctx_lens[i]))
        return O.widen_bf16(k), O.widen_bf16(v)

    t = time.perf_counter()
    if cfg.ctx_kv == "prefill":
        kv = O.prefill_context(weights, [batch.ctx_tokens[i] for i in sample_steps], store_bf16=True)
        fn = lambda j, l: kv[j][l]  # noqa: E731
    O.verify_steps(weights, toks, [int(batch.ctx_lens[i]) for i in sample_steps], fn, cfg.verdict_ids, cfg.tau)
    return time.perf_counter() - t


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return int(max(n)) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    weights = model_weights(cfg.model, cfg.seed)
    batch = make_batch(cfg)
    sample = list(range(min(2, batch.n_steps)))
    for _ in range(args.warmup):
        oracle_sample_run(cfg, weights, batch, sample[:1])
    t = 0.0
    for _ in range(args.steps):
        t += oracle_sample_run(cfg, weights, batch, sample)
    value = len(sample) * args.steps / t
    tok = float(sum(int(batch.step_lens[i]) for i in sample)) * args.steps / t
    desc = f"steps {sample} of the {batch.n_steps}-step batch per pass, context K/V generation included"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "tokens_per_s": tok,
        "config": {"workload": cfg.name, "model": cfg.model.name, "batch": cfg.batch, "sampled_steps": len(sample)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------------
# rank aggregation (replicas only: no collective on the data path, only on the timings)
# ------------------------------------------------------------------------------------------------
def aggregate_over_ranks(ms: float, ms_e2e: float, n_steps: int, n_tokens: int, device=None):
    """Whole-job figures of N independent replicas: the slowest rank's device times (MAX) and the units all
    ranks processed (SUM). Without an initialised process group it returns the inputs unchanged."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms), float(ms_e2e), float(n_steps), float(n_tokens)
    t = torch.tensor([ms, ms_e2e], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    nb = torch.tensor([n_steps, n_tokens], dtype=torch.float64, device=device)
    dist.all_reduce(nb, op=dist.ReduceOp.SUM)
    return float(t[0]), float(t[1]), float(nb[0]), float(nb[1])


def replica_seed(cfg, rank: int) -> int:
    """Every replica verifies its own seeded batch."""
    return cfg.seed + 7919 * rank


# ------------------------------------------------------------------------------------------------
# CUDA path
# ------------------------------------------------------------------------------------------------
def projections_back_to_back(cfg, T, tensor_peak, tensor_peak_sus, iters=40):
    """The projection kernels that have an entry point of their own (gate/up + SwiGLU, down and O with the residual
    epilogue in its default, ordered mode), launched back to back at the workload's shapes with one event pair around
    the whole series: what a launch costs when nothing serialises it. Six weight sets are rotated, more than L2 holds."""
    import torch
    from paper_2602_18447_b200 import binding as B
    m = cfg.model
    out = {}
    for name, N, K, epi in (("gemm_gateup", m.d_ffn, m.d_model, 2), ("gemm_down", m.d_model, m.d_ffn, 1),
                            ("gemm_o", m.d_model, m.q_dim, 1)):
        a = torch.randn(T, K, device="cuda").half()
        nw = 6
        ws = [(0.02 * torch.randn(N, K, device="cuda")).half() for _ in range(nw)]
        w2 = [(0.02 * torch.randn(N, K, device="cuda")).half() for _ in range(nw)] if epi == 2 else [None] * nw
        o = torch.zeros(T, N, device="cuda", dtype=torch.float32 if epi == 1 else torch.float16)
        for i in range(5):
            B.cs_gemm_f16(a, ws[i % nw], w2[i % nw], o, T, N, K, epi)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            B.cs_gemm_f16(a, ws[i % nw], w2[i % nw], o, T, N, K, epi)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / iters
        tf = 2.0 * T * N * K * (2 if epi == 2 else 1) / (ms * 1e-3) / 1e12
        out[name] = {"ms_per_launch": ms, "tflops": tf, "frac_tensor": tf / tensor_peak,
                     "frac_tensor_sustained": tf / tensor_peak_sus}
        del a, ws, w2, o
    return out


def run_ours(args, cfg):
    import torch
    import torch.distributed as dist
    from paper_2602_18447_b200 import VerifySession, binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the pass has no CPU path")
    if world != args.gpus:
        raise RuntimeError(f"--gpus {args.gpus} but the launcher started {world} process(es)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()

    weights = model_weights(cfg.model, cfg.seed)
    batch = make_batch(cfg, seed=replica_seed(cfg, rank))
    ses = VerifySession(cfg, weights, batch, device=f"cuda:{local}")
    total, pages = page_assignment(cfg, batch.ctx_lens)
    if cfg.ctx_kv == "prefill":
        ses.alloc_cache(pages, total, batch.ctx_lens, room_for_prefill=True)
        ses.prefill_context(batch.ctx_tokens)
    else:
        ses.alloc_cache(pages, total, batch.ctx_lens)
        ses.fill_synthetic_context(lambda i, l: context_kv(cfg, i, l, int(batch.ctx_lens[i])))
    B.cs_reserve(ses.model, batch.n_steps, batch.n_tokens)
    if args.deterministic is not None:
        B.cs_set_deterministic(ses.model, bool(args.deterministic))
    stream = torch.cuda.current_stream()
    K, W = args.steps, max(3, args.warmup)
    counts = work_counts(cfg, batch)

    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(local).uuid).replace("GPU-", ""))
    sampler.start()
    for _ in range(W):
        ses.verify()
    torch.cuda.synchronize()

    # ---- device-resident throughput -------------------------------------------------------------
    # The K-step timed loop is repeated so that the whole timed region lasts seconds: the median repeat is the
    # reported number (the best one is given beside it) and the clock sampler sees the GPU under the power state that
    # the loop settles into, not the first milliseconds after idle.
    def timed_loop():
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        torch.cuda.synchronize()
        ev0.record(stream)
        for _ in range(K):
            ses.verify()
        ev1.record(stream)
        torch.cuda.synchronize()
        barrier()
        return ev0.elapsed_time(ev1)

    B.cs_take_launch_count()
    first = timed_loop()
    launches = B.cs_take_launch_count()            # of one K-step loop
    repeats = max(10, min(400, int(np.ceil(args.min_seconds * 1e3 / max(first, 1e-3)))))
    if world > 1:                                  # every rank must run the same number of loops
        r = torch.tensor([repeats], dtype=torch.int64, device="cuda")
        dist.all_reduce(r, op=dist.ReduceOp.MAX)
        repeats = int(r.item())
    t_wall0 = time.time()
    loop_ms = [timed_loop() for _ in range(repeats)]
    t_wall1 = time.time()
    ms = float(np.median(loop_ms))
    ms_best = float(np.min(loop_ms))
    B.cs_last_status(ses.model)

    # ---- end to end: host tokens in, results read back on the host, every step ---------------------
    conf_host = torch.empty(batch.n_steps, dtype=torch.float32).pin_memory()
    acc_host = torch.empty(batch.n_steps, dtype=torch.uint8).pin_memory()
    for _ in range(2):
        ses.verify(host_tokens=True)
    torch.cuda.synchronize()
    barrier()
    e2e_ms = []
    for _ in range(5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(K):
            ses.verify(host_tokens=True)
            conf_host.copy_(ses.out_conf, non_blocking=True)
            acc_host.copy_(ses.out_accept, non_blocking=True)
            stream.synchronize()                      # the caller reads the mask before its next step
        e1.record(stream)
        torch.cuda.synchronize()
        barrier()
        e2e_ms.append(e0.elapsed_time(e1))
    ms_e2e = float(np.median(e2e_ms))
    h2d_bytes = B.cs_last_h2d_bytes(ses.model)     # tokens + batch metadata, one pinned block per call

    # ---- per-kernel durations (events around every launch; same workload, same process) -------------
    # Read back after every K-step loop (the event pool is reused); repeated like the timed loop, with the clocks
    # sampled over this region on their own, since these are the times the per-kernel roofline figures come from.
    B.cs_profile(ses.model, True)
    prof = None
    t_prof0 = time.time()
    for _ in range(max(3, repeats // 3)):
        for _ in range(K):
            ses.verify()
        torch.cuda.synchronize()
        part = B.cs_profile_read(ses.model)
        prof = part if prof is None else {k: (prof[k][0] + v[0], prof[k][1] + v[1]) for k, v in part.items()}
    t_prof1 = time.time()
    B.cs_profile(ses.model, False)
    sampler.stop()
    clocks = sampler.summary(t_wall0, t_wall1)
    clocks_prof = sampler.summary(t_prof0, t_prof1)

    ms, ms_e2e, all_steps, all_tokens = aggregate_over_ranks(
        ms, ms_e2e, batch.n_steps, batch.n_tokens, device="cuda" if world > 1 else None)

    # Peaks: fp16 and bf16 share the tensor peak. Two measured figures exist: the burst one (cuBLAS timed alone, near
    # the full clock) and the sustained one (seconds of back-to-back GEMMs under the power cap, ~1.3 GHz). Fractions
    # are given against the burst figure - the stricter one - with the sustained reading beside it, and each time also
    # as time x median SM clock so that runs at different clocks can be compared.
    peaks, peak_kind = load_peaks()
    tensor_peak = float(peaks["bf16_tflops"])
    tensor_peak_sus = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    hbm_peak = float(peaks["hbm_gbs"])

    def per_launch_ms(name):
        t_ms, n = prof[name]
        return t_ms / n if n else float("nan")

    L = cfg.model.n_layers
    gu_ms = per_launch_ms("gemm_gateup")
    gu_tf = counts["gemm_gateup_flops"] / (gu_ms * 1e-3) / 1e12
    kernels = {}
    for name, flops in (("gemm_qkv", counts["gemm_qkv_flops"]), ("gemm_o", counts["gemm_o_flops"]),
                        ("gemm_gateup", counts["gemm_gateup_flops"]), ("gemm_down", counts["gemm_down_flops"])):
        t_ms = per_launch_ms(name)
        kernels[name] = {"ms_per_launch": t_ms, "tflops": flops / (t_ms * 1e-3) / 1e12,
                         "frac_tensor": flops / (t_ms * 1e-3) / 1e12 / tensor_peak,
                         "frac_tensor_sustained": flops / (t_ms * 1e-3) / 1e12 / tensor_peak_sus}
    a_ms = per_launch_ms("attention")
    kernels["attention"] = {"ms_per_launch": a_ms, "tflops": counts["attention_flops"] / (a_ms * 1e-3) / 1e12,
                            "frac_tensor": counts["attention_flops"] / (a_ms * 1e-3) / 1e12 / tensor_peak,
                            "frac_tensor_sustained": counts["attention_flops"] / (a_ms * 1e-3) / 1e12 / tensor_peak_sus,
                            "gbs": counts["attention_bytes"] / (a_ms * 1e-3) / 1e9,
                            "frac_hbm": counts["attention_bytes"] / (a_ms * 1e-3) / 1e9 / hbm_peak}
    l_ms = per_launch_ms("lm_head")
    kernels["lm_head"] = {"ms_per_launch": l_ms, "gbs": counts["lm_head_bytes"] / (l_ms * 1e-3) / 1e9,
                          "frac_hbm": counts["lm_head_bytes"] / (l_ms * 1e-3) / 1e9 / hbm_peak}
    back_to_back = projections_back_to_back(cfg, counts["T"], tensor_peak, tensor_peak_sus) if world == 1 else None
    prof_total = sum(v[0] for v in prof.values())
    shares = {k: (v[0] / prof_total if prof_total else 0.0) for k, v in prof.items()}
    all_gemm_flops = sum(counts[k] for k in ("gemm_qkv_flops", "gemm_o_flops", "gemm_gateup_flops", "gemm_down_flops"))
    all_gemm_ms = sum(kernels[k]["ms_per_launch"] for k in ("gemm_qkv", "gemm_o", "gemm_gateup", "gemm_down"))
    kernels["gemm_all_four"] = {"ms_per_layer": all_gemm_ms, "tflops": all_gemm_flops / (all_gemm_ms * 1e-3) / 1e12,
                                "frac_tensor": all_gemm_flops / (all_gemm_ms * 1e-3) / 1e12 / tensor_peak,
                                "frac_tensor_sustained": all_gemm_flops / (all_gemm_ms * 1e-3) / 1e12 / tensor_peak_sus}

    # Whole step against its own roofline: every kernel at the bound that binds it (projections: tensor peak;
    # attention: the slower of its flops at tensor peak and its bytes at copy bandwidth; LM head: its bytes).
    def step_roofline_ms(tp):
        per_layer = all_gemm_flops / (tp * 1e12) + max(counts["attention_flops"] / (tp * 1e12),
                                                       counts["attention_bytes"] / (hbm_peak * 1e9))
        return 1e3 * (L * per_layer + counts["lm_head_bytes"] / (hbm_peak * 1e9))

    step_ms = ms / K
    whole = {"algorithmic_ms": step_roofline_ms(tensor_peak), "algorithmic_ms_sustained": step_roofline_ms(tensor_peak_sus),
             "measured_ms": step_ms}
    whole["frac"] = whole["algorithmic_ms"] / step_ms
    whole["frac_sustained"] = whole["algorithmic_ms_sustained"] / step_ms
    mhz = clocks.get("sm_mhz")
    mhz_prof = clocks_prof.get("sm_mhz")

    out = {
        "metric": METRIC, "value": all_steps * K / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16", "data": "synthetic",
        "tokens_per_s": all_tokens * K / (ms * 1e-3),
        "timing": {"repeats": repeats, "steps_per_repeat": K, "reported": "median repeat", "ms_per_step_median": ms / K,
                   "ms_per_step_best": ms_best / K, "ms_per_step_worst": float(np.max(loop_ms)) / K,
                   "ms_x_sm_mhz": (ms / K * mhz) if mhz else None},
        "whole_step": whole,
        "config": {"workload": cfg.name, "model": cfg.model.name, "layers": cfg.model.n_layers, "batch": cfg.batch, "new_tokens": counts["T"],
                   "ctx_tokens": int(batch.ctx_lens.sum()), "tau": cfg.tau, "page_size": cfg.page_size,
                   "l2": "inputs larger than L2 (3.1 GB of weights streamed every step)",
                   "last_layer": "MLP half on each step's last row only (no other row reaches the LM head); its small "
                                 "launches are timed under 'other', not in the per-launch projection figures",
                   "replicas": world,
                   "deterministic": ("library default (bit-identical passes)" if args.deterministic is None
                                     else bool(args.deterministic))},
        "clocks": clocks,
        "clocks_per_kernel_run": clocks_prof,
        "e2e": {"value": all_steps * K / (ms_e2e * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": int(h2d_bytes),
                "d2h_bytes_per_step": int(batch.n_steps * 5), "ms_per_step": ms_e2e / K},
        "gpu_launches": int(launches),
        "roofline": {"kernel": "gemm_f16_kernel<256, SwiGLU> (gate/up projection)", "bound": "tensor",
                     "achieved": gu_tf, "peak": tensor_peak, "unit": "TFLOP/s", "frac": gu_tf / tensor_peak,
                     "peak_kind": f"{peak_kind} bf16 burst (fp16 has the same nominal peak)",
                     "peak_sustained": tensor_peak_sus, "frac_sustained": gu_tf / tensor_peak_sus,
                     "ms_x_sm_mhz": (gu_ms * mhz_prof) if mhz_prof else None,
                     "traffic": (gateup_traffic(cfg.name) if args.layers is None else None), "traffic_unit": "bytes per launch (DRAM read + write, ncu)",
                     "ms_per_launch": gu_ms, "launches_timed": prof["gemm_gateup"][1]},
        "kernels": kernels,
        "kernels_back_to_back": back_to_back,
        "kernels_note": "kernels: one event pair around EVERY launch of the pass (serialises the launches, ~3 us on each); "
                        "kernels_back_to_back: 40 launches of the same kernel and shape under one event pair",
        "time_shares": shares,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample = list(range(min(6, batch.n_steps)))         # ~15 s of CPU work at the 1.5B shape
        t = oracle_sample_run(cfg, weights, batch, sample)
        out["cpu_baseline"] = {"value": len(sample) / t, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                               "sample": f"one oracle pass over steps {sample} of the {batch.n_steps}-step batch "
                                         f"({t:.1f} s, context K/V generation included)"}
    ses.close()
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def run_cascade(args):
    """Times cs_verify_cascade (draft pass, list of escalated steps, target pass over those steps, final decision)
    on one GPU, host tokens in and the blocking read-back of the list inside the timed region, next to its two
    tiers timed alone: the cost model of Section 4.4 predicts t(draft) + t(target on the escalated steps).
    Both models get the planted verdict rows, otherwise every confidence is ~1/V and every step is escalated."""
    import torch
    from paper_2602_18447_b200 import VerifySession, binding as B
    from paper_2602_18447_b200.runner import CascadeSession
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the pass has no CPU path")
    torch.cuda.set_device(0)
    casc = get_cascade(args.cascade, target_layers=args.layers)
    batch = make_batch(casc.draft)
    tiers = []
    for cfg in (casc.draft, casc.target):
        w = model_weights(cfg.model, cfg.seed)
        plant_verdict_rows(w, cfg.verdict_ids, beta=float(np.log(cfg.model.vocab) + 0.5), seed=cfg.seed)
        ses = VerifySession(cfg, w, batch)
        del w
        total, pages = page_assignment(cfg, batch.ctx_lens)
        if cfg.ctx_kv == "prefill":
            ses.alloc_cache(pages, total, batch.ctx_lens, room_for_prefill=True)
            ses.prefill_context(batch.ctx_tokens)
        else:
            ses.alloc_cache(pages, total, batch.ctx_lens)
            ses.fill_synthetic_context(lambda i, l, cfg=cfg: context_kv(cfg, i, l, int(batch.ctx_lens[i])))
        B.cs_reserve(ses.model, batch.n_steps, batch.n_tokens)
        tiers.append(ses)
    cs = CascadeSession(*tiers)
    tau = casc.draft.tau if args.tau is None else args.tau
    stream = torch.cuda.current_stream()
    K, W = args.steps, max(3, args.warmup)

    def timed(fn):
        for _ in range(W):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(K):
            fn()
            stream.synchronize()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / K

    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(0).uuid).replace("GPU-", ""))
    sampler.start()
    B.cs_take_launch_count()
    t0 = time.time()
    ms = timed(lambda: cs.verify(tau=tau))
    t1 = time.time()
    launches = B.cs_take_launch_count() // (K + W)
    n_esc = cs.n_escalated
    res = cs.results()
    ms_draft = timed(lambda: cs.draft.verify(tau=tau, host_tokens=True))
    ms_target_all = timed(lambda: cs.target.verify(tau=tau, host_tokens=True))
    # the target alone on exactly the escalated steps
    esc = np.nonzero(res["trusted"] == 0)[0]
    ms_target_esc = 0.0
    if esc.size:
        toks = np.concatenate([batch.step_tokens[batch.cu_new[i]:batch.cu_new[i + 1]] for i in esc]).astype(np.int32)
        lens = batch.step_lens[esc].astype(np.int32)
        oc = torch.empty(esc.size, dtype=torch.float32, device="cuda")
        oa = torch.empty(esc.size, dtype=torch.uint8, device="cuda")
        t = cs.target
        ms_target_esc = timed(lambda: B.cs_verify_steps(t.model, t.kv, esc.astype(np.int32), toks, lens,
                                                        casc.draft.verdict_ids, tau, oc, oa, None))
    sampler.stop()
    out = {
        "metric": METRIC, "value": batch.n_steps / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": W,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16",
        "data": "synthetic",
        "config": {"workload": casc.name, "draft": casc.draft.model.name, "target": casc.target.model.name,
                   "batch": batch.n_steps, "new_tokens": int(batch.n_tokens), "ctx_tokens": int(batch.ctx_lens.sum()),
                   "tau": tau, "n_escalated": int(n_esc), "cascade_rate": n_esc / batch.n_steps,
                   "timing": "host tokens in, list of escalated steps read back between the tiers, host waits for "
                             "the final decisions every step",
                   "l2": "inputs larger than L2 (both models' weights streamed every step)"},
        "tiers_ms": {"cascade": ms, "draft_alone": ms_draft, "target_alone_all_steps": ms_target_all,
                     "target_alone_escalated_steps": ms_target_esc,
                     "draft_plus_target_escalated": ms_draft + ms_target_esc},
        "gpu_launches": int(launches), "clocks": sampler.summary(t0, t1),
    }
    cs.close()
    print(json.dumps(out))


def replica_command(n: int, argv, port: int):
    """The launch line for N replicas, one process per GPU: this same file under torch.distributed.run."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def spawn_replicas(n: int, argv) -> int:
    """`python bench.py --gpus N` without a launcher: start the N processes here and hand back their exit status.
    Rank 0 of the children prints the one JSON line."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    return subprocess.run(replica_command(n, list(argv), port)).returncode


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--deterministic", type=int, default=None, choices=[0, 1],
                    help="cs_set_deterministic for the timed model (default: the library's default, which is 1)")
    ap.add_argument("--min-seconds", type=float, default=2.5,
                    help="the K-step timed loop is repeated (at least 10 times) until the timed region lasts this long")
    ap.add_argument("--layers", type=int, default=None,
                    help="run a reduced-depth copy of the workload (for profiler captures of single kernels); "
                         "not a benchmark configuration")
    ap.add_argument("--cascade", default=None,
                    help="time the two-tier pass of this cascade workload instead (one GPU; with --layers the target "
                         "model runs at that depth)")
    ap.add_argument("--tau", type=float, default=None, help="threshold of the two-tier pass (default: the workload's)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.cascade is None:
        sys.exit(spawn_replicas(args.gpus, sys.argv[1:]))
    if args.cascade is not None:
        run_cascade(args)
        return
    cfg = get_config(args.workload)
    if args.layers is not None:
        cfg = scaled_config(args.workload, n_layers=args.layers)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
