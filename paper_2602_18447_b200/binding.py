"""ctypes binding of libconfspec.so: argument marshalling only, every step of the path runs in the CUDA
library. Function names match the C ABI declared in include/confspec.h. There is no fallback: if the library
is missing or a call fails, an exception is raised."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

from . import build as _build

CS_OK, CS_EINVAL, CS_ENOMEM, CS_ECUDA, CS_ETIMEOUT, CS_ESTATE, CS_ELIMIT, CS_ERANGE = range(8)

EXPORTED = [
    "cs_version", "cs_strerror", "cs_last_cuda_error", "cs_model_load", "cs_model_free", "cs_model_set_lm_head_rows",
    "cs_reserve",
    "cs_kv_alloc", "cs_kv_alloc_8bit", "cs_kv_free", "cs_kv_pool_bytes", "cs_kv_set_seq", "cs_kv_fill", "cs_prefill",
    "cs_verify_steps", "cs_verify_cascade", "cs_append_accepted", "cs_escalate_mask", "cs_cascade_select", "cs_set_keep_logits", "cs_set_deterministic", "cs_get_last_logits", "cs_get_last_lse",
    "cs_last_status", "cs_selftest_wait_timeout", "cs_debug_build", "cs_selftest_range_check", "cs_check_workspace", "cs_gemm_f16", "cs_rmsnorm", "cs_lm_head_gate", "cs_lm_head_gate_static", "cs_take_launch_count", "cs_last_h2d_bytes", "cs_profile", "cs_profile_read",
]

PROF_CLASSES = ["embed", "rmsnorm", "gemm_qkv", "rope", "attention", "gemm_o", "gemm_gateup", "gemm_down",
                "lm_head", "gate", "other"]


class ConfSpecError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: status {status}" + (f" ({detail})" if detail else ""))


class cs_model_desc(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ffn", C.c_int32), ("vocab", C.c_int32),
                ("rope_theta", C.c_float), ("rms_eps", C.c_float)]


_PP = C.POINTER(C.c_void_p)


class cs_model_tensors(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("wq", _PP), ("wk", _PP), ("wv", _PP), ("wo", _PP), ("wg", _PP), ("wu", _PP), ("wd", _PP),
                ("norm1", _PP), ("norm2", _PP), ("q_norm", _PP), ("k_norm", _PP)]


_lib: Optional[C.CDLL] = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """dlopen the in-tree library and declare its signatures. Raises if it has not been built."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or _build.LIB_PATH
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} not found: build it with `python -m paper_2602_18447_b200.build` (there is no CPU fallback)")
    lib = C.CDLL(path)
    vp, i32, f32 = C.c_void_p, C.c_int, C.c_float
    sig = {
        "cs_version": (C.c_int, []),
        "cs_strerror": (C.c_char_p, [i32]),
        "cs_last_cuda_error": (C.c_char_p, []),
        "cs_model_load": (C.c_int, [C.POINTER(cs_model_desc), C.POINTER(cs_model_tensors), i32, C.POINTER(vp)]),
        "cs_model_free": (C.c_int, [vp]),
        "cs_model_set_lm_head_rows": (C.c_int, [vp, vp, i32, vp, vp]),
        "cs_reserve": (C.c_int, [vp, i32, i32]),
        "cs_kv_alloc": (C.c_int, [vp, i32, i32, i32, i32, vp, C.POINTER(vp)]),
        "cs_kv_alloc_8bit": (C.c_int, [vp, i32, i32, i32, i32, i32, C.POINTER(vp)]),
        "cs_kv_free": (C.c_int, [vp]),
        "cs_kv_pool_bytes": (C.c_uint64, [vp, i32, i32]),
        "cs_kv_set_seq": (C.c_int, [vp, i32, vp, i32, i32]),
        "cs_kv_fill": (C.c_int, [vp, i32, i32, vp, vp, vp]),
        "cs_prefill": (C.c_int, [vp, vp, vp, vp, vp, i32, vp]),
        "cs_verify_steps": (C.c_int, [vp, vp, vp, i32, vp, i32, vp, vp, i32, f32, vp, vp, vp, vp]),
        "cs_verify_cascade": (C.c_int, [vp, vp, vp, vp, vp, i32, vp, vp, vp, i32, f32, vp, vp, vp, vp, vp, vp, vp, vp, i32,
                                        i32, vp, vp]),
        "cs_append_accepted": (C.c_int, [vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp]),
        "cs_escalate_mask": (C.c_int, [vp, i32, f32, vp, vp, vp, vp]),
        "cs_cascade_select": (C.c_int, [vp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp]),
        "cs_set_keep_logits": (C.c_int, [vp, i32]),
        "cs_set_deterministic": (C.c_int, [vp, i32]),
        "cs_get_last_logits": (C.c_int, [vp, vp, i32, vp]),
        "cs_get_last_lse": (C.c_int, [vp, vp, i32, vp]),
        "cs_last_status": (C.c_int, [vp, vp]),
        "cs_selftest_wait_timeout": (C.c_int, [vp, i32, vp]),
        "cs_debug_build": (C.c_int, []),
        "cs_selftest_range_check": (C.c_int, [vp, vp]),
        "cs_check_workspace": (C.c_int, [vp, vp]),
        "cs_gemm_f16": (C.c_int, [vp, vp, vp, vp, i32, i32, i32, i32, vp]),
        "cs_rmsnorm": (C.c_int, [vp, vp, vp, i32, i32, f32, vp]),
        "cs_lm_head_gate": (C.c_int, [vp, vp, i32, i32, i32, vp, i32, f32, vp, vp, vp, vp, vp]),
        "cs_lm_head_gate_static": (C.c_int, [vp, vp, i32, i32, i32, vp, i32, f32, vp, vp, vp, vp, vp]),
        "cs_take_launch_count": (C.c_int64, []),
        "cs_last_h2d_bytes": (C.c_int64, [vp]),
        "cs_profile": (C.c_int, [vp, i32]),
        "cs_profile_read": (C.c_int, [vp, vp, vp, i32]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)   # AttributeError if the symbol is not exported
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _check(status: int, where: str) -> None:
    if status != CS_OK:
        lib = load_library()
        detail = lib.cs_strerror(status).decode()
        if status in (CS_ECUDA, CS_ENOMEM):
            detail += ": " + lib.cs_last_cuda_error().decode()
        raise ConfSpecError(status, where, detail)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _np_ptr(a: Optional[np.ndarray]) -> Optional[int]:
    return None if a is None else a.ctypes.data


def _dev_ptr(t) -> Optional[int]:
    """Device address of a torch CUDA tensor (or a raw int address, or None)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def cs_version() -> int:
    return load_library().cs_version()


def cs_last_h2d_bytes(model: int) -> int:
    return int(load_library().cs_last_h2d_bytes(model))


def cs_take_launch_count() -> int:
    return int(load_library().cs_take_launch_count())


def cs_model_load(shape, weights: dict) -> int:
    """Load host weights (numpy uint16 bf16 bit patterns / float32 gains, the layout of
    workloads.model_weights) and return the model handle."""
    lib = load_library()
    desc = cs_model_desc(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                         shape.d_ffn, shape.vocab, shape.rope_theta, shape.rms_eps)
    keep = []
    qk = "q_norm" in weights["layers"][0]

    def mat(a, dtype):
        a = np.ascontiguousarray(a, dtype=dtype)
        keep.append(a)
        return a.ctypes.data

    def per_layer(name, dtype):
        arr = (C.c_void_p * shape.n_layers)(*[mat(l[name], dtype) for l in weights["layers"]])
        keep.append(arr)
        return C.cast(arr, _PP)

    t = cs_model_tensors(mat(weights["embed"], np.uint16), mat(weights["lm_head"], np.uint16),
                         mat(weights["final_norm"], np.float32),
                         per_layer("wq", np.uint16), per_layer("wk", np.uint16), per_layer("wv", np.uint16),
                         per_layer("wo", np.uint16), per_layer("wg", np.uint16), per_layer("wu", np.uint16),
                         per_layer("wd", np.uint16), per_layer("norm1", np.float32), per_layer("norm2", np.float32),
                         per_layer("q_norm", np.float32) if qk else None, per_layer("k_norm", np.float32) if qk else None)
    out = C.c_void_p()
    _check(lib.cs_model_load(C.byref(desc), C.byref(t), 0, C.byref(out)), "cs_model_load")
    return out.value


def cs_model_free(model: int) -> None:
    _check(load_library().cs_model_free(model), "cs_model_free")


def cs_model_set_lm_head_rows(model: int, row_ids, rows_bf16: np.ndarray, stream=None) -> None:
    """rows_bf16: uint16 bf16 bit patterns [n_rows, d_model] (host)."""
    ids = _i32(row_ids)
    rows = np.ascontiguousarray(rows_bf16, dtype=np.uint16)
    if rows.ndim != 2 or rows.shape[0] != ids.shape[0]:
        raise ValueError("rows_bf16 must be [n_rows, d_model]")
    _check(load_library().cs_model_set_lm_head_rows(model, _np_ptr(ids), int(ids.shape[0]), _np_ptr(rows),
                                                    _stream_ptr(stream)), "cs_model_set_lm_head_rows")


def cs_reserve(model: int, max_steps: int, max_tokens: int) -> None:
    _check(load_library().cs_reserve(model, max_steps, max_tokens), "cs_reserve")


def cs_kv_pool_bytes(model: int, num_pages: int, page_size: int = 16) -> int:
    return int(load_library().cs_kv_pool_bytes(model, num_pages, page_size))


def cs_kv_alloc(model: int, num_pages: int, page_size: int, max_seqs: int, max_pages_per_seq: int,
                dev_pool=None) -> int:
    out = C.c_void_p()
    _check(load_library().cs_kv_alloc(model, num_pages, page_size, max_seqs, max_pages_per_seq,
                                      _dev_ptr(dev_pool), C.byref(out)), "cs_kv_alloc")
    return out.value


CS_KV_E4M3, CS_KV_E5M2 = 1, 2


def cs_kv_alloc_8bit(model: int, num_pages: int, page_size: int, max_seqs: int, max_pages_per_seq: int,
                     fmt: str = "e4m3") -> int:
    out = C.c_void_p()
    code = {"e4m3": CS_KV_E4M3, "e5m2": CS_KV_E5M2}[fmt]
    _check(load_library().cs_kv_alloc_8bit(model, num_pages, page_size, max_seqs, max_pages_per_seq, code,
                                           C.byref(out)), "cs_kv_alloc_8bit")
    return out.value


def cs_kv_free(kv: int) -> None:
    _check(load_library().cs_kv_free(kv), "cs_kv_free")


def cs_kv_set_seq(kv: int, seq: int, page_ids, ctx_len: int) -> None:
    p = _i32(page_ids)
    _check(load_library().cs_kv_set_seq(kv, seq, _np_ptr(p), int(p.shape[0]), int(ctx_len)), "cs_kv_set_seq")


def cs_kv_fill(kv: int, seq: int, layer: int, host_k: np.ndarray, host_v: np.ndarray, stream=None) -> None:
    """uint16 arrays (bf16 patterns) for a 16-bit cache, uint8 arrays (codes) for a cache from cs_kv_alloc_8bit."""
    dt = np.uint8 if np.asarray(host_k).dtype == np.uint8 else np.uint16
    k = np.ascontiguousarray(host_k, dtype=dt)
    v = np.ascontiguousarray(host_v, dtype=dt)
    _check(load_library().cs_kv_fill(kv, seq, layer, _np_ptr(k), _np_ptr(v), _stream_ptr(stream)), "cs_kv_fill")


def cs_prefill(model: int, kv: int, seq_ids, tokens, lens, stream=None) -> None:
    s, t, l = _i32(seq_ids), _i32(tokens), _i32(lens)
    _check(load_library().cs_prefill(model, kv, _np_ptr(s), _np_ptr(t), _np_ptr(l), int(s.shape[0]),
                                     _stream_ptr(stream)), "cs_prefill")


def cs_verify_steps(model: int, ctx_kv: int, seq_ids, step_tokens, step_lens, verdict_ids: Sequence[int],
                    tau: float, out_conf, out_accept, out_verdict=None, stream=None) -> None:
    """step_tokens: a host int32 array (numpy, or a pinned CPU torch tensor) or a CUDA int32 tensor.
    out_conf (float32), out_accept (uint8), out_verdict (int32 or None): CUDA tensors of length B."""
    s, l, v = _i32(seq_ids), _i32(step_lens), _i32(verdict_ids)
    on_dev = 0
    if hasattr(step_tokens, "is_cuda"):
        if step_tokens.is_cuda:
            on_dev, tok_ptr = 1, _dev_ptr(step_tokens)
        else:
            tok_ptr = step_tokens.data_ptr()
    else:
        step_tokens = _i32(step_tokens)
        tok_ptr = _np_ptr(step_tokens)
    _check(load_library().cs_verify_steps(model, ctx_kv, _np_ptr(s), int(s.shape[0]), tok_ptr, on_dev, _np_ptr(l),
                                          _np_ptr(v), int(v.shape[0]), float(tau), _dev_ptr(out_conf),
                                          _dev_ptr(out_accept), _dev_ptr(out_verdict), _stream_ptr(stream)),
           "cs_verify_steps")


def cs_verify_cascade(draft: int, kv_d: int, target: int, kv_t: int, seq_ids, step_tokens, step_lens,
                      verdict_ids: Sequence[int], tau: float, out_conf_d, out_trusted, out_verdict_d, out_conf_t,
                      out_verdict_t, out_verdict, out_conf, req_offsets=None, accept_index: int = 0, stream=None) -> int:
    """step_tokens: host int32 (numpy or a CPU torch tensor). The out_* are CUDA tensors of length B (out_conf_t and
    out_verdict_t may be None). req_offsets (host int32 [R+1]) turns on the linear-drafting rule. Returns the number
    of steps sent to the target model."""
    s, l, v = _i32(seq_ids), _i32(step_lens), _i32(verdict_ids)
    if hasattr(step_tokens, "is_cuda"):
        if step_tokens.is_cuda:
            raise ValueError("cs_verify_cascade takes the step tokens in host memory")
        tok_ptr = step_tokens.data_ptr()
    else:
        step_tokens = _i32(step_tokens)
        tok_ptr = _np_ptr(step_tokens)
    n_esc = C.c_int32(0)
    ro = None if req_offsets is None else _i32(req_offsets)
    _check(load_library().cs_verify_cascade(draft, kv_d, target, kv_t, _np_ptr(s), int(s.shape[0]), tok_ptr, _np_ptr(l),
                                            _np_ptr(v), int(v.shape[0]), float(tau), _dev_ptr(out_conf_d),
                                            _dev_ptr(out_trusted), _dev_ptr(out_verdict_d), _dev_ptr(out_conf_t),
                                            _dev_ptr(out_verdict_t), _dev_ptr(out_verdict), _dev_ptr(out_conf),
                                            None if ro is None else _np_ptr(ro), 0 if ro is None else int(ro.shape[0]) - 1,
                                            int(accept_index), C.cast(C.byref(n_esc), C.c_void_p), _stream_ptr(stream)),
           "cs_verify_cascade")
    return int(n_esc.value)


def cs_append_accepted(model: int, kv: int, req_seq_ids, req_offsets, prefix_len, step_tokens, step_lens, draft_lens,
                       stream=None) -> np.ndarray:
    """prefix_len: CUDA int32 tensor [R] (out_prefix_len of cs_cascade_select); the other arrays are host int32.
    Returns the prefix lengths that were read back."""
    q, o, t = _i32(req_seq_ids), _i32(req_offsets), _i32(step_tokens)
    l, d = _i32(step_lens), _i32(draft_lens)
    R = int(q.shape[0])
    got = np.zeros(max(R, 1), dtype=np.int32)
    _check(load_library().cs_append_accepted(model, kv, R, _np_ptr(q), _np_ptr(o), _dev_ptr(prefix_len), _np_ptr(t),
                                             _np_ptr(l), _np_ptr(d), _np_ptr(got), _stream_ptr(stream)),
           "cs_append_accepted")
    return got[:R]


def cs_escalate_mask(conf, tau: float, out_accept, out_escalate_idx, out_escalate_count, stream=None) -> None:
    _check(load_library().cs_escalate_mask(_dev_ptr(conf), int(conf.shape[0]), float(tau), _dev_ptr(out_accept),
                                           _dev_ptr(out_escalate_idx), _dev_ptr(out_escalate_count),
                                           _stream_ptr(stream)), "cs_escalate_mask")


def cs_cascade_select(trusted, verdict_d, conf_d, verdict_t, conf_t, req_offsets, accept_index: int, out_prefix_len,
                      out_best, out_pass=None, out_conf=None, stream=None) -> None:
    """All arguments are CUDA tensors (verdict_t / conf_t / out_pass / out_conf may be None); req_offsets int32 [R+1]."""
    _check(load_library().cs_cascade_select(_dev_ptr(trusted), _dev_ptr(verdict_d), _dev_ptr(conf_d), _dev_ptr(verdict_t),
                                            _dev_ptr(conf_t), _dev_ptr(req_offsets), int(req_offsets.shape[0]) - 1,
                                            int(accept_index), _dev_ptr(out_prefix_len), _dev_ptr(out_best),
                                            _dev_ptr(out_pass), _dev_ptr(out_conf), _stream_ptr(stream)),
           "cs_cascade_select")


def cs_set_keep_logits(model: int, keep: bool) -> None:
    _check(load_library().cs_set_keep_logits(model, 1 if keep else 0), "cs_set_keep_logits")


def cs_set_deterministic(model: int, on: bool) -> None:
    _check(load_library().cs_set_deterministic(model, 1 if on else 0), "cs_set_deterministic")


def cs_get_last_logits(model: int, out, B: int, stream=None) -> None:
    _check(load_library().cs_get_last_logits(model, _dev_ptr(out), B, _stream_ptr(stream)), "cs_get_last_logits")


def cs_get_last_lse(model: int, out, B: int, stream=None) -> None:
    _check(load_library().cs_get_last_lse(model, _dev_ptr(out), B, _stream_ptr(stream)), "cs_get_last_lse")


def cs_last_status(model: int, stream=None) -> None:
    _check(load_library().cs_last_status(model, _stream_ptr(stream)), "cs_last_status")


def cs_selftest_wait_timeout(model: int, polls: int = 4096, stream=None) -> None:
    _check(load_library().cs_selftest_wait_timeout(model, int(polls), _stream_ptr(stream)), "cs_selftest_wait_timeout")


def cs_debug_build() -> bool:
    return bool(load_library().cs_debug_build())


def cs_selftest_range_check(model: int, stream=None) -> None:
    _check(load_library().cs_selftest_range_check(model, _stream_ptr(stream)), "cs_selftest_range_check")


def cs_check_workspace(model: int, stream=None) -> None:
    _check(load_library().cs_check_workspace(model, _stream_ptr(stream)), "cs_check_workspace")


def cs_gemm_f16(a, w, w2, out, M: int, N: int, K: int, epilogue: int, stream=None) -> None:
    _check(load_library().cs_gemm_f16(_dev_ptr(a), _dev_ptr(w), _dev_ptr(w2), _dev_ptr(out), M, N, K, epilogue,
                                       _stream_ptr(stream)), "cs_gemm_f16")


def cs_lm_head_gate(w_lm, h, verdict_ids: Sequence[int], tau: float, out_conf, out_accept, out_verdict=None,
                    out_lse=None, stream=None, entry: str = "cs_lm_head_gate") -> None:
    """w_lm: CUDA fp16 [vocab, d]; h: CUDA fp16 [B, d]; outputs: CUDA tensors of B entries."""
    v = _i32(verdict_ids)
    fn = getattr(load_library(), entry)
    _check(fn(_dev_ptr(w_lm), _dev_ptr(h), int(h.shape[0]), int(h.shape[1]), int(w_lm.shape[0]), _np_ptr(v),
              int(v.shape[0]), float(tau), _dev_ptr(out_conf), _dev_ptr(out_accept), _dev_ptr(out_verdict),
              _dev_ptr(out_lse), _stream_ptr(stream)), entry)


def cs_lm_head_gate_static(w_lm, h, verdict_ids: Sequence[int], tau: float, out_conf, out_accept, out_verdict=None,
                           out_lse=None, stream=None) -> None:
    """Same stage through the entry point that never allocates device memory (at most 64 steps per call; calls that
    overlap on the GPU share one scratch array and race: keep them on one stream)."""
    cs_lm_head_gate(w_lm, h, verdict_ids, tau, out_conf, out_accept, out_verdict, out_lse, stream,
                    entry="cs_lm_head_gate_static")


def cs_rmsnorm(x, gain, out, rows: int, d: int, eps: float, stream=None) -> None:
    _check(load_library().cs_rmsnorm(_dev_ptr(x), _dev_ptr(gain), _dev_ptr(out), rows, d, float(eps),
                                     _stream_ptr(stream)), "cs_rmsnorm")


def cs_profile(model: int, enable: bool) -> None:
    _check(load_library().cs_profile(model, 1 if enable else 0), "cs_profile")


def cs_profile_read(model: int) -> dict:
    """{class name: (milliseconds, timed launches)} since profiling was enabled or last read."""
    n = len(PROF_CLASSES)
    ms = np.zeros(n, dtype=np.float32)
    calls = np.zeros(n, dtype=np.int32)
    _check(load_library().cs_profile_read(model, _np_ptr(ms), _np_ptr(calls), n), "cs_profile_read")
    return {name: (float(ms[i]), int(calls[i])) for i, name in enumerate(PROF_CLASSES)}
