"""ctypes binding of libhkv.so: the same entry points as include/hkv.h, argument marshalling only.

Device tensors are torch CUDA tensors (torch provides device memory and streams, nothing else);
host tables are numpy arrays.  Every step of the path runs in the library's CUDA kernels; there is
no fallback: importing this module without a built library raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libhkv.so")

HKV_OK = 0
HKV_CAUSAL_WINDOW = 1
HKV_OUT_F32 = 2
HKV_GROUP_MAX = 4
HKV_OFFLOAD_DYNAMIC = 8

STATUS_NAMES = {0: "HKV_OK", 1: "HKV_ERR_INVALID_ARG", 2: "HKV_ERR_SHAPE", 3: "HKV_ERR_BUDGET",
                4: "HKV_ERR_WORKSPACE", 5: "HKV_ERR_UNSUPPORTED", 6: "HKV_ERR_CUDA", 7: "HKV_ERR_TIMEOUT",
                8: "HKV_ERR_INDEX"}

EXPORTS = ["hkv_plan", "hkv_compress", "hkv_decode_attn", "hkv_decode_attn_multi", "hkv_select_chunks",
           "hkv_attend", "hkv_decode_attn_host", "hkv_cache_destroy",
           "hkv_get_static_indices", "hkv_get_selected_chunks", "hkv_get_chunk_scores", "hkv_get_summaries",
           "hkv_window_scores_offset", "hkv_cache_stats", "hkv_last_device_error", "hkv_status_string",
           "hkv_topk_chunks_noalloc", "hkv_decode_cluster_capacity", "hkv_allocate_budgets", "hkv_append", "hkv_decode_step_host",
           "hkv_classify_workspace", "hkv_classify_heads", "hkv_plan_offload", "hkv_compress_offload"]


class hkv_config(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("max_seq_len", C.c_int32), ("chunk_size", C.c_int32),
                ("obs_window", C.c_int32), ("softmax_scale", C.c_float), ("flags", C.c_uint32),
                ("append_capacity", C.c_int32)]


class hkv_stats(C.Structure):
    _fields_ = [("retained_tokens", C.c_int64), ("kv_bytes_resident", C.c_int64), ("summary_bytes", C.c_int64),
                ("algorithmic_bytes_per_step", C.c_int64), ("cache_bytes", C.c_int64),
                ("workspace_bytes", C.c_int64), ("n_static", C.c_int32), ("n_dynamic", C.c_int32),
                ("n_splits", C.c_int32), ("launches_per_decode", C.c_int32)]

    def as_dict(self):
        return {f: int(getattr(self, f)) for f, _ in self._fields_}


class HkvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {STATUS_NAMES.get(int(status), status)} ({status_string(status)})")


def _load(path: str = _LIB_PATH) -> C.CDLL:
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2604_05887_b200.build` "
            "(or __graft_entry__.build()); there is no fallback path")
    lib = C.CDLL(path)
    vp, i32p, u8p = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_uint8)
    cfgp = C.POINTER(hkv_config)
    lib.hkv_plan.argtypes = [cfgp, i32p, u8p, i32p, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    lib.hkv_compress.argtypes = [cfgp, vp, vp, vp, vp, vp, i32p, u8p, i32p, vp, C.c_size_t, vp, C.c_size_t, vp,
                                 C.POINTER(vp)]
    lib.hkv_plan_offload.argtypes = [cfgp, i32p, u8p, i32p, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t),
                                     C.POINTER(C.c_size_t)]
    lib.hkv_compress_offload.argtypes = [cfgp, vp, vp, vp, vp, vp, i32p, u8p, i32p, vp, C.c_size_t, vp, C.c_size_t,
                                         vp, C.c_size_t, vp, C.POINTER(vp)]
    lib.hkv_decode_attn.argtypes = [vp, vp, vp, vp]
    lib.hkv_decode_attn_multi.argtypes = [C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.c_int32, vp]
    lib.hkv_select_chunks.argtypes = [vp, vp, vp]
    lib.hkv_attend.argtypes = [vp, vp, vp, vp]
    lib.hkv_decode_attn_host.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.hkv_cache_destroy.argtypes = [vp]
    lib.hkv_decode_step_host.argtypes = [C.POINTER(vp), C.c_int32, vp, vp, vp, vp, vp]
    lib.hkv_append.argtypes = [vp, vp, vp, vp]
    for name in ("hkv_get_static_indices", "hkv_get_selected_chunks"):
        getattr(lib, name).argtypes = [vp, C.c_int32, C.c_int32, i32p, C.c_int32, i32p, vp]
    lib.hkv_get_chunk_scores.argtypes = [vp, C.c_int32, C.c_int32, C.POINTER(C.c_float), C.c_int32, i32p, vp]
    lib.hkv_get_summaries.argtypes = [vp, C.c_int32, C.c_int32, C.POINTER(C.c_uint16), C.c_int32, i32p, vp]
    lib.hkv_window_scores_offset.argtypes = [vp, C.c_int32, C.c_int32, C.POINTER(C.c_size_t)]
    lib.hkv_cache_stats.argtypes = [vp, C.POINTER(hkv_stats)]
    lib.hkv_last_device_error.argtypes = [vp, i32p, i32p, vp]
    lib.hkv_topk_chunks_noalloc.argtypes = [vp, vp, C.c_int32, C.c_int32, C.c_int32, vp, vp]
    lib.hkv_decode_cluster_capacity.argtypes = [C.c_int32, i32p]
    lib.hkv_allocate_budgets.argtypes = [C.c_int32, u8p, C.POINTER(C.c_double), C.c_int64, C.c_double, C.c_double,
                                         C.c_uint32, i32p]
    lib.hkv_classify_workspace.argtypes = [C.POINTER(hkv_config), C.c_int32, C.POINTER(C.c_size_t),
                                           C.POINTER(C.c_size_t)]
    lib.hkv_classify_heads.argtypes = [C.POINTER(hkv_config), vp, vp, C.c_int32, i32p, i32p, C.c_double, C.c_double,
                                       vp, C.c_size_t, vp, vp, vp]
    lib.hkv_status_string.argtypes = [C.c_int]
    lib.hkv_status_string.restype = C.c_char_p
    for name in EXPORTS:
        if name != "hkv_status_string":
            getattr(lib, name).restype = C.c_int
    return lib


lib = _load()


def use_library(path: Optional[str] = None) -> C.CDLL:
    """Point every wrapper of this module at another build of the same library (build.build_checked(),
    build.build_profile()); None goes back to the product library.  Handles made by one build must be
    used and destroyed with that build."""
    global lib
    lib = _load(path or _LIB_PATH)
    return lib


def status_string(status: int) -> str:
    return lib.hkv_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != HKV_OK:
        raise HkvError(status, where)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.int32)


def _u8(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.uint8)


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def _dev(t) -> Optional[int]:
    """Device address of a torch CUDA tensor (None stays NULL)."""
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if hasattr(stream, "cuda_stream"):
        return stream.cuda_stream or None
    return int(stream) or None


def make_config(batch, n_q_heads, n_kv_heads, head_dim, max_seq_len, chunk_size, obs_window,
                softmax_scale: float = 0.0, flags: int = 0, append_capacity: int = 0) -> hkv_config:
    return hkv_config(batch, n_q_heads, n_kv_heads, head_dim, max_seq_len, chunk_size, obs_window,
                      softmax_scale, flags, append_capacity)


def hkv_plan(cfg: hkv_config, seq_lens, head_type, budgets):
    """-> (cache_bytes, workspace_bytes); host arithmetic only."""
    sl, ht, bu = _i32(seq_lens), _u8(head_type), _i32(budgets)
    cb, wb = C.c_size_t(0), C.c_size_t(0)
    _check(lib.hkv_plan(C.byref(cfg), _ptr(sl, C.c_int32), _ptr(ht, C.c_uint8), _ptr(bu, C.c_int32),
                        C.byref(cb), C.byref(wb)), "hkv_plan")
    return int(cb.value), int(wb.value)


def hkv_compress(cfg: hkv_config, k, v, q_obs, token_scores, is_text, seq_lens, head_type, budgets,
                 cache_mem, workspace, stream=None) -> int:
    """Enqueue the compression of one layer; returns the cache handle (an integer address).
    k, v, q_obs, token_scores, is_text, cache_mem, workspace: torch CUDA tensors (or None)."""
    sl, ht, bu = _i32(seq_lens), _u8(head_type), _i32(budgets)
    handle = C.c_void_p(None)
    _check(lib.hkv_compress(C.byref(cfg), _dev(k), _dev(v), _dev(q_obs), _dev(token_scores), _dev(is_text),
                            _ptr(sl, C.c_int32), _ptr(ht, C.c_uint8), _ptr(bu, C.c_int32),
                            _dev(cache_mem), cache_mem.numel() * cache_mem.element_size(),
                            _dev(workspace), workspace.numel() * workspace.element_size(),
                            _stream(stream), C.byref(handle)), "hkv_compress")
    return handle.value


def hkv_plan_offload(cfg: hkv_config, seq_lens, head_type, budgets):
    """-> (cache_bytes, workspace_bytes, host_bytes) for the variant with the dynamic heads' K/V in host memory."""
    sl, ht, bu = _i32(seq_lens), _u8(head_type), _i32(budgets)
    cb, wb, hb = C.c_size_t(0), C.c_size_t(0), C.c_size_t(0)
    _check(lib.hkv_plan_offload(C.byref(cfg), _ptr(sl, C.c_int32), _ptr(ht, C.c_uint8), _ptr(bu, C.c_int32),
                                C.byref(cb), C.byref(wb), C.byref(hb)), "hkv_plan_offload")
    return int(cb.value), int(wb.value), int(hb.value)


def hkv_compress_offload(cfg: hkv_config, k, v, q_obs, token_scores, is_text, seq_lens, head_type, budgets,
                         cache_mem, host_mem, workspace, stream=None) -> int:
    """hkv_compress with the dynamic heads' K/V planes written to `host_mem`, a pinned CPU tensor (or None when
    the layer has no dynamic head)."""
    sl, ht, bu = _i32(seq_lens), _u8(head_type), _i32(budgets)
    handle = C.c_void_p(None)
    if host_mem is not None and (host_mem.is_cuda or not host_mem.is_pinned() or not host_mem.is_contiguous()):
        raise ValueError("expected a contiguous pinned CPU tensor")
    hp = host_mem.data_ptr() if host_mem is not None else None
    hn = host_mem.numel() * host_mem.element_size() if host_mem is not None else 0
    _check(lib.hkv_compress_offload(C.byref(cfg), _dev(k), _dev(v), _dev(q_obs), _dev(token_scores), _dev(is_text),
                                    _ptr(sl, C.c_int32), _ptr(ht, C.c_uint8), _ptr(bu, C.c_int32),
                                    _dev(cache_mem), cache_mem.numel() * cache_mem.element_size(), hp, hn,
                                    _dev(workspace), workspace.numel() * workspace.element_size(),
                                    _stream(stream), C.byref(handle)), "hkv_compress_offload")
    return handle.value


def hkv_decode_attn(cache: int, q, out, stream=None) -> None:
    _check(lib.hkv_decode_attn(cache, _dev(q), _dev(out), _stream(stream)), "hkv_decode_attn")


def hkv_decode_attn_multi(caches: Sequence[int], qs, outs, stream=None) -> None:
    n = len(caches)
    arr = C.c_void_p * n
    _check(lib.hkv_decode_attn_multi(arr(*caches), arr(*[_dev(t) for t in qs]), arr(*[_dev(t) for t in outs]),
                                     n, _stream(stream)), "hkv_decode_attn_multi")


def hkv_select_chunks(cache: int, q, stream=None) -> None:
    _check(lib.hkv_select_chunks(cache, _dev(q), _stream(stream)), "hkv_select_chunks")


def hkv_attend(cache: int, q, out, stream=None) -> None:
    _check(lib.hkv_attend(cache, _dev(q), _dev(out), _stream(stream)), "hkv_attend")


def hkv_decode_attn_host(cache: int, q_host, out_host, q_dev, out_dev, stream=None) -> None:
    """q_host / out_host: CPU torch tensors (pinned for asynchronous copies); q_dev / out_dev: CUDA staging."""
    if q_host.is_cuda or out_host.is_cuda or not q_host.is_contiguous() or not out_host.is_contiguous():
        raise ValueError("q_host and out_host must be contiguous CPU tensors")
    _check(lib.hkv_decode_attn_host(cache, q_host.data_ptr(), out_host.data_ptr(), _dev(q_dev), _dev(out_dev),
                                    _stream(stream)), "hkv_decode_attn_host")


def hkv_decode_step_host(caches: Sequence[int], q_host, out_host, q_dev, out_dev, stream=None) -> None:
    """One decode step over all layers with host buffers [n, B, Hq, d] (see hkv.h)."""
    n = len(caches)
    if q_host.is_cuda or out_host.is_cuda or not q_host.is_contiguous() or not out_host.is_contiguous():
        raise ValueError("q_host and out_host must be contiguous CPU tensors")
    _check(lib.hkv_decode_step_host((C.c_void_p * n)(*caches), n, q_host.data_ptr(), out_host.data_ptr(), _dev(q_dev),
                                    _dev(out_dev), _stream(stream)), "hkv_decode_step_host")


HKV_NOALLOC_MAX_CHUNKS = 65536


def hkv_topk_chunks_noalloc(q, means, k: int, out_ids, stream=None) -> None:
    """Top-k chunks of one dynamic head with the library's built-in score scratch (no allocation).
    q: bf16 CUDA [group, 128]; means: bf16 CUDA [n_chunks, 128] plain row-major; out_ids: int32 CUDA [min(k, n_chunks)]."""
    _check(lib.hkv_topk_chunks_noalloc(_dev(q), _dev(means), int(q.shape[0]), int(means.shape[0]), int(k),
                                       _dev(out_ids), _stream(stream)), "hkv_topk_chunks_noalloc")


def hkv_append(cache: int, k_new, v_new, stream=None) -> None:
    """k_new, v_new: bf16 CUDA [B, Hkv, d], the new token's key / value of every KV head."""
    _check(lib.hkv_append(cache, _dev(k_new), _dev(v_new), _stream(stream)), "hkv_append")


def hkv_cache_destroy(cache: int) -> None:
    _check(lib.hkv_cache_destroy(cache), "hkv_cache_destroy")


def _get_ints(fn, name, cache, b, h, stream):
    n = C.c_int32(0)
    probe = np.zeros(1, dtype=np.int32)
    st = fn(cache, b, h, _ptr(probe, C.c_int32), 0, C.byref(n), _stream(stream))
    if st not in (HKV_OK, 4):
        raise HkvError(st, name)
    out = np.zeros(max(int(n.value), 1), dtype=np.int32)
    _check(fn(cache, b, h, _ptr(out, C.c_int32), out.size, C.byref(n), _stream(stream)), name)
    return out[:n.value].copy()


def hkv_get_static_indices(cache: int, b: int, h: int, stream=None) -> np.ndarray:
    return _get_ints(lib.hkv_get_static_indices, "hkv_get_static_indices", cache, b, h, stream)


def hkv_get_selected_chunks(cache: int, b: int, h: int, stream=None) -> np.ndarray:
    return _get_ints(lib.hkv_get_selected_chunks, "hkv_get_selected_chunks", cache, b, h, stream)


def hkv_get_chunk_scores(cache: int, b: int, h: int, n_chunks: int, stream=None) -> np.ndarray:
    out = np.zeros(max(n_chunks, 1), dtype=np.float32)
    n = C.c_int32(0)
    _check(lib.hkv_get_chunk_scores(cache, b, h, _ptr(out, C.c_float), out.size, C.byref(n), _stream(stream)),
           "hkv_get_chunk_scores")
    return out[:n.value].copy()


def hkv_get_summaries(cache: int, b: int, h: int, n_chunks: int, head_dim: int = 128, stream=None) -> np.ndarray:
    out = np.zeros((max(n_chunks, 1), head_dim), dtype=np.uint16)
    n = C.c_int32(0)
    _check(lib.hkv_get_summaries(cache, b, h, _ptr(out, C.c_uint16), out.shape[0], C.byref(n), _stream(stream)),
           "hkv_get_summaries")
    return out[:n.value].copy()


def hkv_window_scores_offset(cache: int, b: int, h: int) -> int:
    off = C.c_size_t(0)
    _check(lib.hkv_window_scores_offset(cache, b, h, C.byref(off)), "hkv_window_scores_offset")
    return int(off.value)


def hkv_decode_cluster_capacity(group: int) -> dict:
    """{cluster size: clusters of the decode kernel the current device holds at once}."""
    out = np.zeros(16, dtype=np.int32)
    _check(lib.hkv_decode_cluster_capacity(int(group), _ptr(out, C.c_int32)), "hkv_decode_cluster_capacity")
    return {i + 1: int(out[i]) for i in range(16)}


HKV_BUDGET_PAD_POW2 = 1


def hkv_allocate_budgets(head_type, scores, total_budget: int, r: float, alpha: float, flags: int = 0) -> np.ndarray:
    """Per-head token budgets from a total budget (host arithmetic; see hkv.h)."""
    ht = _u8(head_type).ravel()
    out = np.zeros(ht.size, dtype=np.int32)
    sp = None
    if scores is not None:
        sc = np.ascontiguousarray(np.asarray(scores, dtype=np.float64).ravel())
        sp = _ptr(sc, C.c_double)
    _check(lib.hkv_allocate_budgets(ht.size, _ptr(ht, C.c_uint8), sp, int(total_budget), float(r), float(alpha),
                                    int(flags), _ptr(out, C.c_int32)), "hkv_allocate_budgets")
    return out


def hkv_classify_workspace(cfg: hkv_config, n_text_max: int):
    """(min_bytes, preferred_bytes) of the workspace hkv_classify_heads takes."""
    lo, hi = C.c_size_t(0), C.c_size_t(0)
    _check(lib.hkv_classify_workspace(C.byref(cfg), int(n_text_max), C.byref(lo), C.byref(hi)),
           "hkv_classify_workspace")
    return int(lo.value), int(hi.value)


def hkv_classify_heads(cfg: hkv_config, k, q_text, seq_lens, n_text, topk_fraction: float, theta: float,
                       workspace, scores_out, head_type_out, stream=None):
    """Text-centric sparsity score and static / dynamic label of every (sequence, kv head); see hkv.h.
    k, q_text, workspace, scores_out (float64) and head_type_out (uint8) are CUDA tensors."""
    sl, nt = _i32(seq_lens), _i32(n_text)
    _check(lib.hkv_classify_heads(C.byref(cfg), k.data_ptr(), q_text.data_ptr(), int(q_text.shape[1]),
                                  _ptr(sl, C.c_int32), _ptr(nt, C.c_int32), float(topk_fraction), float(theta),
                                  workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                  scores_out.data_ptr(), head_type_out.data_ptr(), _stream(stream)),
           "hkv_classify_heads")


def hkv_cache_stats(cache: int) -> dict:
    st = hkv_stats()
    _check(lib.hkv_cache_stats(cache, C.byref(st)), "hkv_cache_stats")
    return st.as_dict()


def hkv_last_device_error(cache: int, stream=None):
    code, detail = C.c_int32(0), C.c_int32(0)
    _check(lib.hkv_last_device_error(cache, C.byref(code), C.byref(detail), _stream(stream)),
           "hkv_last_device_error")
    return int(code.value), int(detail.value)
