"""Convenience wrapper: one layer's compressed cache with the device buffers it needs.
Plumbing only (torch allocations, host->device copies of the caller's arrays); every computation is
a call into libhkv through `binding`."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as hkv


def to_device_bf16(bits: np.ndarray, device="cuda", stream_pinned: bool = False) -> torch.Tensor:
    """uint16 bf16 bit patterns (host) -> bf16 CUDA tensor holding the same bytes."""
    t = torch.from_numpy(np.ascontiguousarray(bits))
    if stream_pinned:
        t = t.pin_memory()
    return t.to(device, non_blocking=stream_pinned).view(torch.bfloat16)


class LayerCache:
    """Compresses one layer's K/V on construction and serves decode steps.

    L: any object with the fields of hkv_inputs.LayerInputs (host numpy arrays)."""

    def __init__(self, L, flags: int = 0, token_scores: np.ndarray | None = None, softmax_scale: float = 0.0,
                 device="cuda", keep_workspace: bool = False, k_dev=None, v_dev=None, append_capacity: int = 0):
        self.cfg = hkv.make_config(L.batch, L.n_q_heads, L.n_kv_heads, L.head_dim, L.max_seq_len, L.chunk_size,
                                   L.obs_window, softmax_scale, flags, append_capacity)
        self.flags = flags
        self.shape = (L.batch, L.n_q_heads, L.head_dim)
        self.device = device
        self.host_mem = None
        if flags & hkv.HKV_OFFLOAD_DYNAMIC:
            cache_bytes, ws_bytes, host_bytes = hkv.hkv_plan_offload(self.cfg, L.seq_lens, L.head_type, L.budgets)
            if host_bytes:
                # 256-byte aligned slice of a pinned buffer the device addresses at the same pointer value
                raw = torch.empty(host_bytes + 256, dtype=torch.uint8, pin_memory=True)
                skip = (-raw.data_ptr()) % 256
                self.host_mem = raw[skip:skip + host_bytes]
        else:
            cache_bytes, ws_bytes = hkv.hkv_plan(self.cfg, L.seq_lens, L.head_type, L.budgets)
        self.cache_mem = torch.empty(cache_bytes, dtype=torch.uint8, device=device)
        workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=device)
        k = k_dev if k_dev is not None else to_device_bf16(L.k, device)
        v = v_dev if v_dev is not None else to_device_bf16(L.v, device)
        q_obs = to_device_bf16(L.q_obs, device)
        is_text = torch.from_numpy(np.ascontiguousarray(L.is_text)).to(device)
        ts = None
        if token_scores is not None:
            ts = torch.from_numpy(np.ascontiguousarray(token_scores, dtype=np.float32)).to(device)
        if flags & hkv.HKV_OFFLOAD_DYNAMIC:
            self.handle = hkv.hkv_compress_offload(self.cfg, k, v, q_obs, ts, is_text, L.seq_lens, L.head_type,
                                                   L.budgets, self.cache_mem, self.host_mem, workspace)
        else:
            self.handle = hkv.hkv_compress(self.cfg, k, v, q_obs, ts, is_text, L.seq_lens, L.head_type, L.budgets,
                                           self.cache_mem, workspace)
        self.workspace = workspace if keep_workspace else None
        if not keep_workspace:
            torch.cuda.current_stream().synchronize()   # inputs and workspace are released below
        self.stats = hkv.hkv_cache_stats(self.handle)

    def new_out(self) -> torch.Tensor:
        dt = torch.float32 if self.flags & hkv.HKV_OUT_F32 else torch.bfloat16
        return torch.empty(self.shape, dtype=dt, device=self.device)

    def decode(self, q: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
        if out is None:
            out = self.new_out()
        hkv.hkv_decode_attn(self.handle, q, out)
        return out

    def append(self, k_new: torch.Tensor, v_new: torch.Tensor) -> None:
        """Adds the new token's key / value ([B, Hkv, d] bf16 CUDA tensors) to the cache."""
        hkv.hkv_append(self.handle, k_new, v_new)
        self.stats = hkv.hkv_cache_stats(self.handle)

    def window_scores(self, b: int, h: int, C: int) -> np.ndarray:
        """float32 s_w the compression computed (needs keep_workspace=True)."""
        off = hkv.hkv_window_scores_offset(self.handle, b, h)
        torch.cuda.synchronize()
        return self.workspace[off:off + 4 * C].view(torch.float32).cpu().numpy()

    def close(self):
        if self.handle:
            hkv.hkv_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
