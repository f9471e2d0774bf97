"""HybridKV decode hot path for NVIDIA B200: C-ABI CUDA library (libhkv.so) and its thin binding.

    from paper_2604_05887_b200 import binding as hkv
    cache_bytes, ws_bytes = hkv.hkv_plan(cfg, seq_lens, head_type, budgets)
    handle = hkv.hkv_compress(cfg, k, v, q_obs, None, is_text, seq_lens, head_type, budgets, cache_mem, ws)
    hkv.hkv_decode_attn(handle, q, out)

`layer.py` adds a small convenience wrapper that owns the device buffers of one layer's cache.
"""
