"""Seeded synthetic inputs for the HybridKV decode hot path.

This module is the one thing shared by the CPU oracle's tests and the CUDA path's tests and
benchmark.  It only *draws inputs*: token layouts (text / visual modality masks), K / V / query
tensors as raw bf16 bit patterns, per-head types and per-head token budgets.  It contains none of
the method's arithmetic (no attention, no scoring, no selection, no chunk means).

All tensors are numpy arrays; bf16 tensors are ``uint16`` arrays holding the bit patterns, so that
both sides see identical bytes and no side depends on the other's rounding.

Randomness is counter based: every (seed, layer, tensor, batch index, kv head) plane has its own
Philox key, so the bytes do not depend on thread count or on generation order.

The five workload recipes follow the five benchmark configurations (Qwen2.5-VL-7B head geometry:
28 query heads, 4 KV heads, head_dim 128):

* ``cfg0``  1 layer, B=1, 2048 tokens = 64 text + 1920 visual + 64 text, N(0,1) with 4 outlier
  channels x8, 2 static / 2 dynamic heads, budget 10 %, chunk 32.
* ``cfg1``  28 layers, B=1, 16384 tokens in an image-block layout (1024-token visual blocks between
  16-token text spans), static fraction 0.5, budget 10 %, chunk 32, 8 decode steps.
* ``cfg2``  28 layers, B=4, up to 32768 tokens, video-like: 64 frames x (11 text + 500 visual),
  keys = per-frame mean N(0, 0.5) + N(0,1) noise, lengths 24K-32K, static fraction 0.6, chunk 64.
* ``cfg3``  28 layers, B=8, 50000 tokens, static fraction 0.4, budget 5 %, chunk 32, three planted
  key chunks per dynamic head with decode queries at cosine ~0.6 to the planted direction.
* ``cfg4``  1 layer, B=16, 32768 tokens, a sweep cell (budget, static fraction, chunk size).

Every recipe accepts size overrides so that tests can build small cases of the same structure.
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

N_Q_HEADS = 28
N_KV_HEADS = 4
HEAD_DIM = 128
OBS_WINDOW = 32

# tensor ids for the Philox key
_T_K, _T_V, _T_QOBS, _T_Q, _T_MISC, _T_MEAN, _T_DIR, _T_QTEXT = range(8)


# --------------------------------------------------------------------------------------------
# bf16 bit helpers (input formatting only)
# --------------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16 bit patterns (uint16). Inputs are finite."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(u: np.ndarray) -> np.ndarray:
    """Exact bf16 bit patterns -> float32."""
    return (np.asarray(u, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, layer: int, tensor: int, b: int = 0, h: int = 0) -> np.random.Generator:
    key0 = (int(seed) & 0xFFFFFFFF) | ((int(layer) & 0xFFFFFFFF) << 32)
    key1 = (int(tensor) & 0xFFFF) | ((int(b) & 0xFFFFFF) << 16) | ((int(h) & 0xFFFFFF) << 40)
    return np.random.Generator(np.random.Philox(key=[key0, key1]))


# --------------------------------------------------------------------------------------------
# token layouts: is_text masks
# --------------------------------------------------------------------------------------------
def layout_sandwich(n_text_head: int, n_visual: int, n_text_tail: int) -> np.ndarray:
    """text prefix + one visual span + text query."""
    m = np.zeros(n_text_head + n_visual + n_text_tail, dtype=np.uint8)
    m[:n_text_head] = 1
    m[n_text_head + n_visual:] = 1
    return m


def layout_image_blocks(C: int, block: int = 1024, span: int = 16, tail: int = 64) -> np.ndarray:
    """span text, then [block visual][span text] while at least block+span+tail tokens remain,
    then one shorter visual block, then `tail` text tokens."""
    m = np.zeros(C, dtype=np.uint8)
    pos = 0
    n = min(span, max(C - tail, 0))
    m[pos:pos + n] = 1
    pos += n
    while C - pos >= block + span + tail:
        pos += block
        m[pos:pos + span] = 1
        pos += span
    m[max(C - tail, pos):] = 1
    return m


def layout_video(n_frames: int, frame_visual: int = 500, frame_text: int = 11, edge_text: int = 32):
    """edge text + n_frames x (frame_text text + frame_visual visual) + edge text.
    Returns (is_text, frame_id) with frame_id = -1 on text-only edges."""
    per = frame_text + frame_visual
    C = 2 * edge_text + n_frames * per
    m = np.zeros(C, dtype=np.uint8)
    fid = np.full(C, -1, dtype=np.int32)
    m[:edge_text] = 1
    m[C - edge_text:] = 1
    for f in range(n_frames):
        s = edge_text + f * per
        m[s:s + frame_text] = 1
        fid[s:s + per] = f
    return m, fid


# --------------------------------------------------------------------------------------------
# workload container
# --------------------------------------------------------------------------------------------
@dataclass
class LayerInputs:
    """One layer's inputs.  bf16 tensors are uint16 bit patterns."""
    name: str
    layer: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    max_seq_len: int
    chunk_size: int
    obs_window: int
    seq_lens: np.ndarray            # int32 [B]
    is_text: np.ndarray             # uint8 [B, C_max]
    head_type: np.ndarray           # uint8 [B, Hkv]  0 = static, 1 = dynamic
    budgets: np.ndarray             # int32 [B, Hkv]  tokens
    k: np.ndarray                   # uint16 [B, Hkv, C_max, d]
    v: np.ndarray                   # uint16 [B, Hkv, C_max, d]
    q_obs: np.ndarray               # uint16 [B, w, Hq, d]  queries of the last w prompt tokens
    q: List[np.ndarray] = field(default_factory=list)   # decode queries, each uint16 [B, Hq, d]
    planted: Optional[np.ndarray] = None                # int32 [B, Hkv, 3] planted chunk ids or -1

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


def _normal_bits(rng: np.random.Generator, shape) -> np.ndarray:
    return f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))


def _choose_static(seed: int, layer: int, B: int, Hkv: int, static_fraction: float) -> np.ndarray:
    """Exactly round(f * B * Hkv) of the (b, h) pairs are static, by a seeded permutation."""
    n = B * Hkv
    n_static = int(math.floor(static_fraction * n + 0.5))
    perm = _rng(seed, layer, _T_MISC, 1).permutation(n)
    ht = np.ones(n, dtype=np.uint8)
    ht[perm[:n_static]] = 0
    return ht.reshape(B, Hkv)


def _budget_tokens(fraction: float, seq_lens: np.ndarray, Hkv: int) -> np.ndarray:
    b = np.array([max(1, int(math.ceil(fraction * int(c) - 1e-9))) for c in seq_lens], dtype=np.int32)
    return np.repeat(b[:, None], Hkv, axis=1).astype(np.int32)


def _fill_planes(fn, B: int, Hkv: int, threads: int):
    jobs = [(b, h) for b in range(B) for h in range(Hkv)]
    if threads <= 1:
        for j in jobs:
            fn(*j)
        return
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(lambda j: fn(*j), jobs))


def _make_layer(name, seed, layer, B, C_max, seq_lens, is_text, chunk_size, static_fraction,
                budget_fraction, n_steps, kv_fn, q_fn=None, Hq=N_Q_HEADS, Hkv=N_KV_HEADS,
                d=HEAD_DIM, w=OBS_WINDOW, threads=8, head_type=None) -> LayerInputs:
    seq_lens = np.asarray(seq_lens, dtype=np.int32)
    k = np.zeros((B, Hkv, C_max, d), dtype=np.uint16)
    v = np.zeros((B, Hkv, C_max, d), dtype=np.uint16)

    def plane(b, h):
        kb, vb = kv_fn(b, h, int(seq_lens[b]))
        k[b, h, :seq_lens[b]] = kb
        v[b, h, :seq_lens[b]] = vb

    _fill_planes(plane, B, Hkv, threads)
    q_obs = _normal_bits(_rng(seed, layer, _T_QOBS), (B, w, Hq, d))
    if head_type is None:
        head_type = _choose_static(seed, layer, B, Hkv, static_fraction)
    budgets = _budget_tokens(budget_fraction, seq_lens, Hkv)
    L = LayerInputs(name=name, layer=layer, batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d,
                    max_seq_len=C_max, chunk_size=chunk_size, obs_window=w, seq_lens=seq_lens,
                    is_text=is_text, head_type=np.asarray(head_type, dtype=np.uint8), budgets=budgets,
                    k=k, v=v, q_obs=q_obs)
    for s in range(n_steps):
        if q_fn is None:
            L.q.append(_normal_bits(_rng(seed, layer, _T_Q, s), (B, Hq, d)))
        else:
            L.q.append(q_fn(s, L))
    return L


def _outlier_kv(seed, layer, d, n_out=4, scale=8.0):
    """K, V ~ N(0,1) with `n_out` channels (same for K and V of a head) scaled by `scale`."""
    def fn(b, h, C):
        ch = _rng(seed, layer, _T_MISC, b + 2, h).choice(d, size=n_out, replace=False)
        out = []
        for t in (_T_K, _T_V):
            x = _rng(seed, layer, t, b, h).standard_normal((C, d), dtype=np.float32)
            x[:, ch] *= np.float32(scale)
            out.append(f32_to_bf16_bits(x))
        return out
    return fn


# --------------------------------------------------------------------------------------------
# the five recipes
# --------------------------------------------------------------------------------------------
def cfg0(seed: int = 0, n_text: int = 64, n_visual: int = 1920, chunk_size: int = 32,
         budget_fraction: float = 0.10, n_steps: int = 1, layer: int = 0, threads: int = 4,
         head_type=None, **geom) -> LayerInputs:
    m = layout_sandwich(n_text, n_visual, n_text)
    C = m.size
    d = geom.get("d", HEAD_DIM)
    return _make_layer("cfg0", seed, layer, 1, C, [C], m[None, :].copy(), chunk_size, 0.5,
                       budget_fraction, n_steps, _outlier_kv(seed, layer, d), threads=threads,
                       head_type=head_type, **geom)


def cfg1(layer: int, seed: int = 1, C: int = 16384, block: int = 1024, chunk_size: int = 32,
         budget_fraction: float = 0.10, static_fraction: float = 0.5, n_steps: int = 8,
         threads: int = 8, **geom) -> LayerInputs:
    m = layout_image_blocks(C, block=block)
    d = geom.get("d", HEAD_DIM)

    def kv(b, h, Cb):
        return (_normal_bits(_rng(seed, layer, _T_K, b, h), (Cb, d)),
                _normal_bits(_rng(seed, layer, _T_V, b, h), (Cb, d)))
    return _make_layer("cfg1", seed, layer, 1, C, [C], m[None, :].copy(), chunk_size,
                       static_fraction, budget_fraction, n_steps, kv, threads=threads, **geom)


def cfg2(layer: int, seed: int = 2, B: int = 4, n_frames: int = 64, min_frames: int = 48,
         frame_visual: int = 500, chunk_size: int = 64, budget_fraction: float = 0.10,
         static_fraction: float = 0.6, n_steps: int = 1, threads: int = 8, **geom) -> LayerInputs:
    d = geom.get("d", HEAD_DIM)
    full_mask, full_fid = layout_video(n_frames, frame_visual)
    C_max = full_mask.size
    # sequence 0 has all frames; the others drop trailing frames (same lengths in every layer)
    fr = _rng(seed, 0, _T_MISC, 7).integers(min_frames, n_frames + 1, size=B)
    fr[0] = n_frames
    is_text = np.zeros((B, C_max), dtype=np.uint8)
    fids, seq_lens = [], []
    for b in range(B):
        mb, fb = layout_video(int(fr[b]), frame_visual)
        is_text[b, :mb.size] = mb
        fids.append(fb)
        seq_lens.append(mb.size)

    def kv(b, h, Cb):
        mu = _rng(seed, layer, _T_MEAN, b, h).standard_normal((n_frames, d), dtype=np.float32)
        mu *= np.float32(math.sqrt(0.5))
        x = _rng(seed, layer, _T_K, b, h).standard_normal((Cb, d), dtype=np.float32)
        fb = fids[b]
        vis = fb >= 0
        x[vis] += mu[fb[vis]]
        return (f32_to_bf16_bits(x), _normal_bits(_rng(seed, layer, _T_V, b, h), (Cb, d)))
    return _make_layer("cfg2", seed, layer, B, C_max, seq_lens, is_text, chunk_size, static_fraction,
                       budget_fraction, n_steps, kv, threads=threads, **geom)


def cfg3(layer: int, seed: int = 3, B: int = 8, C: int = 50000, block: int = 1024,
         chunk_size: int = 32, budget_fraction: float = 0.05, static_fraction: float = 0.4,
         n_steps: int = 1, rho: float = 0.6, amp: float = 4.0, threads: int = 8, **geom) -> LayerInputs:
    d = geom.get("d", HEAD_DIM)
    Hq = geom.get("Hq", N_Q_HEADS)
    Hkv = geom.get("Hkv", N_KV_HEADS)
    G = Hq // Hkv
    m = layout_image_blocks(C, block=block)
    n_chunks = (C + chunk_size - 1) // chunk_size
    head_type = _choose_static(seed, layer, B, Hkv, static_fraction)
    planted = np.full((B, Hkv, 3), -1, dtype=np.int32)
    dirs = np.zeros((B, Hkv, d), dtype=np.float32)
    for b in range(B):
        for h in range(Hkv):
            u = _rng(seed, layer, _T_DIR, b, h).standard_normal(d, dtype=np.float32)
            dirs[b, h] = u / np.linalg.norm(u)
            if head_type[b, h] == 1:
                planted[b, h] = np.sort(_rng(seed, layer, _T_MISC, b + 100, h)
                                        .choice(n_chunks, size=3, replace=False)).astype(np.int32)

    def kv(b, h, Cb):
        x = _rng(seed, layer, _T_K, b, h).standard_normal((Cb, d), dtype=np.float32)
        for c in planted[b, h]:
            if c >= 0:
                s, e = int(c) * chunk_size, min((int(c) + 1) * chunk_size, Cb)
                x[s:e] += np.float32(amp) * dirs[b, h][None, :]
        return (f32_to_bf16_bits(x), _normal_bits(_rng(seed, layer, _T_V, b, h), (Cb, d)))

    def qf(step, L):
        n = _rng(seed, layer, _T_Q, step).standard_normal((B, Hq, d), dtype=np.float32)
        u = np.repeat(dirs, G, axis=1)                      # [B, Hq, d]
        q = np.float32(rho * math.sqrt(d)) * u + np.float32(math.sqrt(1.0 - rho * rho)) * n
        return f32_to_bf16_bits(q)

    L = _make_layer("cfg3", seed, layer, B, C, [C] * B, np.repeat(m[None, :], B, axis=0), chunk_size,
                    static_fraction, budget_fraction, n_steps, kv, q_fn=qf, threads=threads,
                    head_type=head_type, **geom)
    L.planted = planted
    return L


def cfg4(budget_fraction: float, static_fraction: float, chunk_size: int, seed: int = 4, B: int = 16,
         C: int = 32768, block: int = 1024, n_steps: int = 1, layer: int = 0, threads: int = 8,
         **geom) -> LayerInputs:
    m = layout_image_blocks(C, block=block)
    d = geom.get("d", HEAD_DIM)
    return _make_layer("cfg4", seed, layer, B, C, [C] * B, np.repeat(m[None, :], B, axis=0),
                       chunk_size, static_fraction, budget_fraction, n_steps,
                       _outlier_kv(seed, layer, d), threads=threads, **geom)


CFG4_BUDGETS = (0.05, 0.10, 0.20, 0.50, 1.00)
CFG4_STATIC_FRACTIONS = (0.0, 0.25, 0.5, 0.75, 1.0)
CFG4_CHUNKS = (16, 32, 64, 128)


def tiny(seed: int = 11, B: int = 2, C: int = 96, chunk_size: int = 8, w: int = 4, Hq: int = 4,
         Hkv: int = 2, d: int = 16, budget_fraction: float = 0.25, n_steps: int = 1,
         ragged: bool = True, head_type=None) -> LayerInputs:
    """A very small case with free geometry, for brute-force checks of the oracle."""
    seq_lens = [C - (5 * b if ragged else 0) for b in range(B)]
    is_text = np.zeros((B, C), dtype=np.uint8)
    for b in range(B):
        is_text[b, :seq_lens[b]] = layout_image_blocks(seq_lens[b], block=24, span=3, tail=w + 2)

    def kv(b, h, Cb):
        return (_normal_bits(_rng(seed, 0, _T_K, b, h), (Cb, d)),
                _normal_bits(_rng(seed, 0, _T_V, b, h), (Cb, d)))
    return _make_layer("tiny", seed, 0, B, C, seq_lens, is_text, chunk_size, 0.5, budget_fraction,
                       n_steps, kv, Hq=Hq, Hkv=Hkv, d=d, w=w, threads=1, head_type=head_type)


def text_queries(L: LayerInputs, n_text: int, seed: int = 5, gain: float = 1.5, n_anchor: int = 4,
                 ragged: bool = True):
    """Queries of the prompt's text tokens for head classification: (q_text uint16 [B, n_text, Hq, d],
    counts int32 [B]).  Every kv head gets a focus level in [0, 1] (cycling 0, 1/3, 2/3, 1 over b * Hkv + h):
    its text queries are N(0,1) noise plus focus * gain * one of `n_anchor` anchor keys of that head, so
    that the heads' attention rows range from diffuse to sharply peaked."""
    B, Hq, Hkv, d, G = L.batch, L.n_q_heads, L.n_kv_heads, L.head_dim, L.group
    counts = np.array([max(1, n_text - (3 * b if ragged else 0)) for b in range(B)], dtype=np.int32)
    q = np.zeros((B, n_text, Hq, d), dtype=np.float32)
    for b in range(B):
        C = int(L.seq_lens[b])
        for h in range(Hkv):
            rng = _rng(seed, L.layer, _T_QTEXT, b, h)
            focus = ((b * Hkv + h) % 4) / 3.0
            anchors = rng.choice(C, size=min(n_anchor, C), replace=False)
            x = rng.standard_normal((n_text, G, d), dtype=np.float32)
            pick = anchors[rng.integers(0, anchors.size, size=(n_text, G))]
            x += np.float32(focus * gain) * bf16_bits_to_f32(L.k[b, h][pick])
            q[b, :, h * G:(h + 1) * G] = x
    return f32_to_bf16_bits(q), counts
