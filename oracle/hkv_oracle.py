"""CPU oracle for HybridKV compression and decode attention.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the hot path computes, written from the paper
(Appendix A "Details of Hybrid KV Cache Compression", Section 3.3).  It is used by the tests, by
the smoke check and by the benchmark's CPU-baseline leg, and by nothing else: the product path
never imports it and shares no code with it.

Arithmetic: bf16 inputs are decoded exactly and everything is computed in float64 with numpy,
except where the method itself fixes a precision:

* chunk metadata (Appendix A, "average of its key vectors") is stored as bf16; it is formed as a
  float32 sum of the chunk's keys in ascending token order, an IEEE float32 division by the chunk
  length and a round-to-nearest-even conversion to bf16;
* a score that decides an index set (window scores for the Top-M visual tokens, chunk scores for
  the top-k chunks) is computed in float64 and rounded once to float32; the decision is taken on
  those float32 values, ties going to the lower index.

Pins (see tests/test_oracle_pins.py): full-budget runs equal textbook softmax attention written
independently; chunk selection equals brute force on tiny inputs; chunk size 1 equals exact top-k
tokens; closed-form chunk means; analytic keep-sets under score override; softmax rows sum to one;
static outputs are independent of dynamic budgets.  Agreement of end-to-end model accuracy with the
paper's tables is NOT pinned (it needs the paper's datasets and weights): parity unpinned for that.

Conventions ("head" always means KV head; G = query heads per KV head):
  k, v      uint16 [C, d]      bf16 bit patterns of one (sequence, kv head) plane
  q         uint16 [G, d]      the G query heads that share the kv head
  q_obs     uint16 [w, G, d]   queries of the last w prompt tokens (observation window)
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np


# ---------------------------------------------------------------------------------------------
# number formats
# ---------------------------------------------------------------------------------------------
def bf16_to_f64(u: np.ndarray) -> np.ndarray:
    """Exact decode of bf16 bit patterns."""
    f32 = (np.asarray(u, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)
    return f32.astype(np.float64)


def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns, round to nearest, ties to even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    return ((u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


def _softmax_rows(logits: np.ndarray) -> np.ndarray:
    m = logits.max(axis=-1, keepdims=True)
    e = np.exp(logits - m)
    return e / e.sum(axis=-1, keepdims=True)


# ---------------------------------------------------------------------------------------------
# static heads: observation-window scores and the keep-set  (Appendix A, first paragraph)
# ---------------------------------------------------------------------------------------------
def window_scores(q_obs: np.ndarray, k: np.ndarray, scale: float, causal: bool = False) -> np.ndarray:
    """s_w of Appendix A for one static kv head.

    S_w = softmax(Q[C-w:C] K^T / sqrt(d_k)) row by row over ALL C tokens of the prompt, and s_w is
    the mean of the rows.  Under grouped-query attention the rows are the w window positions of
    every one of the G query heads that share this kv head (mean over w*G rows).
    `causal=True` masks key j > position of the window row (variant; the paper's equation has no
    mask and says the window attends to the entire prompt).
    Returns float64 [C].
    """
    w, G, d = q_obs.shape
    C = k.shape[0]
    Q = bf16_to_f64(q_obs).reshape(w * G, d)
    K = bf16_to_f64(k)
    logits = (Q @ K.T) * scale                                   # [w*G, C]
    if causal:
        pos = np.repeat(np.arange(C - w, C), G)                  # window row i sits at position pos
        logits = np.where(np.arange(C)[None, :] > pos[:, None], -np.inf, logits)
    P = _softmax_rows(logits)
    return P.mean(axis=0)


def _top_by_score(cand: np.ndarray, scores_f32: np.ndarray, m: int) -> np.ndarray:
    """The m candidates with the largest float32 score; equal scores -> lower position first."""
    if m <= 0:
        return np.zeros(0, dtype=np.int64)
    if m >= cand.size:
        return cand.copy()
    s = scores_f32[cand]
    order = np.lexsort((cand, -s.astype(np.float64)))            # primary: score desc, then position asc
    return cand[order[:m]]


def static_keep_set(scores: np.ndarray, is_text: np.ndarray, C: int, w: int, budget: int) -> np.ndarray:
    """Positions kept for a static head, ascending (Appendix A: the three sets).

    (i) the observation window [C-w, C); (ii) every text token before the window; (iii) the Top-M
    visual tokens before the window by s_w, M = budget - w - |text before window|.
    When the budget cannot hold (i)+(ii) (the paper assumes it can): M = 0 and the text tokens are
    themselves ranked by s_w for the budget - w places left; when budget < w the last `budget`
    tokens are kept.  |keep| = min(budget, C) always.
    """
    budget = int(min(budget, C))
    if budget <= w:
        return np.arange(C - budget, C, dtype=np.int64)
    s32 = np.asarray(scores, dtype=np.float64).astype(np.float32)
    hist = np.arange(0, C - w, dtype=np.int64)
    txt = hist[is_text[:C - w] != 0]
    vis = hist[is_text[:C - w] == 0]
    window = np.arange(C - w, C, dtype=np.int64)
    room = budget - w
    if txt.size >= room:
        keep_hist = _top_by_score(txt, s32, room)
    else:
        keep_hist = np.concatenate([txt, _top_by_score(vis, s32, room - txt.size)])
    keep = np.sort(np.concatenate([keep_hist, window]))
    return keep


# ---------------------------------------------------------------------------------------------
# dynamic heads: chunk metadata, chunk scores, top-k chunks  (Appendix A, second paragraph)
# ---------------------------------------------------------------------------------------------
def n_chunks_of(C: int, cs: int) -> int:
    return (C + cs - 1) // cs


def chunk_summaries(k: np.ndarray, cs: int) -> np.ndarray:
    """Metadata of every chunk: the average of its key vectors, stored as bf16 bits [n_chunks, d].
    float32 running sum in ascending token order, float32 division by the chunk's own length (the
    last chunk may be shorter), round-to-nearest-even to bf16."""
    C, d = k.shape
    K32 = (np.asarray(k, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)
    n = n_chunks_of(C, cs)
    out = np.zeros((n, d), dtype=np.uint16)
    for c in range(n):
        s, e = c * cs, min((c + 1) * cs, C)
        acc = np.zeros(d, dtype=np.float32)
        for t in range(s, e):
            acc = acc + K32[t]                                    # float32 adds, one token at a time
        out[c] = f32_to_bf16(acc / np.float32(e - s))
    return out


def chunk_scores(q: np.ndarray, summaries: np.ndarray, group_max: bool = False) -> np.ndarray:
    """Inner product between the query and each chunk's metadata; for a group of G query heads that
    share the kv head the score is the sum over the group (variant `group_max`: the largest of the
    group's inner products, i.e. a chunk counts as much as its keenest query head wants it).
    No scale, no softmax: ranking only.  float64 -> one rounding to float32.  Returns float32 [n_chunks]."""
    Q = bf16_to_f64(q)                                            # [G, d]
    M = bf16_to_f64(summaries)                                    # [n, d]
    dots = M @ Q.T                                                # [n, G]
    return (dots.max(axis=1) if group_max else dots.sum(axis=1)).astype(np.float32)


def n_selected_chunks(budget: int, cs: int, n_chunks: int) -> int:
    """Number of chunks loaded: set by the per-head budget and the chunk size, rounded up."""
    return int(min(n_chunks, (int(budget) + cs - 1) // cs))


def select_chunks(scores_f32: np.ndarray, k: int) -> np.ndarray:
    """Ids of the k highest-scoring chunks, ascending; equal scores -> lower chunk id."""
    n = scores_f32.size
    ids = np.arange(n, dtype=np.int64)
    return np.sort(_top_by_score(ids, scores_f32, k))


def chunk_tokens(chunks: np.ndarray, cs: int, C: int) -> np.ndarray:
    """Token positions covered by the given chunks."""
    if len(chunks) == 0:
        return np.zeros(0, dtype=np.int64)
    return np.concatenate([np.arange(int(c) * cs, min((int(c) + 1) * cs, C), dtype=np.int64) for c in chunks])


# ---------------------------------------------------------------------------------------------
# attention over a retained token set
# ---------------------------------------------------------------------------------------------
def attend(q: np.ndarray, k: np.ndarray, v: np.ndarray, tokens: np.ndarray, scale: float,
           return_weights: bool = False):
    """o_g = sum_j softmax_j(<q_g, k_j> * scale) v_j over the retained tokens only. float64 [G, d]."""
    Q = bf16_to_f64(q)
    K = bf16_to_f64(k[tokens])
    V = bf16_to_f64(v[tokens])
    P = _softmax_rows((Q @ K.T) * scale)
    O = P @ V
    return (O, P) if return_weights else O


# ---------------------------------------------------------------------------------------------
# whole-layer drivers
# ---------------------------------------------------------------------------------------------
@dataclass
class OracleHead:
    kind: int                                   # 0 static, 1 dynamic
    C: int
    keep: Optional[np.ndarray] = None           # static: kept positions, ascending
    scores: Optional[np.ndarray] = None         # static: s_w rounded to float32 [C]
    summaries: Optional[np.ndarray] = None      # dynamic: bf16 bits [n_chunks, d]
    n_sel: int = 0                              # dynamic: chunks per step


@dataclass
class OracleCache:
    heads: Dict[Tuple[int, int], OracleHead] = field(default_factory=dict)


def _scale_of(L, scale: Optional[float]) -> float:
    return float(scale) if scale else 1.0 / math.sqrt(L.head_dim)


def compress_layer(L, token_scores: Optional[np.ndarray] = None, scale: Optional[float] = None,
                   causal_window: bool = False, only: Optional[List[Tuple[int, int]]] = None) -> OracleCache:
    """Compression of one layer: every static head gets its keep-set, every dynamic head its chunk
    metadata.  `token_scores` (float32 [B, Hkv, C_max]) replaces the observation-window scores.
    `only` restricts the work to the listed (b, h) pairs."""
    sc = _scale_of(L, scale)
    G = L.group
    cache = OracleCache()
    for b in range(L.batch):
        C = int(L.seq_lens[b])
        for h in range(L.n_kv_heads):
            if only is not None and (b, h) not in only:
                continue
            k = L.k[b, h, :C]
            if L.head_type[b, h] == 0:
                if token_scores is not None:
                    s = np.asarray(token_scores[b, h, :C], dtype=np.float64)
                else:
                    s = window_scores(L.q_obs[b, :, h * G:(h + 1) * G, :], k, sc, causal_window)
                keep = static_keep_set(s, L.is_text[b, :C], C, L.obs_window, int(L.budgets[b, h]))
                cache.heads[(b, h)] = OracleHead(0, C, keep=keep, scores=s.astype(np.float32))
            else:
                summ = chunk_summaries(k, L.chunk_size)
                cache.heads[(b, h)] = OracleHead(1, C, summaries=summ,
                                                 n_sel=n_selected_chunks(int(L.budgets[b, h]), L.chunk_size,
                                                                         summ.shape[0]))
    return cache


def append_token(L, cache: OracleCache, k_new: np.ndarray, v_new: np.ndarray) -> None:
    """Adds the token just generated (k_new, v_new: uint16 [B, Hkv, d]) to one layer's compressed cache
    (Appendix A / Section 3.3 only say the GPU buffer is "updated"; reading taken: a static head always
    retains the new token, a dynamic head's chunking simply covers the longer sequence, its metadata being
    what chunk_summaries gives for that longer sequence, and the number of chunks per step follows the
    unchanged budget).  L.k / L.v must have room (max_seq_len > seq_len); L and cache are updated in place."""
    for b in range(L.batch):
        C = int(L.seq_lens[b])
        assert C < L.k.shape[2], "no room for another token"
        L.k[b, :, C] = k_new[b]
        L.v[b, :, C] = v_new[b]
        L.seq_lens[b] = C + 1
        for h in range(L.n_kv_heads):
            hd = cache.heads.get((b, h))
            if hd is None:
                continue
            hd.C = C + 1
            if hd.kind == 0:
                hd.keep = np.concatenate([hd.keep, np.array([C], dtype=np.int64)])
            else:
                hd.summaries = chunk_summaries(L.k[b, h, :C + 1], L.chunk_size)
                hd.n_sel = n_selected_chunks(int(L.budgets[b, h]), L.chunk_size, hd.summaries.shape[0])


def decode_layer(L, cache: OracleCache, q: np.ndarray, scale: Optional[float] = None,
                 chunk_override: Optional[Dict[Tuple[int, int], np.ndarray]] = None,
                 keep_override: Optional[Dict[Tuple[int, int], np.ndarray]] = None, group_max: bool = False):
    """One decode step of one layer.  q: uint16 [B, Hq, d].
    Static head: attention over its keep-set.  Dynamic head: score the chunks with the query, take
    the top-k, attend over the tokens of those chunks only.  Heads are independent.
    Returns (out float64 [B, Hq, d], selected {(b,h): chunk ids}, scores {(b,h): float32 [n_chunks]})."""
    sc = _scale_of(L, scale)
    G = L.group
    out = np.zeros((L.batch, L.n_q_heads, L.head_dim), dtype=np.float64)
    selected, scores = {}, {}
    for (b, h), hd in cache.heads.items():
        C = hd.C
        qg = q[b, h * G:(h + 1) * G, :]
        k, v = L.k[b, h, :C], L.v[b, h, :C]
        if hd.kind == 0:
            toks = hd.keep if keep_override is None or (b, h) not in keep_override else np.asarray(keep_override[(b, h)])
        else:
            s = chunk_scores(qg, hd.summaries, group_max)
            scores[(b, h)] = s
            sel = select_chunks(s, hd.n_sel)
            if chunk_override is not None and (b, h) in chunk_override:
                sel = np.sort(np.asarray(chunk_override[(b, h)], dtype=np.int64))
            selected[(b, h)] = sel
            toks = chunk_tokens(sel, L.chunk_size, C)
        out[b, h * G:(h + 1) * G, :] = attend(qg, k, v, toks, sc)
    return out, selected, scores
