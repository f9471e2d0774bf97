"""CPU oracle for the text-centric head classification of HybridKV (paper Section 3.1).  TEST INFRASTRUCTURE ONLY.

For one KV head: S_text = softmax(Q_text K_context^T / sqrt(d_k)) row by row over ALL C context tokens (the
text-centric attention of Section 2.1, no mask printed); the text-centric sparsity score is the mean over the
text rows of the sum of each row's k largest entries; a head whose score reaches the threshold theta is
static, otherwise dynamic.  Float64 throughout.

Readings (the paper's equation has a stray inner index and gives no k): the inner sum is the sum of the k
largest entries of the row; k = ceil(fraction * C) with the 5 % the paper uses for its focus count; under
grouped-query attention the rows are the text positions of every query head of the group (mean over T * G
rows), as for the observation-window scores.

Pins (tests/test_classify.py): one-hot rows give 1, uniform rows give k / C, k = C gives 1, the score is
monotone in k and lies in [k / C, 1], brute force by full sort on small inputs, library softmax + topk.
"""
from __future__ import annotations

import math

import numpy as np


def _bf16_to_f64(u: np.ndarray) -> np.ndarray:
    return (np.asarray(u, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def topk_count(C: int, fraction: float) -> int:
    return max(1, min(int(C), int(math.ceil(fraction * C - 1e-9))))


def sparsity_score(q_text: np.ndarray, k: np.ndarray, scale: float, fraction: float = 0.05) -> float:
    """q_text: uint16 [T, G, d] queries of the T text tokens for the G query heads of the group;
    k: uint16 [C, d] keys of the whole context.  Returns S_{l,h} in (0, 1]."""
    T, G, d = q_text.shape
    C = k.shape[0]
    kk = topk_count(C, fraction)
    Q = _bf16_to_f64(q_text).reshape(T * G, d)
    K = _bf16_to_f64(k)
    total = 0.0
    for r0 in range(0, T * G, 256):                      # row blocks only bound the memory in use
        logits = (Q[r0:r0 + 256] @ K.T) * scale
        logits -= logits.max(axis=1, keepdims=True)
        P = np.exp(logits)
        P /= P.sum(axis=1, keepdims=True)
        top = np.partition(P, C - kk, axis=1)[:, C - kk:]
        total += float(top.sum())
    return total / float(T * G)


def classify(score: float, theta: float) -> int:
    """0 = static (score >= theta), 1 = dynamic."""
    return 0 if score >= theta else 1
