"""Text-centric head classification (Section 3.1): oracle pins (CPU) and GPU parity."""
import math

import numpy as np
import pytest
import torch

import hkv_inputs as hi
from oracle import hkv_classify_oracle as co


def bits(x):
    return hi.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_oracle_closed_forms():
    d, C = 16, 200
    rng = np.random.default_rng(0)
    # identical keys -> every row uniform -> score = k / C
    k = np.repeat(bits(rng.standard_normal((1, d))), C, axis=0)
    q = bits(rng.standard_normal((5, 2, d)))
    assert co.sparsity_score(q, k, 0.25, 0.05) == pytest.approx(co.topk_count(C, 0.05) / C, rel=1e-12)
    # one key that every query matches overwhelmingly -> rows are one-hot -> score = 1
    k2 = bits(rng.standard_normal((C, d)) * 0.01)
    k2[17] = bits(np.full(d, 8.0))
    q2 = bits(np.full((4, 2, d), 8.0))
    assert co.sparsity_score(q2, k2, 1.0, 0.05) == pytest.approx(1.0, abs=1e-12)
    # k = C keeps the whole row
    assert co.sparsity_score(q, bits(rng.standard_normal((C, d))), 0.25, 1.0) == pytest.approx(1.0, rel=1e-12)
    assert co.topk_count(32768, 0.05) == 1639 and co.topk_count(10, 0.05) == 1 and co.topk_count(100, 0.05) == 5


def test_oracle_equals_full_sort_and_library_routines():
    rng = np.random.default_rng(1)
    d, C, T, G = 32, 333, 7, 3
    q, k = bits(rng.standard_normal((T, G, d))), bits(rng.standard_normal((C, d)) * 2)
    s = co.sparsity_score(q, k, 1 / math.sqrt(d), 0.05)
    kk = co.topk_count(C, 0.05)
    Q = torch.from_numpy(q.reshape(T * G, d).copy()).view(torch.bfloat16).double()
    K = torch.from_numpy(k.copy()).view(torch.bfloat16).double()
    P = torch.softmax(Q @ K.T / math.sqrt(d), dim=1)
    ref = P.topk(kk, dim=1).values.sum(dim=1).mean().item()
    assert s == pytest.approx(ref, rel=1e-12)
    # brute force, row by row, by a full sort
    acc = 0.0
    for r in range(T * G):
        row = sorted(P[r].tolist(), reverse=True)
        acc += sum(row[:kk])
    assert s == pytest.approx(acc / (T * G), rel=1e-12)


def test_oracle_monotone_and_bounded():
    rng = np.random.default_rng(2)
    d, C = 16, 500
    q, k = bits(rng.standard_normal((6, 2, d))), bits(rng.standard_normal((C, d)))
    prev = 0.0
    for f in (0.01, 0.05, 0.2, 0.5, 1.0):
        s = co.sparsity_score(q, k, 0.25, f)
        assert prev < s <= 1.0 + 1e-12 and s >= co.topk_count(C, f) / C - 1e-12
        prev = s
    assert co.classify(0.95, 0.9) == 0 and co.classify(0.9, 0.9) == 0 and co.classify(0.85, 0.9) == 1
