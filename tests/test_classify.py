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


# ---------------------------------------------------------------------------------------------
# CUDA path against the oracle
# ---------------------------------------------------------------------------------------------
SCORE_TOL = 1e-4     # float32 softmax arithmetic against float64


def _oracle_scores(L, q_text, counts, fraction):
    G = L.group
    scale = 1.0 / math.sqrt(L.head_dim)
    out = np.zeros((L.batch, L.n_kv_heads))
    for b in range(L.batch):
        C, T = int(L.seq_lens[b]), int(counts[b])
        for h in range(L.n_kv_heads):
            out[b, h] = co.sparsity_score(q_text[b, :T, h * G:(h + 1) * G], L.k[b, h, :C], scale, fraction)
    return out


def _gpu_scores(L, q_text, counts, fraction, theta, workspace="preferred"):
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import to_device_bf16
    cfg = hkv.hkv_config(batch=L.batch, n_q_heads=L.n_q_heads, n_kv_heads=L.n_kv_heads, head_dim=L.head_dim,
                         max_seq_len=L.max_seq_len, chunk_size=L.chunk_size, obs_window=L.obs_window,
                         softmax_scale=0.0, flags=0, append_capacity=0)
    lo, hi = hkv.hkv_classify_workspace(cfg, q_text.shape[1])
    assert 0 < lo <= hi
    ws = torch.empty(lo if workspace == "min" else hi, dtype=torch.uint8, device="cuda")
    scores = torch.full((L.batch, L.n_kv_heads), -1.0, dtype=torch.float64, device="cuda")
    types = torch.full((L.batch, L.n_kv_heads), 9, dtype=torch.uint8, device="cuda")
    hkv.hkv_classify_heads(cfg, to_device_bf16(L.k), to_device_bf16(q_text), L.seq_lens, counts, fraction, theta,
                           ws, scores, types)
    torch.cuda.synchronize()
    return scores.cpu().numpy(), types.cpu().numpy()


def _check_case(L, n_text, fraction, theta=None, workspace="preferred", seed=5):
    q_text, counts = hi.text_queries(L, n_text, seed=seed)
    ref = _oracle_scores(L, q_text, counts, fraction)
    if theta is None:
        srt = np.sort(ref.ravel())
        theta = float(0.5 * (srt[srt.size // 2 - 1] + srt[srt.size // 2])) if srt.size > 1 else 0.9
    got, types = _gpu_scores(L, q_text, counts, fraction, theta, workspace)
    err = np.abs(got - ref).max()
    assert err <= SCORE_TOL, (err, got, ref)
    for b in range(L.batch):
        for h in range(L.n_kv_heads):
            if abs(ref[b, h] - theta) > SCORE_TOL:
                assert types[b, h] == co.classify(ref[b, h], theta), (b, h, ref[b, h], theta)
            assert types[b, h] == (0 if got[b, h] >= theta else 1)
    return ref, got


@pytest.mark.gpu
@pytest.mark.parametrize("workspace", ["preferred", "min"])
def test_gpu_classify_ragged_batch(workspace):
    L = hi.tiny(seed=31, B=3, C=3000, chunk_size=32, w=8, Hq=28, Hkv=4, d=128)
    ref, _ = _check_case(L, 20, 0.05, workspace=workspace)
    assert ref.max() - ref.min() > 0.3            # the heads really span diffuse to peaked
    _check_case(L, 20, 0.05, theta=0.9, workspace=workspace)


@pytest.mark.gpu
@pytest.mark.parametrize("fraction", [1e-6, 0.01, 0.5, 1.0])
def test_gpu_classify_topk_counts(fraction):
    L = hi.tiny(seed=32, B=2, C=1500, chunk_size=32, w=8, Hq=8, Hkv=2, d=128)
    ref, got = _check_case(L, 9, fraction)
    if fraction == 1.0:
        assert np.abs(got - 1.0).max() < 1e-5


@pytest.mark.gpu
def test_gpu_classify_several_row_blocks_in_one_pass():
    """420 rows per unit in one pass: two resident 256-row blocks per key range (the second partly padding)."""
    L = hi.tiny(seed=36, B=2, C=1400, chunk_size=32, w=8, Hq=28, Hkv=4, d=128)
    _check_case(L, 60, 0.05)
    _check_case(L, 60, 0.05, workspace="min")


@pytest.mark.gpu
@pytest.mark.parametrize("C", [32768, 32765, 31745, 1023, 5])
def test_gpu_classify_rows_kept_in_registers(C):
    """Rows of up to 32768 entries take the pipelined kernel (the row in registers, the next row's copy in flight):
    the longest such row, lengths that are no multiple of four, a last piece of one vector, rows shorter than one
    piece, and rows of a handful of entries."""
    L = hi.tiny(seed=41, B=2 if C < 2000 else 1, C=C, chunk_size=32 if C >= 64 else 1, w=8 if C >= 64 else 2, Hq=8, Hkv=2,
                d=128, ragged=False)
    _check_case(L, 5, 0.05)


@pytest.mark.gpu
@pytest.mark.parametrize("C", [32769, 49152])
def test_gpu_classify_rows_kept_in_shared_memory(C):
    """Between 32769 and 49152 entries a row stays in shared memory (the general kernel), beyond that in the workspace."""
    L = hi.tiny(seed=42, B=1, C=C, chunk_size=32, w=8, Hq=4, Hkv=2, d=128, ragged=False)
    _check_case(L, 3, 0.05)


@pytest.mark.gpu
def test_gpu_classify_rows_longer_than_shared_memory():
    L = hi.tiny(seed=33, B=1, C=50021, chunk_size=32, w=8, Hq=8, Hkv=2, d=128)
    _check_case(L, 3, 0.05)


@pytest.mark.gpu
def test_gpu_classify_more_sequences_than_one_launch_group():
    L = hi.tiny(seed=34, B=70, C=400, chunk_size=32, w=8, Hq=4, Hkv=2, d=128, ragged=False)
    _check_case(L, 4, 0.05)


@pytest.mark.gpu
def test_gpu_classify_uniform_rows_and_errors():
    from paper_2604_05887_b200 import binding as hkv
    L = hi.tiny(seed=35, B=1, C=640, chunk_size=32, w=8, Hq=4, Hkv=2, d=128, ragged=False)
    L.k[:] = L.k[:, :, :1]                         # identical keys: every row is uniform, score = k / C
    q_text, counts = hi.text_queries(L, 5)
    got, types = _gpu_scores(L, q_text, counts, 0.05, 0.9)
    assert np.abs(got - 32 / 640).max() < 1e-6 and np.all(types == 1)
    cfg = hkv.hkv_config(batch=1, n_q_heads=4, n_kv_heads=2, head_dim=128, max_seq_len=640, chunk_size=32,
                         obs_window=8, softmax_scale=0.0, flags=0, append_capacity=0)
    lo, _ = hkv.hkv_classify_workspace(cfg, 5)
    ws = torch.empty(lo, dtype=torch.uint8, device="cuda")
    sc = torch.zeros((1, 2), dtype=torch.float64, device="cuda")
    ty = torch.zeros((1, 2), dtype=torch.uint8, device="cuda")
    k = torch.zeros((1, 2, 640, 128), dtype=torch.bfloat16, device="cuda")
    q = torch.zeros((1, 5, 4, 128), dtype=torch.bfloat16, device="cuda")
    for kwargs, status in ((dict(seq_lens=[641]), 2), (dict(n_text=[6]), 2), (dict(n_text=[0]), 2),
                           (dict(fraction=0.0), 1), (dict(fraction=1.5), 1), (dict(ws=ws[:lo - 256]), 4)):
        a = dict(seq_lens=[640], n_text=[5], fraction=0.05, ws=ws)
        a.update(kwargs)
        with pytest.raises(hkv.HkvError) as e:
            hkv.hkv_classify_heads(cfg, k, q, a["seq_lens"], a["n_text"], a["fraction"], 0.9, a["ws"], sc, ty)
        assert e.value.status == status


@pytest.mark.gpu
@pytest.mark.parametrize("case", range(10))
def test_gpu_classify_random_shapes(case):
    """Seeded random geometry: batch, lengths, group size, text-token counts, top-k fraction, workspace size."""
    rng = np.random.default_rng(7000 + case)
    Hkv = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([1, 2, 4, 7, 8, 16]))
    B = int(rng.integers(1, 5))
    C = int(rng.integers(40, 6000))
    T = int(rng.integers(1, 80))
    fraction = float(rng.choice([0.01, 0.05, 0.05, 0.2, 0.5]))
    L = hi.tiny(seed=7100 + case, B=B, C=C, chunk_size=32, w=8, Hq=G * Hkv, Hkv=Hkv, d=128,
                ragged=bool(rng.integers(0, 2)) and C > 5 * B + 16)
    _check_case(L, T, fraction, workspace=str(rng.choice(["preferred", "min"])), seed=case)
