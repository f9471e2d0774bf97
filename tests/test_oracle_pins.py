"""Pins for the CPU oracle: every function is checked against something other than itself —
closed forms, brute force on tiny inputs, library routines reached by a different route,
invariants, and special cases that reduce to textbook attention.  CPU only."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import hkv_inputs as hi
from oracle import hkv_oracle as o

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits(x):
    """float -> bf16 bits through torch (an independent RNE implementation)."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.uint16).numpy().copy()


def vals(u):
    return torch.from_numpy(np.ascontiguousarray(u)).view(torch.bfloat16).to(torch.float64).numpy()


# ------------------------------------------------------------------ number formats
def test_bf16_decode_is_exact_and_rne_matches_torch():
    rng = np.random.default_rng(0)
    u = rng.integers(0, 0x7F80, size=5000).astype(np.uint16)          # positive finite
    u = np.concatenate([u, u | np.uint16(0x8000)])
    assert np.array_equal(o.bf16_to_f64(u), vals(u))
    x = rng.standard_normal(20000).astype(np.float32) * np.float32(37.0)
    assert np.array_equal(o.f32_to_bf16(x), bits(x))
    # exact ties: 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    t = np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, -(1 + 2.0 ** -8)], dtype=np.float32)
    assert o.f32_to_bf16(t).tolist() == [0x3F80, 0x3F82, 0xBF80]


# ------------------------------------------------------------------ window scores (Appendix A, s_w)
def test_window_scores_two_token_closed_form():
    # C = 2, w = 1, G = 1: s_w[0] = 1 / (1 + exp((l1 - l0))) with l_j = <q, k_j> * scale
    q = bits([[[1.0, 2.0, -1.0, 0.5]]])                               # [w=1, G=1, d=4]
    k = bits([[0.5, -1.0, 2.0, 1.0], [1.5, 0.25, -0.5, 2.0]])
    scale = 0.5
    l0 = (1 * 0.5 + 2 * -1.0 + -1 * 2.0 + 0.5 * 1.0) * scale
    l1 = (1 * 1.5 + 2 * 0.25 + -1 * -0.5 + 0.5 * 2.0) * scale
    s = o.window_scores(q, k, scale)
    assert s[0] == pytest.approx(1.0 / (1.0 + math.exp(l1 - l0)), rel=1e-14)
    assert s[1] == pytest.approx(1.0 / (1.0 + math.exp(l0 - l1)), rel=1e-14)


def test_window_scores_sum_to_one_uniform_keys_and_library_softmax():
    L = hi.tiny(C=80, w=5, Hq=6, Hkv=2, d=16)
    G, C, sc = L.group, int(L.seq_lens[0]), 1 / math.sqrt(16)
    s = o.window_scores(L.q_obs[0, :, 0:G], L.k[0, 0, :C], sc)
    assert s.shape == (C,) and abs(s.sum() - 1.0) < 1e-12 and (s > 0).all()
    # identical keys -> every row uniform -> s_w = 1/C
    ku = np.repeat(L.k[0, 0, :1], C, axis=0)
    assert np.allclose(o.window_scores(L.q_obs[0, :, 0:G], ku, sc), 1.0 / C, rtol=1e-13)
    # mean over the w*G rows of a library softmax (torch, float64), rows taken one at a time
    Q = torch.from_numpy(vals(L.q_obs[0, :, 0:G]))                    # [w, G, d]
    K = torch.from_numpy(vals(L.k[0, 0, :C]))
    acc = torch.zeros(C, dtype=torch.float64)
    for i in range(L.obs_window):
        for g in range(G):
            acc += torch.softmax((K @ Q[i, g]) * sc, dim=0)
    assert np.allclose(s, (acc / (L.obs_window * G)).numpy(), rtol=1e-12, atol=0)


def test_window_scores_use_the_last_w_queries_of_the_right_group():
    # rows come from q_obs as given: changing another group's queries must not matter,
    # changing one of ours must.
    L = hi.tiny(C=64, w=4, Hq=4, Hkv=2, d=16)
    G, C, sc = 2, int(L.seq_lens[0]), 0.25
    s = o.window_scores(L.q_obs[0, :, 0:G], L.k[0, 0, :C], sc)
    q2 = L.q_obs.copy()
    q2[0, :, G:] ^= np.uint16(0x8000)
    assert np.array_equal(s, o.window_scores(q2[0, :, 0:G], L.k[0, 0, :C], sc))
    q2[0, 1, 0] ^= np.uint16(0x8000)
    assert not np.allclose(s, o.window_scores(q2[0, :, 0:G], L.k[0, 0, :C], sc))


def test_window_scores_causal_variant_masks_later_keys():
    L = hi.tiny(C=40, w=4, Hq=2, Hkv=2, d=16, ragged=False)
    C, sc = 40, 0.25
    s = o.window_scores(L.q_obs[0, :, 0:1], L.k[0, 0, :C], sc, causal=True)
    assert abs(s.sum() - 1.0) < 1e-12
    # the last token is visible to the last window row only: s[C-1] = softmax row's own weight / w
    Q, K = vals(L.q_obs[0, :, 0:1]), vals(L.k[0, 0, :C])
    row = np.exp((K @ Q[-1, 0]) * sc)
    assert s[C - 1] == pytest.approx(row[C - 1] / row.sum() / 4, rel=1e-12)


# ------------------------------------------------------------------ static keep-set (Appendix A, three sets)
def test_keep_set_analytic_under_score_override():
    C, w, budget = 60, 6, 20
    is_text = np.zeros(C, dtype=np.uint8)
    is_text[[0, 1, 2, 30, 31, 50]] = 1                                  # 6 text tokens before the window
    is_text[C - w:] = 1
    scores = np.zeros(C)
    vis = [j for j in range(C - w) if not is_text[j]]
    rng = np.random.default_rng(5)
    perm = rng.permutation(len(vis))
    for rank, p in enumerate(perm):                                     # vis[p] has the rank-th largest score
        scores[vis[p]] = 1.0 - rank * 0.01
    scores[C - w:] = -5.0                                               # the window is kept whatever it scores
    scores[[0, 1, 2]] = -9.0                                            # so is text
    M = budget - w - 6
    expect = sorted([0, 1, 2, 30, 31, 50] + list(range(C - w, C)) + [vis[p] for p in perm[:M]])
    keep = o.static_keep_set(scores, is_text, C, w, budget)
    assert keep.tolist() == expect and keep.size == budget


def test_keep_set_properties_and_edge_cases():
    rng = np.random.default_rng(1)
    for C, w, nt in [(50, 4, 5), (33, 8, 0), (64, 1, 20), (20, 20, 0)]:
        is_text = np.zeros(C, dtype=np.uint8)
        if nt:
            is_text[rng.choice(max(C - w, 1), size=min(nt, max(C - w, 1)), replace=False)] = 1
        s = rng.random(C)
        T = np.nonzero(is_text[:C - w])[0]
        for budget in [1, w - 1, w, w + 1, w + len(T), w + len(T) + 3, C - 1, C, C + 7]:
            if budget < 1:
                continue
            keep = o.static_keep_set(s, is_text, C, w, budget)
            assert keep.size == min(budget, C)
            assert np.all(np.diff(keep) > 0) and keep.min() >= 0 and keep.max() < C
            if budget >= w:
                assert set(range(C - w, C)) <= set(keep.tolist())
            else:
                assert keep.tolist() == list(range(C - budget, C))
            if budget >= w + len(T):
                assert set(T.tolist()) <= set(keep.tolist())
                extra = [j for j in keep if j < C - w and not is_text[j]]
                rest = [j for j in range(C - w) if not is_text[j] and j not in extra]
                if extra and rest:                                       # kept visual tokens outrank the dropped ones
                    assert min(s[extra].astype(np.float32)) >= max(s[rest].astype(np.float32))
            else:                                                        # text itself is ranked, no visual token kept
                hist = [j for j in keep if j < C - w]
                assert all(is_text[j] for j in hist)


def test_keep_set_all_text_prompt_and_ties():
    C, w = 30, 5
    is_text = np.ones(C, dtype=np.uint8)
    keep = o.static_keep_set(np.zeros(C), is_text, C, w, 30)
    assert keep.tolist() == list(range(C))
    # equal scores -> the lower positions win
    is_text[:] = 0
    keep = o.static_keep_set(np.full(C, 0.5), is_text, C, w, 9)
    assert keep.tolist() == [0, 1, 2, 3] + list(range(C - w, C))
    # decision is taken on float32 values: a 1e-12 difference is a tie and position decides
    s = np.full(C, 0.5)
    s[10] += 1e-12
    keep = o.static_keep_set(s, is_text, C, w, 6)
    assert keep.tolist() == [0] + list(range(C - w, C))


# ------------------------------------------------------------------ chunk metadata
def test_chunk_summaries_closed_forms_and_tail():
    d = 8
    # constant chunks -> the constant; keys = token index -> midpoint; tail chunk has its own length
    C, cs = 22, 4
    k = bits(np.repeat(np.arange(C, dtype=np.float32)[:, None], d, axis=1))
    m = vals(o.chunk_summaries(k, cs))
    assert m.shape == (6, d)
    assert np.array_equal(m[:5, 0], [1.5, 5.5, 9.5, 13.5, 17.5])
    assert m[5, 0] == 20.5                                               # tokens 20, 21 only
    kc = bits(np.full((C, d), -3.25, dtype=np.float32))
    assert np.all(vals(o.chunk_summaries(kc, cs)) == -3.25)
    assert o.chunk_summaries(k, 64).shape == (1, d)                      # cs >= C: one chunk
    assert np.array_equal(o.chunk_summaries(k, 1), k)                    # cs = 1: metadata = keys


def test_chunk_summaries_rounding_order_fixture():
    """float32 sum in ascending token order, float32 divide, RNE to bf16 — cases worked by hand in
    tests/golden/chunk_mean_rounding.txt (a float64 sum or a tree-shaped sum gives other bits)."""
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "chunk_mean_rounding.txt")) if ln.strip() and ln[0] != "#"]
    assert len(rows) >= 3
    for r in rows:
        expect = int(r[0], 16)
        keys = np.array([float.fromhex(x) for x in r[1:]], dtype=np.float32)
        kb = bits(keys[:, None])
        assert np.array_equal(vals(kb)[:, 0], keys.astype(np.float64))   # fixture values are bf16 numbers
        got = o.chunk_summaries(kb, len(keys))
        assert int(got[0, 0]) == expect, (r, hex(int(got[0, 0])))


# ------------------------------------------------------------------ chunk scores and selection
def test_chunk_scores_brute_force_and_group_sum():
    L = hi.tiny(C=48, chunk_size=4, Hq=6, Hkv=2, d=8)
    G, C = 3, int(L.seq_lens[1])
    summ = o.chunk_summaries(L.k[1, 1, :C], 4)
    q = L.q[0][1, G:2 * G]
    s = o.chunk_scores(q, summ)
    M, Q = vals(summ), vals(q)
    for c in range(summ.shape[0]):
        tot = 0.0
        for g in range(G):
            for i in range(8):
                tot += Q[g, i] * M[c, i]
        assert s[c] == np.float32(tot) or abs(float(s[c]) - tot) <= 1e-6 * abs(tot)
    # the group score is the SUM over the group's query heads (not max, not the first head)
    q1 = bits([[1.0, 0.0], [1.0, 0.0]])
    m1 = bits([[1.0, 0.0], [0.75, 5.0], [-2.0, 1.0]])
    assert o.chunk_scores(q1, m1).tolist() == [2.0, 1.5, -4.0]
    q2 = bits([[1.0, 0.0], [-1.0, 1.0]])
    assert o.chunk_scores(q2, m1).tolist() == [0.0, 5.0, 1.0]


def test_select_chunks_brute_force_and_ties():
    rng = np.random.default_rng(3)
    for n in [1, 2, 7, 16]:
        s = rng.standard_normal(n).astype(np.float32)
        for k in range(1, n + 1):
            ranked = sorted(range(n), key=lambda c: (-float(s[c]), c))
            assert o.select_chunks(s, k).tolist() == sorted(ranked[:k])
    s = np.array([1.0, 3.0, 3.0, 0.5, 3.0, 1.0], dtype=np.float32)
    assert o.select_chunks(s, 2).tolist() == [1, 2]
    assert o.select_chunks(s, 4).tolist() == [0, 1, 2, 4]
    assert o.select_chunks(s, 6).tolist() == [0, 1, 2, 3, 4, 5]
    assert o.n_selected_chunks(205, 32, 64) == 7 and o.n_selected_chunks(1, 32, 64) == 1
    assert o.n_selected_chunks(4096, 32, 64) == 64 and o.n_selected_chunks(64, 32, 64) == 2


def test_chunk_size_one_selects_exact_top_tokens():
    L = hi.tiny(C=40, chunk_size=1, Hq=4, Hkv=2, d=16, ragged=False, head_type=[[1, 1], [1, 1]])
    L.budgets[:] = 9
    cache = o.compress_layer(L)
    _, sel, _ = o.decode_layer(L, cache, L.q[0])
    for (b, h), chunks in sel.items():
        K, Q = vals(L.k[b, h, :40]), vals(L.q[0][b, 2 * h:2 * h + 2])
        tok = (K @ Q.sum(axis=0))
        assert sorted(np.argsort(-tok, kind="stable")[:9].tolist()) == chunks.tolist()


# ------------------------------------------------------------------ decode attention
def _sdpa_full(L, q, b):
    """Textbook full-cache GQA attention through torch's library routine (float64)."""
    C = int(L.seq_lens[b])
    Q = torch.from_numpy(vals(q[b]))[None, :, None, :]                      # [1, Hq, 1, d]
    K = torch.from_numpy(vals(L.k[b, :, :C])).repeat_interleave(L.group, dim=0)[None]
    V = torch.from_numpy(vals(L.v[b, :, :C])).repeat_interleave(L.group, dim=0)[None]
    return torch.nn.functional.scaled_dot_product_attention(Q, K, V)[0, :, 0].numpy()


@pytest.mark.parametrize("cs", [1, 8, 7, 200])
def test_full_budget_equals_textbook_attention(cs):
    L = hi.tiny(C=96, chunk_size=cs, Hq=6, Hkv=2, d=16, w=4, head_type=[[0, 1], [1, 0]])
    L.budgets[:] = L.seq_lens[:, None]                                      # 100 %
    out, sel, _ = o.decode_layer(L, o.compress_layer(L), L.q[0])
    for b in range(L.batch):
        assert np.allclose(out[b], _sdpa_full(L, L.q[0], b), rtol=1e-11, atol=1e-12)
    for (b, h), c in sel.items():
        assert c.tolist() == list(range(o.n_chunks_of(int(L.seq_lens[b]), cs)))


def test_attend_weights_and_convexity():
    L = hi.tiny(C=64, Hq=4, Hkv=2, d=16)
    toks = np.array([3, 4, 9, 20, 21, 40])
    O, P = o.attend(L.q[0][0, 0:2], L.k[0, 0], L.v[0, 0], toks, 0.25, return_weights=True)
    assert np.allclose(P.sum(axis=1), 1.0, rtol=1e-14) and (P > 0).all()
    V = vals(L.v[0, 0][toks])
    assert (O <= V.max(axis=0) + 1e-12).all() and (O >= V.min(axis=0) - 1e-12).all()
    # a single retained token returns its value row; scale matters; order of tokens does not
    O1 = o.attend(L.q[0][0, 0:2], L.k[0, 0], L.v[0, 0], np.array([7]), 0.25)
    assert np.array_equal(O1[0], vals(L.v[0, 0][7])) and np.array_equal(O1[1], O1[0])
    assert not np.allclose(O, o.attend(L.q[0][0, 0:2], L.k[0, 0], L.v[0, 0], toks, 0.5))
    assert np.allclose(O, o.attend(L.q[0][0, 0:2], L.k[0, 0], L.v[0, 0], toks[::-1], 0.25), rtol=1e-12)
    # two tokens, one head, closed form
    q, k, v = bits([[2.0, 0.0]]), bits([[1.0, 0.0], [0.0, 1.0]]), bits([[1.0, 0.0], [0.0, 1.0]])
    O2 = o.attend(q, k, v, np.array([0, 1]), 0.5)
    p0 = math.e / (math.e + 1.0)
    assert np.allclose(O2[0], [p0, 1 - p0], rtol=1e-14)


def test_partial_budget_equals_attention_over_retained_tokens_only():
    L = hi.tiny(C=96, chunk_size=8, Hq=4, Hkv=2, d=16, head_type=[[0, 1], [1, 0]])
    cache = o.compress_layer(L)
    out, sel, _ = o.decode_layer(L, cache, L.q[0])
    for (b, h), hd in cache.heads.items():
        C = hd.C
        toks = hd.keep if hd.kind == 0 else o.chunk_tokens(sel[(b, h)], 8, C)
        n_expected = min(int(L.budgets[b, h]), C) if hd.kind == 0 else None
        if hd.kind == 0:
            assert toks.size == n_expected
        else:
            k = math.ceil(int(L.budgets[b, h]) / 8)
            assert sel[(b, h)].size == k
            assert toks.size == k * 8 - (8 * o.n_chunks_of(C, 8) - C if (o.n_chunks_of(C, 8) - 1) in sel[(b, h)] else 0)
        Kf = torch.from_numpy(vals(L.k[b, h][toks]))
        Vf = torch.from_numpy(vals(L.v[b, h][toks]))
        for g in range(2):
            qv = torch.from_numpy(vals(L.q[0][b, 2 * h + g]))
            ref = torch.softmax((Kf @ qv) / 4.0, dim=0) @ Vf
            assert np.allclose(out[b, 2 * h + g], ref.numpy(), rtol=1e-11, atol=1e-13)


def test_static_output_unchanged_by_dynamic_budget_and_heads_independent():
    L = hi.tiny(C=96, chunk_size=8, Hq=4, Hkv=2, d=16, head_type=[[0, 1], [1, 0]])
    out1, _, _ = o.decode_layer(L, o.compress_layer(L), L.q[0])
    for b in range(2):
        for h in range(2):
            if L.head_type[b, h] == 1:
                L.budgets[b, h] = 57
    out2, _, _ = o.decode_layer(L, o.compress_layer(L), L.q[0])
    for b in range(2):
        for h in range(2):
            same = np.array_equal(out1[b, 2 * h:2 * h + 2], out2[b, 2 * h:2 * h + 2])
            assert same == (L.head_type[b, h] == 0)


def test_planted_chunks_are_recovered():
    L = hi.cfg3(layer=0, B=2, C=2000, block=256, chunk_size=32, budget_fraction=0.05)
    cache = o.compress_layer(L, only=[(b, h) for b in range(2) for h in range(4) if L.head_type[b, h] == 1])
    _, sel, _ = o.decode_layer(L, cache, L.q[0])
    assert len(sel) > 0
    for (b, h), c in sel.items():
        assert set(L.planted[b, h].tolist()) <= set(c.tolist())


def test_selection_exhaustive_subsets_tiny():
    """Brute force over all k-subsets: the selected set maximises the total score."""
    L = hi.tiny(C=24, chunk_size=4, Hq=2, Hkv=1, d=8, B=1, head_type=[[1]])
    L.budgets[:] = 9                                                      # ceil(9/4) = 3 chunks of 6
    cache = o.compress_layer(L)
    _, sel, sc = o.decode_layer(L, cache, L.q[0])
    s = sc[(0, 0)].astype(np.float64)
    best = max(itertools.combinations(range(6), 3), key=lambda S: sum(s[list(S)]))
    assert sorted(best) == sel[(0, 0)].tolist()


def test_chunk_score_group_max_variant():
    """The max-over-group variant: hand values, equality with the sum for a group of one, and a case where the two
    rankings differ (one keen head against many lukewarm ones)."""
    f = lambda a: hi.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))
    m = f([[1, 0], [0, 1], [1, 1]])
    q = f([[3, 0], [0, 2], [-1, -1]])           # dots: chunk0 (3, 0, -1), chunk1 (0, 2, -1), chunk2 (3, 2, -2)
    assert o.chunk_scores(q, m, group_max=True).tolist() == [3.0, 2.0, 3.0]
    assert o.chunk_scores(q, m).tolist() == [2.0, 1.0, 3.0]
    assert o.chunk_scores(q[:1], m, group_max=True).tolist() == o.chunk_scores(q[:1], m).tolist()
    q2 = f([[4, 0], [0, 1], [0, 1], [0, 1], [0, 1], [0, 1]])      # chunk0: max 4 / sum 4; chunk1: max 1 / sum 5
    assert np.argmax(o.chunk_scores(q2, m[:2], group_max=True)) == 0 and np.argmax(o.chunk_scores(q2, m[:2])) == 1
    rng = np.random.default_rng(3)
    qq, mm = f(rng.standard_normal((7, 16))), f(rng.standard_normal((9, 16)))
    ref = [max(float(np.dot(hi.bf16_bits_to_f32(mm[c]).astype(np.float64), hi.bf16_bits_to_f32(qq[g]).astype(np.float64)))
               for g in range(7)) for c in range(9)]
    assert np.allclose(o.chunk_scores(qq, mm, group_max=True), np.float32(ref), rtol=0, atol=0)
