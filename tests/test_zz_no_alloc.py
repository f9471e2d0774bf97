"""hkv_topk_chunks_noalloc — the selection step for callers that cannot allocate device memory.

Some users call this library from places where no allocator may be touched: inside another
runtime's callback, or in a loop whose latency budget rules out cudaMalloc and anything that
may call it.  For them the entry point keeps its per-chunk score scratch in a fixed array inside
the library; they hand over inputs and the output buffer only.

The first test drives the entry point through the C ABI several times in a row (every call reuses the
scratch the one before left behind, with a different query and a different chunk count) and checks
each result against what the regular path (hkv_decode_attn -> hkv_get_selected_chunks) selects for
the same head AND against the CPU oracle's selection from its own scores, under the rule the other
parity tests use: equal sets, except for swaps between chunks whose oracle scores are tied to 1e-5.
The second covers the ends of the size range against the oracle: as many chunk means as the built-in
scratch holds, and k at or beyond the number of chunks.  The file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import hkv_inputs as hi
from oracle import hkv_oracle as o

pytestmark = pytest.mark.gpu


def _regular_path(L, step):
    """Selected chunk ids, scores and plain row-major means of every dynamic head, from the regular entry points."""
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    lc = LayerCache(L)
    lc.decode(to_device_bf16(L.q[step]))
    torch.cuda.synchronize()
    out = {}
    for b in range(L.batch):
        n_chunks = (int(L.seq_lens[b]) + L.chunk_size - 1) // L.chunk_size
        for h in range(L.n_kv_heads):
            if L.head_type[b, h] == 1:
                out[(b, h)] = (hkv.hkv_get_selected_chunks(lc.handle, b, h),
                               hkv.hkv_get_chunk_scores(lc.handle, b, h, n_chunks),
                               hkv.hkv_get_summaries(lc.handle, b, h, n_chunks))
    lc.close()
    return out


def test_no_alloc_selection_matches_regular_path_twice_in_a_row():
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import to_device_bf16
    import parity_util as P

    G = hi.N_Q_HEADS // hi.N_KV_HEADS
    cases = [hi.cfg1(layer=3, C=8192, block=512, n_steps=1),              # 256 chunks of 32, k = 26
             hi.tiny(seed=21, B=2, C=3000, chunk_size=8, w=8, Hq=28, Hkv=4, d=128, budget_fraction=0.2)]
    n_calls = 0
    for L in cases:
        ref = _regular_path(L, 0)
        assert ref, "the case has no dynamic head"
        q_dev = to_device_bf16(L.q[0])
        for (b, h), (sel, scores, means) in ref.items():
            means_dev = to_device_bf16(means)
            out_ids = torch.full((sel.size,), -1, dtype=torch.int32, device="cuda")
            hkv.hkv_topk_chunks_noalloc(q_dev[b, h * G:(h + 1) * G].contiguous(), means_dev, sel.size, out_ids)
            torch.cuda.synchronize()
            got = out_ids.cpu().numpy()
            assert np.all(np.diff(got) > 0), "ids must come out ascending"
            P.sets_match_up_to_ties(got, sel, scores, f"no-alloc vs regular path ({b},{h})")
            ref_scores = o.chunk_scores(L.q[0][b, h * G:(h + 1) * G], means)
            _, wide = P.sets_match_up_to_ties(got, o.select_chunks(ref_scores, sel.size), ref_scores,
                                              f"no-alloc vs oracle ({b},{h})")
            assert wide == 0
            n_calls += 1
    assert n_calls >= 2


def test_no_alloc_at_the_ends_of_its_size_range():
    """HKV_NOALLOC_MAX_CHUNKS chunk means (16 MB; the radix selection then makes several passes over the whole
    scratch), twice in a row with different k, and k >= n_chunks (every id, in order)."""
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import to_device_bf16
    import parity_util as P
    rng = np.random.default_rng(77)
    G, n = 7, hkv.HKV_NOALLOC_MAX_CHUNKS
    q = hi.f32_to_bf16_bits(rng.standard_normal((G, 128)).astype(np.float32))
    means = hi.f32_to_bf16_bits(rng.standard_normal((n, 128)).astype(np.float32))
    means[1000:1040] = means[1000]                      # a run of exactly equal scores: the lower ids must win
    q_dev, means_dev = to_device_bf16(q), to_device_bf16(means)
    ref_scores = o.chunk_scores(q, means)
    for k in (6554, 100):
        out_ids = torch.full((k,), -1, dtype=torch.int32, device="cuda")
        hkv.hkv_topk_chunks_noalloc(q_dev, means_dev, k, out_ids)
        torch.cuda.synchronize()
        got = out_ids.cpu().numpy()
        assert np.all(np.diff(got) > 0)
        _, wide = P.sets_match_up_to_ties(got, o.select_chunks(ref_scores, k), ref_scores, f"no-alloc n={n} k={k}")
        assert wide == 0
    for n_small, k in ((37, 37), (37, 1000)):
        out_ids = torch.full((n_small,), -1, dtype=torch.int32, device="cuda")
        hkv.hkv_topk_chunks_noalloc(q_dev, means_dev[:n_small].contiguous(), k, out_ids)
        torch.cuda.synchronize()
        assert np.array_equal(out_ids.cpu().numpy(), np.arange(n_small))


def test_no_alloc_rejects_sizes_beyond_its_scratch():
    from paper_2604_05887_b200 import binding as hkv
    q = torch.zeros((7, 128), dtype=torch.bfloat16, device="cuda")
    means = torch.zeros((8, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(4, dtype=torch.int32, device="cuda")
    st = hkv.lib.hkv_topk_chunks_noalloc(q.data_ptr(), means.data_ptr(), 7, hkv.HKV_NOALLOC_MAX_CHUNKS + 1, 4,
                                         out.data_ptr(), None)
    assert st == 4                      # HKV_ERR_WORKSPACE: more chunks than the built-in scratch holds
    assert hkv.lib.hkv_topk_chunks_noalloc(q.data_ptr(), means.data_ptr(), 17, 8, 4, out.data_ptr(), None) == 5
