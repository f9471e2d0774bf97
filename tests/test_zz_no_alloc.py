"""hkv_topk_chunks_noalloc — the selection step for callers that cannot allocate device memory.

Some users call this library from places where no allocator may be touched: inside another
runtime's callback, or in a loop whose latency budget rules out cudaMalloc and anything that
may call it.  For them the entry point keeps its per-chunk score scratch in a fixed array inside
the library; they hand over inputs and the output buffer only.

The test drives the entry point through the C ABI twice in a row (the second call reuses the
scratch the first one left behind, with a different query and a different chunk count) and checks
each result against what the regular path (hkv_decode_attn -> hkv_get_selected_chunks) selects for
the same head, under the same rule the other parity tests use: equal sets, except for swaps between
chunks whose scores are tied to 1e-5.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import hkv_inputs as hi

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
            P.sets_match_up_to_ties(got, sel, scores, f"no-alloc ({b},{h})")
            n_calls += 1
    assert n_calls >= 2


def test_no_alloc_rejects_sizes_beyond_its_scratch():
    from paper_2604_05887_b200 import binding as hkv
    q = torch.zeros((7, 128), dtype=torch.bfloat16, device="cuda")
    means = torch.zeros((8, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(4, dtype=torch.int32, device="cuda")
    st = hkv.lib.hkv_topk_chunks_noalloc(q.data_ptr(), means.data_ptr(), 7, hkv.HKV_NOALLOC_MAX_CHUNKS + 1, 4,
                                         out.data_ptr(), None)
    assert st == 4                      # HKV_ERR_WORKSPACE: more chunks than the built-in scratch holds
    assert hkv.lib.hkv_topk_chunks_noalloc(q.data_ptr(), means.data_ptr(), 17, 8, 4, out.data_ptr(), None) == 5
