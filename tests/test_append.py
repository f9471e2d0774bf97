"""hkv_append: the token just generated joins the compressed cache; GPU vs oracle after every append."""
import numpy as np
import pytest
import torch

import hkv_inputs as hi
from oracle import hkv_oracle as o


def _with_room(L, cap):
    """The same inputs with `cap` unused token slots at the end of every sequence's row."""
    pad = lambda a, ax: np.concatenate([a, np.zeros(a.shape[:ax] + (cap,) + a.shape[ax + 1:], dtype=a.dtype)], axis=ax)
    L.k, L.v, L.is_text = pad(L.k, 2), pad(L.v, 2), pad(L.is_text, 1)
    L.max_seq_len += cap
    return L


def test_oracle_append_equals_compressing_the_longer_sequence_for_dynamic_heads():
    """Pin: appended metadata = metadata of the longer sequence built from scratch; the static keep-set only grows."""
    L = _with_room(hi.tiny(seed=3, B=2, C=61, chunk_size=8, w=4, Hq=4, Hkv=2, d=16, budget_fraction=0.3), 20)
    oc = o.compress_layer(L)
    keep0 = {k: v.keep.copy() for k, v in oc.heads.items() if v.kind == 0}
    rng = np.random.default_rng(0)
    for t in range(20):
        kn = hi.f32_to_bf16_bits(rng.standard_normal((2, 2, 16)).astype(np.float32))
        o.append_token(L, oc, kn, kn)
    for (b, h), hd in oc.heads.items():
        C = int(L.seq_lens[b])
        assert hd.C == C
        if hd.kind == 1:
            assert np.array_equal(hd.summaries, o.chunk_summaries(L.k[b, h, :C], 8))
            assert hd.n_sel == o.n_selected_chunks(int(L.budgets[b, h]), 8, (C + 7) // 8)
        else:
            assert np.array_equal(hd.keep[:keep0[(b, h)].size], keep0[(b, h)])
            assert hd.keep[-20:].tolist() == list(range(C - 20, C))


@pytest.mark.gpu
@pytest.mark.parametrize("cs,C,budget,cap,offload", [(16, 500, 0.2, 40, False), (32, 1000, 1.0, 70, False),
                                                     (8, 333, 0.5, 19, False), (64, 700, 0.1, 130, False),
                                                     (16, 450, 0.3, 25, True)])
def test_append_matches_oracle_step_by_step(cs, C, budget, cap, offload):
    import parity_util as P
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    L = hi.tiny(seed=cs + C, B=2, C=C, chunk_size=cs, w=8, Hq=28, Hkv=4, d=128, budget_fraction=budget, n_steps=1)
    if budget >= 1.0:
        L.budgets[:] = 10 ** 6                                   # "everything", also after the sequence has grown
    L = _with_room(L, cap)
    lc = LayerCache(L, flags=hkv.HKV_OUT_F32 | (hkv.HKV_OFFLOAD_DYNAMIC if offload else 0), append_capacity=cap)
    oc = o.compress_layer(L)
    rng = np.random.default_rng(cs)
    G = L.group
    for t in range(cap):
        kn = hi.f32_to_bf16_bits(rng.standard_normal((L.batch, L.n_kv_heads, 128)).astype(np.float32))
        vn = hi.f32_to_bf16_bits(rng.standard_normal((L.batch, L.n_kv_heads, 128)).astype(np.float32))
        lc.append(to_device_bf16(kn), to_device_bf16(vn))
        o.append_token(L, oc, kn, vn)
        if t % 7 and t != cap - 1:
            continue                                             # check every few tokens and at the end
        q_bits = hi.f32_to_bf16_bits(rng.standard_normal((L.batch, L.n_q_heads, 128)).astype(np.float32))
        out = lc.decode(to_device_bf16(q_bits))
        torch.cuda.synchronize()
        assert hkv.hkv_last_device_error(lc.handle) == (0, 0)
        _, ref_sel, ref_scores = o.decode_layer(L, oc, q_bits)
        override = {}
        for (b, h), hd in oc.heads.items():
            if hd.kind == 0:
                assert np.array_equal(hkv.hkv_get_static_indices(lc.handle, b, h), hd.keep)
            else:
                assert np.array_equal(hkv.hkv_get_summaries(lc.handle, b, h, hd.summaries.shape[0]), hd.summaries)
                gsel = hkv.hkv_get_selected_chunks(lc.handle, b, h)
                if P.sets_match_up_to_ties(gsel, ref_sel[(b, h)], ref_scores[(b, h)], f"step {t} ({b},{h})")[0]:
                    override[(b, h)] = gsel
        ref_out, _, _ = o.decode_layer(L, oc, q_bits, chunk_override=override or None)
        P.check_outputs(out.cpu().numpy(), ref_out, f"after {t + 1} appended tokens")
    assert lc.stats["retained_tokens"] > 0
    with pytest.raises(hkv.HkvError) as e:                       # capacity used up
        lc.append(to_device_bf16(kn), to_device_bf16(vn))
    assert e.value.status == 4
    lc.close()
