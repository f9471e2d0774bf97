"""CUDA path vs CPU oracle, through the C ABI, on the same seeded inputs (needs a B200)."""
import math

import numpy as np
import pytest
import torch

import hkv_inputs as hi
from oracle import hkv_oracle as o

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import parity_util
    return parity_util


def _geom(L, **kw):
    for k, v in kw.items():
        setattr(L, k, v)
    return L


def small(seed=5, B=2, C=700, cs=16, w=8, Hq=28, Hkv=4, budget=0.2, ragged=True, head_type=None, n_steps=2):
    """cfg0-like values with free sizes (head_dim stays 128)."""
    L = hi.tiny(seed=seed, B=B, C=C, chunk_size=cs, w=w, Hq=Hq, Hkv=Hkv, d=128, budget_fraction=budget,
                n_steps=n_steps, ragged=ragged, head_type=head_type)
    return L


def test_cfg0_parity(P):
    L = hi.cfg0(n_steps=3)
    rep = P.compare_layer(L)
    assert rep["stats"]["n_static"] == 2 and rep["stats"]["n_dynamic"] == 2
    print("cfg0", rep)


def test_cfg0_bf16_output(P):
    L = hi.cfg0()
    rep = P.compare_layer(L, flags=0)
    print("cfg0 bf16 out", rep)


@pytest.mark.parametrize("cs", [1, 7, 8, 16, 24, 32, 64, 128, 1000])
def test_chunk_sizes(P, cs):
    L = small(cs=cs, C=700, budget=0.23)
    P.compare_layer(L)


@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (8, 2), (28, 4), (16, 2), (24, 2), (16, 1)])
def test_group_sizes(P, Hq, Hkv):
    L = small(Hq=Hq, Hkv=Hkv, C=500, cs=16, B=2)
    P.compare_layer(L)


@pytest.mark.parametrize("budget_tokens", [1, 3, 8, 9, 40, 41, 300, 499, 500, 10 ** 6])
def test_budget_edges(P, budget_tokens):
    # window w = 8; #text before the window is ~ 30: covers budget < w, = w, window+text not fitting, full
    L = small(C=500, cs=16, w=8, ragged=False, B=1, head_type=[[0, 1, 0, 1]])
    L.budgets[:] = budget_tokens
    rep = P.compare_layer(L)
    if budget_tokens >= 500:
        assert rep["stats"]["retained_tokens"] == 4 * 500


def test_full_budget_matches_textbook_attention(P):
    """100 % budget: both head types reduce to full-cache GQA attention (library routine)."""
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    L = small(C=1500, cs=32, B=2, head_type=[[0, 1, 1, 0], [1, 0, 0, 1]])
    L.budgets[:] = L.seq_lens[:, None]
    lc = LayerCache(L, flags=hkv.HKV_OUT_F32)
    out = lc.decode(to_device_bf16(L.q[0])).cpu().numpy()
    for b in range(L.batch):
        C = int(L.seq_lens[b])
        f = lambda u: torch.from_numpy(np.ascontiguousarray(u)).view(torch.bfloat16).to(torch.float64)
        Q = f(L.q[0][b])[None, :, None, :]
        K = f(L.k[b, :, :C]).repeat_interleave(L.group, dim=0)[None]
        V = f(L.v[b, :, :C]).repeat_interleave(L.group, dim=0)[None]
        ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V)[0, :, 0].numpy()
        P.check_outputs(out[b], ref, "full budget")


def test_token_scores_override(P):
    L = small(C=600, cs=16, B=2)
    rng = np.random.default_rng(9)
    ts = rng.standard_normal((L.batch, L.n_kv_heads, L.max_seq_len)).astype(np.float32)
    ts[0, :, 100:140] = 0.25          # a run of exact ties: the lower positions must win
    ts[1, :, 7] = -0.0
    ts[1, :, 9] = 0.0
    P.compare_layer(L, token_scores=ts)


def test_causal_window_variant(P):
    from paper_2604_05887_b200 import binding as hkv
    L = small(C=400, cs=16, w=16)
    P.compare_layer(L, flags=hkv.HKV_OUT_F32 | hkv.HKV_CAUSAL_WINDOW)


@pytest.mark.parametrize("w,Hq,Hkv,causal", [(48, 28, 4, False), (48, 28, 4, True), (40, 32, 2, False), (32, 8, 4, True)])
def test_window_rows_beyond_one_resident_block(P, w, Hq, Hkv, causal):
    """w * G = 336 and 640 window rows: the window-score kernels run once per block of 256 rows, the later blocks
    adding to s_w; (32, 8, 4) has 64 rows, a quarter of one block, the rest being padding."""
    from paper_2604_05887_b200 import binding as hkv
    L = small(B=2, C=900, cs=16, w=w, Hq=Hq, Hkv=Hkv, budget=0.3, n_steps=1)
    P.compare_layer(L, flags=hkv.HKV_OUT_F32 | (hkv.HKV_CAUSAL_WINDOW if causal else 0))


@pytest.mark.parametrize("Hq,Hkv", [(28, 4), (32, 2), (4, 4), (16, 2)])
def test_group_max_scoring_variant(P, Hq, Hkv):
    """HKV_GROUP_MAX: the chunk score is the largest inner product of the group (groups of 7, 16, 1, 8)."""
    from paper_2604_05887_b200 import binding as hkv
    L = small(B=2, C=1100, cs=16, w=8, Hq=Hq, Hkv=Hkv, budget=0.25, n_steps=2, head_type=np.ones((2, Hkv), np.uint8))
    rep = P.compare_layer(L, flags=hkv.HKV_OUT_F32 | hkv.HKV_GROUP_MAX)
    assert rep["stats"]["n_dynamic"] == 2 * Hkv


def test_offloaded_dynamic_heads_variant(P):
    """HKV_OFFLOAD_DYNAMIC: the dynamic heads' K/V planes sit in pinned host memory; same results, two steps."""
    from paper_2604_05887_b200 import binding as hkv
    L = small(B=2, C=1300, cs=16, w=8, budget=0.2, n_steps=2)
    rep = P.compare_layer(L, flags=hkv.HKV_OUT_F32 | hkv.HKV_OFFLOAD_DYNAMIC)
    assert rep["stats"]["n_dynamic"] > 0
    # all static: no host buffer at all
    Ls = small(B=1, C=600, cs=16, w=8, budget=0.2, n_steps=1, head_type=np.zeros((1, 4), np.uint8))
    P.compare_layer(Ls, flags=hkv.HKV_OUT_F32 | hkv.HKV_OFFLOAD_DYNAMIC)
    # the plain entry points refuse the flag, the offload ones its absence, and device memory is not host memory
    cfg = hkv.make_config(L.batch, L.n_q_heads, L.n_kv_heads, 128, L.max_seq_len, 16, 8, 0.0, hkv.HKV_OFFLOAD_DYNAMIC, 0)
    with pytest.raises(hkv.HkvError):
        hkv.hkv_plan(cfg, L.seq_lens, L.head_type, L.budgets)
    cfg0 = hkv.make_config(L.batch, L.n_q_heads, L.n_kv_heads, 128, L.max_seq_len, 16, 8, 0.0, 0, 0)
    with pytest.raises(hkv.HkvError):
        hkv.hkv_plan_offload(cfg0, L.seq_lens, L.head_type, L.budgets)
    cb, wb, hb = hkv.hkv_plan_offload(cfg, L.seq_lens, L.head_type, L.budgets)
    assert hb > 0 and hb % 256 == 0
    import torch
    dev_buf = torch.empty(hb, dtype=torch.uint8, device="cuda")
    z = torch.zeros(8, dtype=torch.uint8, device="cuda")
    st = hkv.lib.hkv_compress_offload(hkv.C.byref(cfg), z.data_ptr(), z.data_ptr(), z.data_ptr(), None, z.data_ptr(),
                                      hkv._ptr(hkv._i32(L.seq_lens), hkv.C.c_int32),
                                      hkv._ptr(hkv._u8(L.head_type), hkv.C.c_uint8),
                                      hkv._ptr(hkv._i32(L.budgets), hkv.C.c_int32),
                                      torch.empty(cb, dtype=torch.uint8, device="cuda").data_ptr(), cb,
                                      dev_buf.data_ptr(), hb, torch.empty(wb, dtype=torch.uint8, device="cuda").data_ptr(),
                                      wb, None, hkv.C.byref(hkv.C.c_void_p(None)))
    assert st == 1        # HKV_ERR_INVALID_ARG before anything is launched


def test_second_geometry_qwen25_vl_3b(P):
    """16 query / 2 KV heads (group of 8), head_dim 128: the smaller model the paper also evaluates."""
    L = small(B=3, C=5000, cs=32, w=32, Hq=16, Hkv=2, budget=0.1, n_steps=2)
    rep = P.compare_layer(L)
    assert rep["stats"]["n_static"] + rep["stats"]["n_dynamic"] == 6


def test_custom_scale(P):
    L = small(C=300, cs=8)
    P.compare_layer(L, softmax_scale=0.05)


def test_ragged_tail_chunk_and_many_splits(P):
    L = small(C=5003, cs=32, B=3, budget=0.6, w=32)
    rep = P.compare_layer(L)
    assert rep["stats"]["n_splits"] > L.batch * L.n_kv_heads


def test_more_chunks_than_fit_shared_memory(P):
    """chunk size 1 on a few thousand tokens: the selection works on scores and id lists in global memory."""
    L = small(C=2600, cs=1, B=1, budget=0.3, w=16, head_type=[[1, 0, 1, 1]])
    rep = P.compare_layer(L)
    L = small(C=2300, cs=1, B=2, budget=1.0, w=16)          # every chunk selected: no list at all
    P.compare_layer(L)


def test_back_to_back_steps_overlap_safely(P):
    """Several decode launches in a row on one stream (each may start before its predecessor has
    finished): every step's output must still match a step run in isolation."""
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    L = hi.cfg1(layer=0, C=4096, block=512, n_steps=6)
    lc = LayerCache(L)
    qs = [to_device_bf16(q) for q in L.q]
    alone = []
    for q in qs:
        alone.append(lc.decode(q).clone())
        torch.cuda.synchronize()
    outs = [lc.new_out() for _ in qs]
    for rep in range(3):
        for q, o_ in zip(qs, outs):
            lc.decode(q, o_)
    torch.cuda.synchronize()
    for a, b in zip(alone, outs):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    lc.close()


def test_determinism_and_static_independent_of_dynamic_budget():
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    L = small(C=3000, cs=32, B=2, head_type=[[0, 1, 1, 0], [1, 0, 0, 1]])
    q = to_device_bf16(L.q[0])
    outs = []
    for rep in range(2):
        lc = LayerCache(L)
        a = lc.decode(q).clone()
        b = lc.decode(q).clone()
        torch.cuda.synchronize()
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
        outs.append(a)
        lc.close()
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))
    L.budgets[L.head_type == 1] = 1700
    lc = LayerCache(L)
    c = lc.decode(q)
    torch.cuda.synchronize()
    G = L.group
    for b in range(L.batch):
        for h in range(L.n_kv_heads):
            same = torch.equal(c[b, h * G:(h + 1) * G].view(torch.int16), outs[0][b, h * G:(h + 1) * G].view(torch.int16))
            assert same == (L.head_type[b, h] == 0)


def test_multi_layer_launch_equals_single_calls():
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    Ls = [hi.cfg1(layer=l, C=2048, block=256, n_steps=1) for l in range(3)]
    lcs = [LayerCache(L) for L in Ls]
    qs = [to_device_bf16(L.q[0]) for L in Ls]
    single = [lc.decode(q).clone() for lc, q in zip(lcs, qs)]
    outs = [lc.new_out() for lc in lcs]
    hkv.hkv_decode_attn_multi([lc.handle for lc in lcs], qs, outs)
    torch.cuda.synchronize()
    for a, b in zip(single, outs):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_cfg1_layer(P):
    L = hi.cfg1(layer=2, n_steps=2)
    rep = P.compare_layer(L)
    print("cfg1", rep)


def test_cfg2_reduced(P):
    L = hi.cfg2(layer=1, B=2, n_frames=12, min_frames=9)
    rep = P.compare_layer(L)
    print("cfg2 reduced", rep)


def test_cfg3_reduced_planted_chunks(P):
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    L = hi.cfg3(layer=0, B=2, C=5000, block=512)
    P.compare_layer(L)
    lc = LayerCache(L)
    lc.decode(to_device_bf16(L.q[0]))
    for b in range(L.batch):
        for h in range(L.n_kv_heads):
            if L.head_type[b, h] == 1:
                sel = hkv.hkv_get_selected_chunks(lc.handle, b, h)
                assert set(L.planted[b, h].tolist()) <= set(sel.tolist())


@pytest.mark.parametrize("budget,sf,cs", [(0.05, 0.5, 16), (0.2, 0.25, 128), (0.5, 0.75, 64), (1.0, 0.5, 32)])
def test_cfg4_cells_reduced(P, budget, sf, cs):
    L = hi.cfg4(budget, sf, cs, B=4, C=4096, block=512)
    P.compare_layer(L)


def test_cfg2_full_size_sampled_units(P):
    """Bench configuration at full size (B=4, 32768 tokens, chunk 64): the launch shape bench.py times;
    the oracle checks a sample of (b, h) units one by one."""
    L = hi.cfg2(layer=0)
    units = [(0, 0), (0, 3), (1, 1), (2, 2), (3, 0), (3, 3)]
    rep = P.compare_layer(L, units=units)
    print("cfg2 full", rep)


def test_cfg3_full_length_sampled_units(P):
    L = hi.cfg3(layer=0, B=2)
    rep = P.compare_layer(L, units=[(0, 0), (0, 1), (1, 2), (1, 3)])
    print("cfg3 50000", rep)


def test_cfg4_full_size_cell_sampled(P):
    L = hi.cfg4(0.10, 0.5, 32)
    rep = P.compare_layer(L, units=[(0, 0), (5, 1), (9, 2), (15, 3)])
    print("cfg4 cell", rep)


@pytest.mark.parametrize("budget,sf,cs,units", [
    (1.00, 0.5, 64, [(0, 0), (7, 2), (15, 3)]),       # full budget: both head types equal full-cache attention
    (0.05, 0.25, 16, [(1, 1), (8, 0), (14, 2)]),      # 2048 chunk means per head, k = 103
    (0.50, 0.75, 128, [(2, 3), (9, 1), (13, 0)]),
])
def test_cfg4_full_size_more_cells_sampled(P, budget, sf, cs, units):
    """More cells of the B=16, 32768-token sweep at full size, in the launch shape the sweep times."""
    L = hi.cfg4(budget, sf, cs)
    rep = P.compare_layer(L, units=units)
    if budget >= 1.0:
        # the oracle's answer at 100 % is itself pinned to textbook attention (test_oracle_pins); check one unit here too
        b, h = units[0]
        C, G = int(L.seq_lens[b]), L.group
        f = lambda u: torch.from_numpy(np.ascontiguousarray(u)).view(torch.bfloat16).to(torch.float64)
        from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
        lc = LayerCache(L, flags=2)
        out = lc.decode(to_device_bf16(L.q[0])).cpu().numpy()
        Q = f(L.q[0][b, h * G:(h + 1) * G])[None, :, None, :]
        K = f(L.k[b, h, :C])[None, None].expand(1, G, C, 128)
        V = f(L.v[b, h, :C])[None, None].expand(1, G, C, 128)
        ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V)[0, :, 0].numpy()
        P.check_outputs(out[b, h * G:(h + 1) * G], ref, "full budget vs textbook attention")
        lc.close()
    print("cfg4 cell", budget, sf, cs, {k: rep[k] for k in ("max_abs", "mean_abs", "swaps_dynamic")})


def test_host_buffer_entry_points_equal_device_calls():
    """hkv_decode_attn_host (one layer) and hkv_decode_step_host (all layers, one transfer each way)."""
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    Ls = [hi.cfg1(layer=l, C=2048, block=256, n_steps=1) for l in range(3)]
    lcs = [LayerCache(L) for L in Ls]
    qs = [to_device_bf16(L.q[0]) for L in Ls]
    ref = [lc.decode(q).clone() for lc, q in zip(lcs, qs)]
    torch.cuda.synchronize()
    q_host = torch.stack([q.cpu() for q in qs]).pin_memory()
    out_host = torch.zeros_like(q_host).pin_memory()
    q_dev, out_dev = torch.empty_like(q_host, device="cuda"), torch.empty_like(q_host, device="cuda")
    hkv.hkv_decode_step_host([lc.handle for lc in lcs], q_host, out_host, q_dev, out_dev)
    torch.cuda.synchronize()
    for i in range(3):
        assert torch.equal(out_host[i].view(torch.int16), ref[i].cpu().view(torch.int16))
    one = torch.zeros_like(q_host[1]).pin_memory()
    hkv.hkv_decode_attn_host(lcs[1].handle, q_host[1], one, q_dev[1], out_dev[1])
    torch.cuda.synchronize()
    assert torch.equal(one.view(torch.int16), ref[1].cpu().view(torch.int16))
    for lc in lcs:
        lc.close()


def test_more_units_than_clusters_fit(P):
    """200 (sequence, head) units: the launch falls back to one CTA per unit (no cluster, no cross-CTA merge)."""
    L = small(B=50, C=260, cs=16, w=8, budget=0.3, n_steps=1)
    rep = P.compare_layer(L)
    assert rep["stats"]["n_splits"] == 200


def _expected_cluster(caps, units, tiles):
    c = max([1] + [t for t in range(2, 17, 2) if caps[t] >= units and 2 * t <= tiles])
    return 10 if c > 10 and tiles <= 160 else c


def test_unit_counts_that_select_every_cluster_size(P):
    """1, 2, 4, 6, 8, 10, 12 or 16 CTAs per unit: the launch picks the largest even size (or 1) that fits all units
    in one wave and leaves a CTA two tiles, capped at 10 for short token lists; sizes need not be powers of two."""
    from paper_2604_05887_b200 import binding as hkv
    caps = hkv.hkv_decode_cluster_capacity(7)
    seen = set()
    for B in (1, 6, 8, 10, 12, 30, 50):
        L = small(B=B, C=2200, cs=32, w=8, budget=0.5, n_steps=1, ragged=False)
        rep = P.compare_layer(L, units=[(0, 0), (B - 1, 3), (B // 2, 1), (B // 2, 2)])
        size = rep["stats"]["n_splits"] // (4 * B)
        assert size == _expected_cluster(caps, 4 * B, (1100 + 31) // 32), (B, size, caps)
        seen.add(size)
    for B in (1, 4):                       # long lists (188 tiles per unit): the cap does not apply
        L = small(B=B, C=6000, cs=32, w=8, budget=1.0, n_steps=1, ragged=False)
        rep = P.compare_layer(L, units=[(0, 0), (B - 1, 3)])
        size = rep["stats"]["n_splits"] // (4 * B)
        assert size == _expected_cluster(caps, 4 * B, (6000 + 31) // 32), (B, size, caps)
        seen.add(size)
    assert {1, 2, 4, 6, 8, 10, 12, 16} <= seen, (seen, caps)


@pytest.mark.parametrize("case", range(24))
def test_random_shapes(P, case):
    """Seeded random geometry: batch, lengths, chunk size, window, group size, per-head budgets and types."""
    rng = np.random.default_rng(1000 + case)
    Hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 4, 7, 8, 12, 16]))
    B = int(rng.integers(1, 7))
    C = int(rng.integers(80, 3000))
    cs = int(rng.choice([1, 3, 8, 16, 20, 32, 64, 96, 128, 500]))
    w = int(rng.integers(1, min(48, C - 5 * B - 1)))
    L = hi.tiny(seed=2000 + case, B=B, C=C, chunk_size=cs, w=w, Hq=G * Hkv, Hkv=Hkv, d=128, budget_fraction=0.2,
                n_steps=2, ragged=bool(case & 1))
    L.head_type = rng.integers(0, 2, size=(B, Hkv)).astype(np.uint8)
    L.budgets = rng.integers(1, C + 50, size=(B, Hkv)).astype(np.int32)
    units = [(b, h) for b in range(B) for h in range(Hkv)]
    if len(units) > 8:
        units = [units[i] for i in rng.choice(len(units), size=8, replace=False)]
    P.compare_layer(L, units=units)

