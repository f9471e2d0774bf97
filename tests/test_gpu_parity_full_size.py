"""The five workloads at their stated sizes, CUDA path vs CPU oracle through the C ABI (needs a B200).

Each case runs in the launch shape the benchmark times (same batch, lengths, chunk size, budgets, hence the same
cluster size and tile split); the oracle checks units one by one.  Index sets must match under the strict tie rule:
`swaps_wide` (swaps that only the wide form of the rule would accept) is asserted to be zero on every workload."""
import numpy as np
import pytest
import torch

import hkv_inputs as hi

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import parity_util
    return parity_util


def _textbook(L, q_bits, b, h):
    """Full-cache softmax attention of one (sequence, kv head) group by the library routine, float64."""
    C, G = int(L.seq_lens[b]), L.group
    f = lambda u: torch.from_numpy(np.ascontiguousarray(u)).view(torch.bfloat16).to(torch.float64)
    Q = f(q_bits[b, h * G:(h + 1) * G])[None, :, None, :]
    K = f(L.k[b, h, :C])[None, None].expand(1, G, C, 128)
    V = f(L.v[b, h, :C])[None, None].expand(1, G, C, 128)
    return torch.nn.functional.scaled_dot_product_attention(Q, K, V)[0, :, 0].numpy()


def test_cfg0_every_unit_and_step(P):
    rep = P.compare_layer(hi.cfg0(n_steps=4))
    assert rep["swaps_wide"] == 0, rep


@pytest.mark.parametrize("layer", [0, 17])
def test_cfg1_all_eight_steps(P, layer):
    """28 layers x 8 consecutive steps, each query seeded: two layers, every unit, all 8 steps."""
    L = hi.cfg1(layer=layer, n_steps=8)
    rep = P.compare_layer(L)
    assert rep["swaps_wide"] == 0, rep
    print("cfg1 layer", layer, {k: rep[k] for k in ("max_abs", "mean_abs", "swaps_static", "swaps_dynamic", "swaps_wide")})


@pytest.mark.parametrize("layer", [0, 5])
def test_cfg2_all_sixteen_units(P, layer):
    """B=4, 24K-32K tokens, chunk 64: every (sequence, kv head) unit of two layers, two seeded queries."""
    L = hi.cfg2(layer=layer, n_steps=2)
    rep = P.compare_layer(L)
    assert rep["stats"]["n_static"] == 10 and rep["stats"]["n_dynamic"] == 6
    assert rep["swaps_wide"] == 0, rep
    print("cfg2 layer", layer, {k: rep[k] for k in ("max_abs", "mean_abs", "swaps_static", "swaps_dynamic", "swaps_wide")})


def test_cfg3_batch_eight_planted_chunks_recovered(P):
    """B=8, 50 000 tokens, 5 %, chunk 32 (32 units, 1563 chunks, k = 79): the oracle on ten sampled units of both
    types, and the three planted chunks among the selected ones on EVERY dynamic unit."""
    from paper_2604_05887_b200 import binding as hkv
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    L = hi.cfg3(layer=0)
    assert L.batch == 8 and int(L.seq_lens[0]) == 50000
    dyn = [(b, h) for b in range(8) for h in range(4) if L.head_type[b, h] == 1]
    sta = [(b, h) for b in range(8) for h in range(4) if L.head_type[b, h] == 0]
    units = dyn[::3][:6] + sta[::4][:4]
    rep = P.compare_layer(L, units=units)
    assert rep["swaps_wide"] == 0, rep
    lc = LayerCache(L)
    lc.decode(to_device_bf16(L.q[0]))
    torch.cuda.synchronize()
    assert hkv.hkv_last_device_error(lc.handle) == (0, 0)
    for (b, h) in dyn:
        sel = hkv.hkv_get_selected_chunks(lc.handle, b, h)
        assert sel.size == 79
        assert set(L.planted[b, h].tolist()) <= set(sel.tolist()), (b, h)
    lc.close()
    print("cfg3 B=8", {k: rep[k] for k in ("max_abs", "mean_abs", "swaps_static", "swaps_dynamic", "swaps_wide")})


@pytest.mark.parametrize("sf,cs", [(0.5, 64), (0.0, 16), (1.0, 128)])
def test_cfg4_full_budget_cells_equal_textbook_attention(P, sf, cs):
    """The 100 % cells at full size (B=16, 32768 tokens): every sampled unit against full-cache attention."""
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    L = hi.cfg4(1.00, sf, cs)
    lc = LayerCache(L, flags=2)
    out = lc.decode(to_device_bf16(L.q[0])).cpu().numpy()
    torch.cuda.synchronize()
    G = L.group
    for (b, h) in [(0, 0), (3, 1), (7, 2), (11, 3), (15, 0), (8, 1)]:
        P.check_outputs(out[b, h * G:(h + 1) * G], _textbook(L, L.q[0], b, h), f"100 % cell sf={sf} cs={cs} unit ({b},{h})")
    lc.close()


def test_cfg4_all_hundred_cells_reduced_length(P):
    """Every (budget, static fraction, chunk) cell of the sweep at B=4 and 4096 tokens: indices, scores, outputs."""
    wide = swaps = 0
    for bf in hi.CFG4_BUDGETS:
        for sf in hi.CFG4_STATIC_FRACTIONS:
            for cs in hi.CFG4_CHUNKS:
                L = hi.cfg4(bf, sf, cs, B=4, C=4096, block=512)
                rep = P.compare_layer(L)
                wide += rep["swaps_wide"]
                swaps += rep["swaps_static"] + rep["swaps_dynamic"]
    assert wide == 0
    print("cfg4 100 cells: swaps under the strict tie rule", swaps)
