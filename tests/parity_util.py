"""Comparison of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs.

Index sets must be equal; an element may only be swapped for one whose ORACLE float32 score is tied
with it: |s_a - s_b| < 1e-5 * max(|s_a|, |s_b|).  A wider form, < 1e-5 * max|s| over the candidates
that are actually ranked (it covers thresholds near score zero, where a purely relative test is
ill-conditioned under a different float32 summation order), is accepted too but counted apart
("swaps_wide"): the tests of the five workloads assert that it was never needed.  Where sets differ by
permitted swaps, outputs are compared with the oracle re-run on the GPU's index set.  Outputs: max-abs
<= 2e-2 and mean-abs <= 2e-3.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import hkv_oracle as o
from paper_2604_05887_b200 import binding as hkv
from paper_2604_05887_b200.layer import LayerCache, to_device_bf16

MAX_ABS, MEAN_ABS = 2e-2, 2e-3
TIE_REL = 1e-5


def sets_match_up_to_ties(gpu_ids, ref_ids, scores_f32, what="", ranked=None):
    """Equal sets pass.  Otherwise every element the GPU took instead of one of the oracle's must be tied with
    it in the ORACLE's float32 scores.  Returns (swaps, wide): `swaps` = elements exchanged; `wide` = those of
    them that are ties only in the wide form, |s_a - s_b| < 1e-5 * max|s| over the RANKED candidates (`ranked`:
    their indices; default all), not in the strict relative form |s_a - s_b| < 1e-5 * max(|s_a|, |s_b|)."""
    g, r = set(int(x) for x in gpu_ids), set(int(x) for x in ref_ids)
    assert len(g) == len(gpu_ids), f"{what}: duplicate ids from the GPU"
    assert len(g) == len(r), f"{what}: {len(g)} ids from the GPU, {len(r)} from the oracle"
    if g == r:
        return 0, 0
    only_g = sorted(g - r, key=lambda i: -float(scores_f32[i]))
    only_r = sorted(r - g, key=lambda i: -float(scores_f32[i]))
    pool = np.asarray(scores_f32)[np.asarray(ranked, dtype=np.int64)] if ranked is not None else np.asarray(scores_f32)
    smax = float(np.abs(pool).max()) if pool.size else 0.0
    wide = 0
    for a, b in zip(only_g, only_r):
        sa, sb = float(scores_f32[a]), float(scores_f32[b])
        strict = abs(sa - sb) < TIE_REL * max(abs(sa), abs(sb))
        if not strict:
            assert abs(sa - sb) < TIE_REL * smax, f"{what}: GPU kept {a} (score {sa}) instead of {b} (score {sb}): not a tie"
            wide += 1
    return len(only_g), wide


def ranked_static_candidates(is_text_row, C, w, budget):
    """Positions whose window score takes part in a static head's ranking: the visual tokens before the window,
    or, when window + text do not fit the budget, the text tokens before it (none when budget <= w)."""
    budget = int(min(budget, C))
    if budget <= w:
        return np.zeros(0, dtype=np.int64)
    hist = np.arange(0, C - w, dtype=np.int64)
    txt = hist[np.asarray(is_text_row[:C - w]) != 0]
    return txt if txt.size >= budget - w else hist[np.asarray(is_text_row[:C - w]) == 0]


def check_outputs(gpu_out, ref_out, what=""):
    diff = np.abs(np.asarray(gpu_out, dtype=np.float64) - ref_out)
    assert np.isfinite(gpu_out).all(), f"{what}: non-finite output"
    assert diff.max() <= MAX_ABS, f"{what}: max-abs {diff.max():.3e} > {MAX_ABS}"
    assert diff.mean() <= MEAN_ABS, f"{what}: mean-abs {diff.mean():.3e} > {MEAN_ABS}"
    return float(diff.max()), float(diff.mean())


def compare_layer(L, flags=hkv.HKV_OUT_F32, token_scores=None, units=None, steps=None, check_scores=True,
                  softmax_scale=0.0):
    """Compress + decode one layer on the GPU and on the oracle; assert parity. Returns a report."""
    causal = bool(flags & hkv.HKV_CAUSAL_WINDOW)
    group_max = bool(flags & hkv.HKV_GROUP_MAX)
    lc = LayerCache(L, flags=flags, token_scores=token_scores, keep_workspace=True, softmax_scale=softmax_scale)
    code, detail = hkv.hkv_last_device_error(lc.handle)
    assert code == 0, f"device error {code}/{detail} after compress"
    all_units = [(b, h) for b in range(L.batch) for h in range(L.n_kv_heads)]
    units = all_units if units is None else units
    oc = o.compress_layer(L, token_scores=token_scores, causal_window=causal, only=units,
                          scale=softmax_scale or None)
    rep = {"swaps_static": 0, "swaps_dynamic": 0, "swaps_wide": 0, "max_abs": 0.0, "mean_abs": 0.0, "sw_rel": 0.0}
    keep_override = {}
    for (b, h) in units:
        hd = oc.heads[(b, h)]
        if hd.kind == 0:
            gi = hkv.hkv_get_static_indices(lc.handle, b, h)
            assert np.all(np.diff(gi) > 0), f"static ({b},{h}): indices not ascending"
            assert gi.size == 0 or (gi[0] >= 0 and gi[-1] < hd.C)
            if token_scores is None and check_scores:
                sw = lc.window_scores(b, h, hd.C)
                ref = hd.scores.astype(np.float64)
                rel = np.abs(sw - ref).max() / ref.max()
                rep["sw_rel"] = max(rep["sw_rel"], float(rel))
                assert rel < 2e-5, f"s_w ({b},{h}): max error {rel:.2e} of the largest score"
                assert abs(float(sw.astype(np.float64).sum()) - 1.0) < 1e-4
            n, wide = sets_match_up_to_ties(gi, hd.keep, hd.scores, f"static ({b},{h})",
                                            ranked=ranked_static_candidates(L.is_text[b], hd.C, L.obs_window, L.budgets[b, h]))
            rep["swaps_static"] += n
            rep["swaps_wide"] += wide
            if n:
                keep_override[(b, h)] = np.sort(gi.astype(np.int64))
        else:
            gs = hkv.hkv_get_summaries(lc.handle, b, h, hd.summaries.shape[0])
            assert np.array_equal(gs, hd.summaries), f"chunk means ({b},{h}) are not bit-exact"
    qs = L.q if steps is None else [L.q[s] for s in steps]
    for q_bits in qs:
        q = to_device_bf16(q_bits)
        out = lc.decode(q)
        torch.cuda.synchronize()
        code, detail = hkv.hkv_last_device_error(lc.handle)
        assert code == 0, f"device error {code}/{detail} after decode"
        _, ref_sel, ref_scores = o.decode_layer(L, oc, q_bits, scale=softmax_scale or None, group_max=group_max)
        chunk_override = {}
        for (b, h) in units:
            hd = oc.heads[(b, h)]
            if hd.kind != 1:
                continue
            gsel = hkv.hkv_get_selected_chunks(lc.handle, b, h)
            assert np.all(np.diff(gsel) > 0), f"dynamic ({b},{h}): chunk ids not ascending"
            if check_scores:
                gsc = hkv.hkv_get_chunk_scores(lc.handle, b, h, hd.summaries.shape[0])
                smax = float(np.abs(ref_scores[(b, h)]).max()) + 1e-30
                assert np.abs(gsc - ref_scores[(b, h)]).max() / smax < 1e-5, f"chunk scores ({b},{h})"
            n, wide = sets_match_up_to_ties(gsel, ref_sel[(b, h)], ref_scores[(b, h)], f"dynamic ({b},{h})")
            rep["swaps_dynamic"] += n
            rep["swaps_wide"] += wide
            if n:
                chunk_override[(b, h)] = gsel
        ref_out, _, _ = o.decode_layer(L, oc, q_bits, chunk_override=chunk_override or None,
                                       keep_override=keep_override or None, scale=softmax_scale or None,
                                       group_max=group_max)
        G = L.group
        rows = np.concatenate([np.arange(h * G, (h + 1) * G) + 0 for (_, h) in units]) if units else []
        g_out = out.float().cpu().numpy()
        mask = np.zeros((L.batch, L.n_q_heads), dtype=bool)
        for (b, h) in units:
            mask[b, h * G:(h + 1) * G] = True
        mx, mn = check_outputs(g_out[mask], ref_out[mask], f"{L.name} outputs")
        rep["max_abs"], rep["mean_abs"] = max(rep["max_abs"], mx), max(rep["mean_abs"], mn)
    rep["stats"] = lc.stats
    lc.close()
    return rep
