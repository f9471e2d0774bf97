"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, plans sizes, and rejects bad arguments before any launch."""
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def hkv():
    from paper_2604_05887_b200.build import build_library
    build_library()
    from paper_2604_05887_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(hkv):
    header = open(os.path.join(ROOT, "include", "hkv.h")).read()
    # the development section (checked / profiling builds) is not part of the product library
    dev = re.findall(r"#ifdef HKV_(?:CHECKED|PROFILE)\n(.*?)#endif", header, flags=re.S)
    product = header
    for block in dev:
        product = product.replace(block, "")
    declared = set(re.findall(r"\b(hkv_[a-z_]+)\s*\(", product))
    assert declared, "no declarations found"
    assert declared == set(hkv.EXPORTS)
    for name in declared:
        assert hasattr(hkv.lib, name), name
    dev_names = set(re.findall(r"\b(hkv_[a-z_]+)\s*\(", "".join(dev)))
    assert dev_names == {"hkv_selftest_wait_timeout", "hkv_clear_device_error", "hkv_profile_attach"}
    for name in dev_names:
        assert not hasattr(hkv.lib, name), f"{name} must not be in the product library"


def test_development_builds_export_their_extra_symbols():
    """The checked and the profiling build are the same sources with one more macro; each exports the product's
    symbols plus its own (nothing is launched here)."""
    import ctypes
    from paper_2604_05887_b200 import build
    for path, extra in ((build.build_checked(), ["hkv_selftest_wait_timeout", "hkv_clear_device_error"]),
                        (build.build_profile(), ["hkv_profile_attach"])):
        lib = ctypes.CDLL(path)
        for name in list(hkv_exports()) + extra:
            assert hasattr(lib, name), (path, name)


def hkv_exports():
    from paper_2604_05887_b200 import binding
    return binding.EXPORTS


def test_status_strings(hkv):
    assert hkv.status_string(0) == "ok"
    assert len({hkv.status_string(i) for i in range(9)}) == 9


def _cfg(hkv, **kw):
    base = dict(batch=2, n_q_heads=28, n_kv_heads=4, head_dim=128, max_seq_len=1000, chunk_size=32, obs_window=32)
    base.update(kw)
    return hkv.make_config(**base)


def test_plan_sizes_grow_with_budget_and_are_aligned(hkv):
    sl, ht = [1000, 900], [[0, 1, 0, 1]] * 2
    c1, w1 = hkv.hkv_plan(_cfg(hkv), sl, ht, np.full((2, 4), 100))
    c2, w2 = hkv.hkv_plan(_cfg(hkv), sl, ht, np.full((2, 4), 500))
    assert c1 % 256 == 0 and w1 % 256 == 0 and c2 > c1 and w1 == w2
    # dynamic heads keep the whole K/V resident: at least 2 * 256 B per token
    assert c1 > 2 * 2 * 256 * 900


@pytest.mark.parametrize("kw,sl,ht,bu,status", [
    (dict(head_dim=64), [1000, 900], 0, 100, 5),
    (dict(n_q_heads=30), [1000, 900], 0, 100, 2),
    (dict(n_q_heads=68, n_kv_heads=4), [1000, 900], 0, 100, 5),
    (dict(), [1001, 900], 0, 100, 2),
    (dict(), [1000, 0], 0, 100, 2),
    (dict(obs_window=901), [1000, 900], 0, 100, 2),
    (dict(), [1000, 900], 2, 100, 1),
    (dict(), [1000, 900], 0, 0, 3),
    (dict(chunk_size=0), [1000, 900], 0, 100, 2),
    (dict(flags=64), [1000, 900], 0, 100, 1),
])
def test_plan_rejects_bad_arguments(hkv, kw, sl, ht, bu, status):
    with pytest.raises(hkv.HkvError) as e:
        hkv.hkv_plan(_cfg(hkv, **kw), sl, np.full((2, 4), ht), np.full((2, 4), bu))
    assert e.value.status == status


def test_null_pointers_are_rejected(hkv):
    import ctypes as C
    cb, wb = C.c_size_t(0), C.c_size_t(0)
    assert hkv.lib.hkv_plan(None, None, None, None, C.byref(cb), C.byref(wb)) == 1
    assert hkv.lib.hkv_decode_attn(None, None, None, None) == 1
    assert hkv.lib.hkv_cache_stats(None, None) == 1
    h = C.c_void_p(None)
    cfg = _cfg(hkv)
    assert hkv.lib.hkv_compress(C.byref(cfg), None, None, None, None, None, None, None, None, None, 0, None, 0, None,
                                C.byref(h)) == 1
    assert h.value is None
    assert hkv.lib.hkv_cache_destroy(None) == 0


def test_plan_of_bench_shape_keeps_only_the_compressed_cache(hkv):
    """cfg2-shaped layer: cache_mem stays far below the layer's full K/V."""
    from paper_2604_05887_b200.binding import hkv_config
    import ctypes as C
    sl = [32768, 30000, 27000, 25000]
    ht = np.array([[0, 1, 0, 0], [1, 0, 1, 0], [0, 0, 1, 1], [0, 1, 0, 0]])
    bu = np.array([[int(np.ceil(0.1 * c))] * 4 for c in sl])
    cfg = _cfg(hkv, batch=4, max_seq_len=32768, chunk_size=64)
    cache_bytes, _ = hkv.hkv_plan(cfg, sl, ht, bu)
    assert cache_bytes < 2 * 256 * 32768 * 16      # far below the full KV of the layer


def test_classification_workspace_sizes(hkv):
    """hkv_classify_workspace is host arithmetic: 256 B error word + row sums + at least 16 rows of logits per
    (sequence, kv head) for the minimum, every row (up to half a gigabyte of logits) for the preferred size."""
    cfg = _cfg(hkv, max_seq_len=1000)
    lo, hi = hkv.hkv_classify_workspace(cfg, 10)
    units, r_max, c_stride = 2 * 4, 10 * 7, 1024          # rows padded to a multiple of 128 floats
    head = 256 + -(-units * r_max * 4 // 256) * 256
    assert lo == head + 16 * c_stride * 4 * units
    assert hi == head + 80 * c_stride * 4 * units          # 70 rows rounded up to a multiple of 16
    lo2, hi2 = hkv.hkv_classify_workspace(cfg, 1000)
    assert lo2 > lo and hi2 > hi and lo2 <= hi2
    big = _cfg(hkv, batch=16, max_seq_len=32768)
    lo3, hi3 = hkv.hkv_classify_workspace(big, 768)
    assert hi3 - lo3 < (512 << 20) + (16 << 20) and hi3 > (256 << 20)
    for bad, status in ((dict(head_dim=64), 5), (dict(n_q_heads=30), 2), (dict(batch=0), 2)):
        with pytest.raises(hkv.HkvError) as e:
            hkv.hkv_classify_workspace(_cfg(hkv, **bad), 10)
        assert e.value.status == status
    with pytest.raises(hkv.HkvError):
        hkv.hkv_classify_workspace(cfg, 0)
