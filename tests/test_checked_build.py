"""The checked build of the library (same sources, -DHKV_CHECKED and a wait limit of a fraction of a second)
through the C ABI on a B200: index validation must stay silent on valid inputs, and a device-side wait that can
never be satisfied must give up by itself, leave HKV_ERR_TIMEOUT in the error word and leave the context usable.
Nothing here faults, traps or spins without a bound: the only "failure" is a barrier that nothing arrives on,
waited for by a loop with a cycle limit."""
import ctypes

import numpy as np
import pytest
import torch

import hkv_inputs as hi

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def checked():
    from paper_2604_05887_b200 import binding, build
    lib = binding.use_library(build.build_checked())
    lib.hkv_selftest_wait_timeout.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
    lib.hkv_selftest_wait_timeout.restype = ctypes.c_int
    lib.hkv_clear_device_error.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
    lib.hkv_clear_device_error.restype = ctypes.c_int
    yield binding
    binding.use_library(None)


def _small(**kw):
    base = dict(seed=5, B=2, C=700, chunk_size=16, w=8, Hq=28, Hkv=4, d=128, budget_fraction=0.2, n_steps=2, ragged=True)
    base.update(kw)
    return hi.tiny(**base)


@pytest.mark.parametrize("case", ["cfg0", "ragged", "cs7", "many_chunks", "wide_group", "one_cta_per_unit"])
def test_checked_build_matches_the_oracle_and_reports_no_error(checked, case):
    """Every index check of the decode kernel is live in this build; compare_layer asserts the error word is (0, 0)
    after compression and after every decode step, and parity as in the product build."""
    import parity_util as P
    L = {"cfg0": lambda: hi.cfg0(n_steps=2),
         "ragged": lambda: _small(C=5003, chunk_size=32, B=3, budget_fraction=0.6, w=32),
         "cs7": lambda: _small(chunk_size=7, C=700, budget_fraction=0.23),
         "many_chunks": lambda: _small(C=2600, chunk_size=1, B=1, budget_fraction=0.3, w=16, head_type=[[1, 0, 1, 1]]),
         "wide_group": lambda: _small(Hq=32, Hkv=2, C=900, chunk_size=16),
         "one_cta_per_unit": lambda: _small(B=50, C=260, chunk_size=16, budget_fraction=0.3, n_steps=1)}[case]()
    rep = P.compare_layer(L)
    assert rep["max_abs"] <= P.MAX_ABS


def test_a_wait_that_cannot_end_gives_up_and_the_device_stays_usable(checked):
    import parity_util as P
    from paper_2604_05887_b200.layer import LayerCache, to_device_bf16
    hkv = checked
    L = hi.cfg0(n_steps=2)
    lc = LayerCache(L, flags=hkv.HKV_OUT_F32)
    q = to_device_bf16(L.q[0])
    before = lc.decode(q).clone()
    torch.cuda.synchronize()
    assert hkv.hkv_last_device_error(lc.handle) == (0, 0)
    # one thread block waits on a barrier nobody arrives on; the call is asynchronous and must come back by itself
    assert hkv.lib.hkv_selftest_wait_timeout(lc.handle, None) == 0
    torch.cuda.synchronize()                       # returns: the wait gave up at its cycle limit
    assert hkv.hkv_last_device_error(lc.handle) == (7, 6)      # HKV_ERR_TIMEOUT, place = the self-test
    # the context is intact: same cache, same query, same bits; the error word is sticky until cleared
    after = lc.decode(q).clone()
    torch.cuda.synchronize()
    assert torch.equal(before, after)
    assert hkv.hkv_last_device_error(lc.handle) == (7, 6)
    assert hkv.lib.hkv_clear_device_error(lc.handle, None) == 0
    assert hkv.hkv_last_device_error(lc.handle) == (0, 0)
    lc.close()
    # and a fresh cache on the same device still matches the oracle
    P.compare_layer(hi.cfg0(n_steps=1))
