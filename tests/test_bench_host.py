"""Host-side pieces of bench.py that need no GPU: the kernel revision the profiler counters are keyed by, the lookup
of those counters, the statistics of a list of step times and the algorithmic byte count of a layer."""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
import hkv_inputs as hi  # noqa: E402


def test_kernel_revision_ignores_comments_and_spacing(tmp_path, monkeypatch):
    src = os.path.join(ROOT, "paper_2604_05887_b200", "csrc")
    fake = tmp_path / "paper_2604_05887_b200" / "csrc"
    fake.mkdir(parents=True)
    for f in ("hkv_decode.cu", "hkv_device.cuh", "hkv_internal.h"):
        (fake / f).write_text(open(os.path.join(src, f)).read())
    rev = bench.kernel_revision()
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.kernel_revision() == rev
    p = fake / "hkv_decode.cu"
    p.write_text("// a new comment\n\n" + p.read_text().replace("\n", "\n   ", 3) + "/* and a block\n comment */\n")
    assert bench.kernel_revision() == rev                       # comments and blank space do not count
    p.write_text(p.read_text() + "\nint one_more_symbol;\n")
    assert bench.kernel_revision() != rev                       # code does


def test_traffic_lookup_is_keyed_by_workload_and_revision(tmp_path, monkeypatch):
    (tmp_path / "profiles").mkdir()
    (tmp_path / "profiles" / "decode_kernel_traffic.txt").write_text(
        "# comment\ncfg2 aaaaaaaaaaaa 111\ncfg2 bbbbbbbbbbbb 222\ncfg4 bbbbbbbbbbbb 333\n")
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    monkeypatch.setattr(bench, "kernel_revision", lambda: "bbbbbbbbbbbb")
    assert bench.ncu_traffic("cfg2") == 222.0 and bench.ncu_traffic("cfg4") == 333.0
    assert bench.ncu_traffic("cfg3") is None
    monkeypatch.setattr(bench, "kernel_revision", lambda: "cccccccccccc")
    assert bench.ncu_traffic("cfg2") is None                    # counters of an older kernel are not quoted


def test_committed_traffic_table_parses():
    path = os.path.join(ROOT, "profiles", "decode_kernel_traffic.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert rows and all(len(r) == 3 and len(r[1]) == 12 and float(r[2]) > 0 for r in rows)


def test_spread():
    s = bench.spread([3.0, 1.0, 2.0, 10.0])
    assert s == {"median": 2.5, "min": 1.0, "mean": 4.0, "replays": 4}


def test_layer_algo_bytes_matches_the_definition():
    """512 B per retained token of a static head; 512 B per token of the selected chunks + 256 B per chunk mean."""
    L = hi.tiny(seed=3, B=2, C=100, chunk_size=8, w=4, Hq=4, Hkv=2, d=16, budget_fraction=0.25, ragged=False,
                head_type=[[0, 1], [1, 0]])
    bud = int(L.budgets[0, 0])
    nch, k = 13, -(-bud // 8)
    per_dyn = 512 * min(k * 8, 100) + 256 * nch
    assert bench.layer_algo_bytes(L) == 2 * (512 * bud) + 2 * per_dyn
