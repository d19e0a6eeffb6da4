"""Host logic of bench.py that needs no GPU: the recorded DRAM traffic is reported only while the
product kernels' sources still have the digest stored beside it."""
import hashlib
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


def _digest(root, names):
    h = hashlib.sha256()
    for name in names:
        h.update(name.encode())
        h.update(open(os.path.join(root, "paper_2106_08301_b200", "csrc", name), "rb").read())
    return h.hexdigest()[:16]


def test_recorded_traffic_follows_the_source_digest(tmp_path, monkeypatch):
    csrc = tmp_path / "paper_2106_08301_b200" / "csrc"
    csrc.mkdir(parents=True)
    (csrc / "a.cu").write_text("kernel one\n")
    (csrc / "b.cuh").write_text("header\n")
    prof = tmp_path / "profiles"
    prof.mkdir()
    good = _digest(str(tmp_path), ["a.cu", "b.cuh"])
    (prof / "dram_traffic.txt").write_text(
        "| workload | kernels | bytes | digest | sources |\n|---|---|---|---|---|\n"
        f"| w1 | k | 12345 | {good} | a.cu b.cuh |\n"
        f"| w2 | k | 777 | {'0' * 16} | a.cu |\n"
        f"| w3 | k | 5 | {good} | a.cu missing.cu |\n")
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.recorded_traffic("w1") == 12345
    assert bench.recorded_traffic("w2") is None          # digest of other sources
    assert bench.recorded_traffic("w3") is None          # a named source is gone
    assert bench.recorded_traffic("absent") is None
    (csrc / "a.cu").write_text("kernel one, changed\n")
    assert bench.recorded_traffic("w1") is None          # the kernel changed after the capture


def test_committed_traffic_table_is_well_formed():
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    rows = [[c.strip() for c in ln.strip().strip("|").split("|")] for ln in open(path) if ln.startswith("| c")]
    assert rows, "no workload rows"
    for r in rows:
        assert len(r) == 5 and r[2].isdigit() and len(r[3]) == 16
        for name in r[4].split():
            assert os.path.exists(os.path.join(ROOT, "paper_2106_08301_b200", "csrc", name))
