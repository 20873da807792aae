"""profiles/ncu_traffic.json feeds bench.py's `roofline.traffic`: an entry counts only while the
kernel sources still hash to what they were when ncu counted the bytes."""
import json
import os

from paper_2506_14435_b200 import traffic

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_entries_are_well_formed_and_point_at_committed_summaries():
    entries = json.load(open(os.path.join(ROOT, "profiles", "ncu_traffic.json")))["entries"]
    assert entries
    for e in entries:
        assert e["impl"] in ("tensor", "stream") and e["dram_bytes_per_launch"] > 0
        assert os.path.exists(os.path.join(ROOT, e["summary"])), e["summary"]
        assert len(e["digest"]) == 16


def test_lookup_needs_a_matching_digest(tmp_path, monkeypatch):
    reg = tmp_path / "t.json"
    monkeypatch.setattr(traffic, "_JSON", str(reg))
    traffic.add("w", "stage", "tensor", 123.0, "profiles/x.md")
    assert traffic.lookup("w", "stage", "tensor") == 123.0
    assert traffic.lookup("w", "stage", "stream") is None and traffic.lookup("w", "other", "tensor") is None
    data = json.load(open(reg))
    data["entries"][0]["digest"] = "0" * 16                 # the kernel has changed since the capture
    json.dump(data, open(reg, "w"))
    assert traffic.lookup("w", "stage", "tensor") is None
