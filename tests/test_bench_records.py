"""bench.py reads the dense chain's DRAM traffic from the tracked profile summary and drops it when
the kernel sources have changed since the counters were taken (no GPU needed)."""
import importlib
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_traffic_record_follows_the_kernel_sources(monkeypatch):
    bench = importlib.import_module("bench")
    path = os.path.join(ROOT, "profiles", "dense_chain_llada8b_b1.md")
    m = re.search(r"bench-traffic:\s*workload=(\S+)\s+dram_bytes_per_launch=([0-9.eE+]+)\s+kernel_sha256=([0-9a-f]+)",
                  open(path).read())
    assert m and m.group(1) == "llada8b_b1"
    got = bench._traffic_record("llada8b_b1")
    if m.group(3) == bench._kernel_hash():
        # per launch: weights of one layer (436 MB) plus what the phases spill, well under 1.2 x
        assert got == float(m.group(2)) and 436e6 < got < 1.2 * 436.3e6
    else:
        assert got is None
    # a changed kernel, or a workload without a summary: no figure rather than a stale one
    monkeypatch.setattr(bench, "_kernel_hash", lambda: "0" * 16)
    assert bench._traffic_record("llada8b_b1") is None
    assert bench._traffic_record("dream7b_b4") is None
