"""Host-side logic of bench.py that needs no GPU: how many timed blocks a run takes, and when the DRAM
traffic figure of an ncu capture may be quoted."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench


def test_blocks_cover_the_requested_time_within_the_cap():
    assert bench.blocks_for(0.083, 20, 1000.0, 40000) == 603          # 1 s of 83 us calls in blocks of 20
    assert bench.blocks_for(0.083, 2000, 1000.0, 40000) == 7
    assert bench.blocks_for(5.0, 20, 1000.0, 40000) == 10
    assert bench.blocks_for(0.001, 20, 1000.0, 40000) == 2000         # capped by the number of calls
    assert bench.blocks_for(100.0, 20, 1.0, 40000) == 1               # never fewer than one block


def test_traffic_is_quoted_only_for_the_sources_the_capture_was_taken_from(tmp_path, monkeypatch):
    value, src = bench.ncu_traffic("verify_attn", "c4")
    assert value is None and "no ncu capture" in src
    value, src = bench.ncu_traffic("verify_attn", "c3")
    text = open(os.path.join(ROOT, "profiles", bench.TRAFFIC_PROFILES[("verify_attn", "c3")])).read()
    recorded = [l.split(":")[1].strip() for l in text.splitlines() if l.startswith("source-sha256-16:")][0]
    if recorded == bench.source_digest("verify_attn"):
        assert value and value > 3.0e8 and "not this run" in src
    else:
        assert value is None and "changed since the capture" in src
    # a digest that cannot match: the figure is withheld
    monkeypatch.setattr(bench, "source_digest", lambda kind: "0" * 16)
    value, src = bench.ncu_traffic("verify_attn", "c3")
    assert value is None and "changed since the capture" in src


def test_median_and_l2_rule():
    assert bench.median([3.0, 1.0, 2.0]) == 2.0

    class W:
        def __init__(self, b):
            self.b = b

        def attn_algorithmic_bytes(self):
            return self.b
    assert bench.fits_l2(W(18e6)) and bench.fits_l2(W(226e6)) and not bench.fits_l2(W(328e6))
