"""Host-side pieces of the measurement harness (no GPU)."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def test_recorded_dram_traffic_is_dropped_when_the_kernel_sources_change(tmp_path, monkeypatch):
    import bench
    from paper_2604_19906_b200 import profile_summary
    digest = profile_summary.source_digest()
    assert len(digest) == 16 and digest == profile_summary.source_digest()
    prof = tmp_path / "profiles"
    prof.mkdir()
    (prof / "dram_traffic.json").write_text(json.dumps({
        "cfg3": {"bytes_per_element": 67000.0, "source_digest": digest},
        "cfg4": {"bytes_per_element": 16000.0, "source_digest": "0" * 16}}))
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.ncu_traffic_bytes_per_element(3) == 67000.0     # same sources: kept
    assert bench.ncu_traffic_bytes_per_element(4) is None        # sources changed: null
    assert bench.ncu_traffic_bytes_per_element(5) is None        # never captured


def test_nominal_and_derived_peaks():
    import bench
    assert abs(bench.FP64_PEAK_TFLOPS - 148 * 64 * 2 * 1.965 / 1e3) < 1e-9
    assert bench.NOMINAL_HBM_GBS == 8000.0 and bench.NOMINAL_FP64_TFLOPS >= 37.0
