"""The arithmetic behind the benchmark line's roofline fields, checked by hand-worked numbers (no GPU)."""
import pytest

import bench


def test_algorithmic_bytes_and_flops_of_the_decode_batch():
    n, d, V = 256, 896, 151936
    # W once (2 bytes per weight) + h once + 17 bytes of outputs per row + the count
    assert bench.algorithmic_bytes(n, d, V) == 2 * 151936 * 896 + 2 * 256 * 896 + 17 * 256 + 4 == 272732420
    assert bench.algorithmic_flops(n, d, V) == 2 * 256 * 896 * 151936 == 69700943872
    # an 8-bit head: one byte per weight plus one fp32 scale per vocabulary row
    assert bench.algorithmic_bytes(16, d, V, fp8=True) == 151936 * 896 + 4 * 151936 + 2 * 16 * 896 + 17 * 16 + 4


def test_fractions_follow_from_one_duration_and_the_three_peaks():
    peaks = {"hbm_gbs": 6541.1, "bf16_tflops": 1630.3, "bf16_tflops_sustained": 1385.8}
    f = bench.roofline_fractions(256, 896, 151936, 58.8e-6, peaks)
    # 272 732 420 B / 58.8 us = 4638 GB/s -> 0.709 of 6541.1; 69.70 GFLOP / 58.8 us = 1185 TFLOP/s
    assert f["hbm_frac"] == pytest.approx(0.7091, abs=2e-4)
    assert f["tensor_frac_burst"] == pytest.approx(1185.4 / 1630.3, abs=2e-4)
    assert f["tensor_frac_sustained"] == pytest.approx(1185.4 / 1385.8, abs=2e-4)
    # ridge reading: the longer of t_mem = 41.70 us and t_mma = 42.75 us over the measured time
    assert f["ridge_frac"] == pytest.approx(42.754 / 58.8, abs=2e-4)
    # against the datasheet figures (8 TB/s, 2.25 PFLOP/s dense bf16): 4638 / 8000 and 1185.4 / 2250
    assert f["hbm_frac_of_nominal"] == pytest.approx(0.5798, abs=2e-4)
    assert f["tensor_frac_of_nominal"] == pytest.approx(0.5268, abs=2e-4)
    # a tensor-bound shape: the HBM fraction is tiny and the ridge reading equals the tensor one
    g = bench.roofline_fractions(8192, 896, 151936, 1.7717e-3, peaks)
    assert g["tensor_frac_sustained"] == pytest.approx(0.908, abs=2e-3) and g["hbm_frac"] < 0.03
    assert g["ridge_frac"] == g["tensor_frac_burst"]


def test_fallback_peaks_are_used_only_without_the_measured_file(tmp_path, monkeypatch):
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    peaks, kind = bench.measured_peaks()
    assert kind == "fallback" and peaks["hbm_gbs"] == 6650.0 and peaks["bf16_tflops"] == 1590.0
    (tmp_path / "MEASURED_PEAKS.json").write_text('{"hbm_gbs": 1.0, "bf16_tflops": 2.0}')
    peaks, kind = bench.measured_peaks()
    assert kind == "measured" and peaks["hbm_gbs"] == 1.0
