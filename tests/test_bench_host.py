"""Host-side logic of bench.py that needs no GPU: the algorithmic byte and flop counts the
reported throughput is built on, and the staleness rule of the DRAM-traffic table."""
import hashlib
import json

import adama_workloads as wl
import bench


def test_headline_step_byte_and_flop_counts():
    """18 B/param per bf16 fold (2 read g + 8 read + 8 write m, v), 24 B/param per apply, and for
    the fused call 16 B/param of m, v plus the bf16 inputs; 2*T flops per parameter."""
    n, NA, NB = wl.CONFIG2_FULL_N, wl.CONFIG2.n_micro, wl.CONFIG3.n_micro
    T, d_in, d_out = wl.CONFIG3.tokens, wl.CONFIG3.d_in, wl.CONFIG3.d_out
    flat, lin, flops, lin_call = bench.step_bytes_and_flops(n, NA, T, d_in, d_out, NB)
    assert flat == n * (18 * 8 + 24) == 56_280_000_000
    assert lin_call == 16 * 4096 * 4096 + 2 * 4096 * (4096 + 4096) == 335_544_320
    assert lin == 4 * lin_call + 24 * 4096 * 4096
    assert flops == 4 * 2.0 * 4096 ** 3


def test_traffic_entry_is_dropped_when_a_source_changes(tmp_path, monkeypatch):
    src = tmp_path / "k.cu"
    src.write_text("kernel v1")
    prof = tmp_path / "profiles"
    prof.mkdir()
    entry = {"bytes_per_launch": 123, "sources": ["k.cu"],
             "sha256": hashlib.sha256(b"kernel v1").hexdigest()}
    (prof / "traffic.json").write_text(json.dumps({"_note": "x", "fold_bf16": entry}))
    monkeypatch.setattr(bench, "ROOT", tmp_path)
    assert bench.load_traffic() == {"fold_bf16": 123}
    src.write_text("kernel v2")
    assert bench.load_traffic() == {}
    (prof / "traffic.json").write_text("not json")
    assert bench.load_traffic() == {}


def test_peaks_come_from_the_measured_file_when_present(tmp_path, monkeypatch):
    monkeypatch.setattr(bench, "ROOT", tmp_path)
    assert bench.peaks()["source"] == "fallback"
    (tmp_path / "MEASURED_PEAKS.json").write_text(json.dumps(
        {"hbm_gbs": 6000.0, "bf16_tflops": 1500.0, "bf16_tflops_sustained": 1300.0}))
    pk = bench.peaks()
    assert pk == {"hbm_gbs": 6000.0, "bf16_tflops": 1500.0, "bf16_tflops_sustained": 1300.0,
                  "source": "measured"}
