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


def test_traffic_entry_is_scaled_to_the_run_and_dropped_when_a_source_changes(tmp_path, monkeypatch):
    src = tmp_path / "k.cu"
    src.write_text("kernel v1")
    prof = tmp_path / "profiles"
    prof.mkdir()
    sha = hashlib.sha256(b"kernel v1").hexdigest()
    table = {"_note": "x",
             "fold_bf16": {"captured_params": 1000, "captured_bytes": 17000, "sources": ["k.cu"], "sha256": sha},
             "wgrad_fold": {"shape": [64, 128, 256], "captured_bytes": 555, "sources": ["k.cu"], "sha256": sha}}
    (prof / "traffic.json").write_text(json.dumps(table))
    monkeypatch.setattr(bench, "ROOT", tmp_path)
    got = bench.load_traffic(5000, 64, 128, 256)
    assert got["fold_bf16"]["bytes_per_launch"] == 85000      # scaled by this run's size
    assert "scaled" in got["fold_bf16"]["note"] and "1000-param" in got["fold_bf16"]["note"]
    same = bench.load_traffic(1000, 64, 128, 256)             # the captured size itself: no scaling
    assert same["fold_bf16"]["bytes_per_launch"] == 17000 and "of this size" in same["fold_bf16"]["note"]
    assert got["wgrad_fold"]["bytes_per_launch"] == 555
    assert "wgrad_fold" not in bench.load_traffic(5000, 64, 128, 512)   # another shape: no figure
    src.write_text("kernel v2")
    assert bench.load_traffic(5000, 64, 128, 256) == {}
    (prof / "traffic.json").write_text("not json")
    assert bench.load_traffic(5000, 64, 128, 256) == {}


def test_one_oracle_sample_serves_both_arms():
    """The cpu_baseline of the default run and the --impl reference arm time the oracle on the
    same bounded sample of the headline step."""
    import inspect
    src = inspect.getsource(bench)
    assert src.count("time_oracle(*ORACLE_SAMPLE") == 2
    assert bench.ORACLE_SAMPLE == (1 << 24, 256, 512, 512)


def test_gpus_flag_without_a_launcher_starts_the_ranks_itself():
    """`python bench.py --gpus 2` with no WORLD_SIZE in the environment re-launches itself as
    two ranks (gloo here, no GPU work) and prints ONE line that says n_gpus: 2."""
    import os
    import subprocess
    import sys
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    res = subprocess.run([sys.executable, str(bench.ROOT / "bench.py"), "--gpus", "2",
                          "--workload", "launch_check", "--backend", "gloo"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["metric"] == "launch_check"
    assert line["ms_per_step"] >= 20.0      # the max over the ranks (rank 1 sleeps 20 ms)


def test_peaks_come_from_the_measured_file_when_present(tmp_path, monkeypatch):
    monkeypatch.setattr(bench, "ROOT", tmp_path)
    assert bench.peaks()["source"] == "fallback"
    (tmp_path / "MEASURED_PEAKS.json").write_text(json.dumps(
        {"hbm_gbs": 6000.0, "bf16_tflops": 1500.0, "bf16_tflops_sustained": 1300.0}))
    pk = bench.peaks()
    assert pk == {"hbm_gbs": 6000.0, "bf16_tflops": 1500.0, "bf16_tflops_sustained": 1300.0,
                  "source": "measured"}
