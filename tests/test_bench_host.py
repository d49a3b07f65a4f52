"""Host-side logic of bench.py: the reference arm's JSON line and the work / launch accounting (no GPU)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2604_08133_b200 import synth  # noqa: E402


def test_reference_arm_prints_one_contract_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == bench.METRIC and d["unit"] == bench.UNIT
    assert d["n_gpus"] == 1 and d["steps"] == 1 and d["higher_is_better"] is True and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": bench.UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["gpu_launches"] == 0 and "c1" in d["config"]["workload"]


def test_launch_count_follows_the_librarys_choices():
    c = synth.CONFIGS
    assert bench.kernels_per_layer(c["c2"], c["c2"].budget) == 5      # gate, routing, 2 GEMMs, combine: no gather
    assert bench.kernels_per_layer(c["d8"], c["d8"].budget) == 5
    assert bench.kernels_per_layer(c["c3"], c["c3"].budget) == 6      # + the row gather above 32 rows per expert
    assert bench.kernels_per_layer(c["c5"], c["c5"].budget) == 6
    big = c["c3"].with_(T=8193)
    assert bench.kernels_per_layer(big, 3 * 8193) == 9                # select + count / scan / place past 8192 tokens


def test_algorithmic_work_matches_the_formulas_by_hand():
    cfg = synth.CONFIGS["c2"]
    touched = 60
    flops, by = bench.algorithmic_work(cfg, cfg.budget, touched)
    H, I, T, N, S, B = cfg.H, cfg.I, cfg.T, cfg.N, cfg.S, cfg.budget
    assert flops == (B + S * T) * 6.0 * H * I + 2.0 * T * H * N
    assert by == (touched + S) * 6.0 * H * I + T * H * 2 + B * H * 2 + 2 * B * H * 2 + T * H * 2 + T * H * 2
    gf, gb = bench.gemm1_work(cfg, cfg.budget, touched)
    assert gf == (B + S * T) * 4.0 * H * I
    assert gb == (touched + S) * 4.0 * H * I + B * H * 2 + T * H * 2 + B * I * 2 + S * T * I * 2
    # the weights dominate at decode: within 1 % of W13 of the touched experts alone
    assert abs(gb / ((touched + S) * 4.0 * H * I) - 1) < 0.01


def test_ncu_traffic_is_quoted_only_for_the_kernel_source_it_was_taken_on(tmp_path, monkeypatch):
    prof = tmp_path / "profiles"
    prof.mkdir()
    sha = bench.kernel_source_sha16()
    (prof / "ncu_traffic.txt").write_text(
        "# comment\n"
        "ffn_gemm_kernel<true, 256>\tc2\t192\t720600000\t%s\tabc1234\tncu\n"
        "ffn_gemm_pair_kernel<true>\tc3\t12288\t886000000\t0000000000000000\tabc1234\tncu\n" % sha)
    real_join = os.path.join
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    # the fingerprint still reads the real sources
    monkeypatch.setattr(bench, "kernel_source_sha16", lambda: sha)
    assert bench.ncu_traffic_bytes("ffn_gemm_kernel<true, 256>", "c2", 192) == 720600000.0
    assert bench.ncu_traffic_bytes("ffn_gemm_kernel<true, 256>", "c2", 384) is None          # another budget
    assert bench.ncu_traffic_bytes("ffn_gemm_pair_kernel<true>", "c3", 12288) is None        # stale fingerprint
    assert real_join is os.path.join


def test_median_and_default_steps():
    assert bench.median([3.0, 1.0, 2.0]) == 2.0 and bench.median([4.0, 1.0, 2.0, 3.0]) == 2.5
    c = synth.CONFIGS
    assert bench.default_steps(c["c2"])[0] >= 200 and bench.default_steps(c["c4"])[0] <= 20
    assert bench.default_steps(c["c5"])[0] < bench.default_steps(c["c3"])[0]
    for name in ("c2", "c3", "c4", "c5"):
        assert bench.default_steps(c[name])[1] >= 3                                          # at least three warm-ups
