"""Host-side arithmetic of bench.py: algorithmic work per kernel, the DRAM-traffic lookup and its scaling rule."""
import os

import numpy as np

import bench
from paper_2603_06626_b200 import synth


def test_algorithmic_flops_add_up_to_18_d_F_per_routed_row():
    w = synth.WORKLOADS["large"]
    counts = np.full(w.E_tgt, w.R // w.E_tgt, dtype=np.int64)
    work = bench.kernel_work(w, counts, 16384)
    flops = sum(v for kind, v in work.values() if kind == "flop")
    assert flops == 18.0 * w.d * w.ffn * w.R
    movers = [work[k][1] for k in bench.MOVER_SLOTS]
    assert all(m == (w.T + w.R) * w.d * 2.0 for m in movers)
    assert set(bench.GEMM_SLOTS) | set(bench.MOVER_SLOTS) <= set(work)


def test_algorithmic_dram_bytes_of_the_products():
    w = synth.WORKLOADS["skewed"]
    R, d, F, E = w.R, w.d, w.ffn, w.E_tgt
    up = bench.algorithmic_dram_bytes(w, "gemm_up_swiglu")
    assert up == R * d * 2 + E * 2 * F * d * 2 + 3 * R * F * 2          # Xp and W_gu read; G, U, H' written
    wg = bench.algorithmic_dram_bytes(w, "wgrad_gate_up")
    assert wg == 2 * R * F * 2 + R * d * 2 + E * 2 * F * d * 4          # [dG|dU] and Xp read; fp32 dW_gu written
    assert bench.algorithmic_dram_bytes(w, "plan_hist") == 0.0


def test_traffic_lookup_scales_a_small_capture_and_forgets_old_builds(tmp_path, monkeypatch):
    tag = bench.kernel_source_tag()
    f = tmp_path / "dram_traffic.txt"
    f.write_text(f"# comment\nskewed gemm_down 1300000000 {tag}   # trailing words\nskewed gemm_dX 2000000000 000000000000\n")
    monkeypatch.setattr(bench, "TRAFFIC_FILE", str(f))
    sk, lg = synth.WORKLOADS["skewed"], synth.WORKLOADS["large"]
    assert bench.recorded_traffic(sk, "gemm_down") == 1.3e9                                  # the captured workload itself
    want = 1.3e9 * bench.algorithmic_dram_bytes(lg, "gemm_down") / bench.algorithmic_dram_bytes(sk, "gemm_down")
    assert abs(bench.recorded_traffic(lg, "gemm_down") - want) < 1.0                          # scaled by algorithmic bytes
    assert bench.recorded_traffic(lg, "gemm_dX") is None                                      # taken with other sources
    assert bench.recorded_traffic(lg, "gemm_up_swiglu") is None                               # no line at all
    monkeypatch.setattr(bench, "TRAFFIC_FILE", str(tmp_path / "absent.txt"))
    assert bench.recorded_traffic(lg, "gemm_down") is None


def test_committed_traffic_file_is_well_formed():
    path = os.path.join(bench.ROOT, "profiles", "dram_traffic.txt")
    lines = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert lines and all(len(p) >= 4 and p[0] in synth.WORKLOADS and float(p[2]) >= 0 and len(p[3]) == 12 for p in lines)
    assert {p[1] for p in lines} >= set(bench.GEMM_SLOTS) | set(bench.MOVER_SLOTS)
