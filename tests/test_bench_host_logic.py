"""Host-side logic of bench.py that needs no GPU: the table of profiler counters and its staleness rule, the
algorithmic-byte model, the binding report's arithmetic and the slope fit."""
import os

import numpy as np

import bench
from workloads import configs


def test_counters_table_parses_and_goes_stale_when_a_source_changes(tmp_path, monkeypatch):
    good = bench.source_hash(["sample.cu"])
    table = tmp_path / "ncu_counters.md"
    table.write_text(
        "# title\n\n| class | sources | source hash | workload | heads captured | dram bytes per launch at capture | issue % | tensor % | lsu % |\n"
        "|---|---|---|---|---|---|---|---|---|\n"
        f"| walk_merge | sample.cu | {good} | pointcloud-gmm16-N32768 | 2 | 11420736 | 71.6 | 0.0 | 63.9 |\n"
        "| gather_contract | attn_gather_tc.cu tc_common.cuh | 0000000000000000 | pointcloud-gmm16-N32768 | 2 | 1147654784 | 44.0 | 47.1 | 5.8 |\n")
    monkeypatch.setattr(bench, "COUNTERS_FILE", str(table))
    c = bench.load_counters()
    assert set(c) == {"walk_merge", "gather_contract"}
    assert c["walk_merge"]["stale"] is False and c["walk_merge"]["dram_bytes"] == 11420736 and c["walk_merge"]["heads"] == 2
    assert c["gather_contract"]["stale"] is True          # the recorded hash is not that of the sources
    assert c["gather_contract"]["sources"] == ["attn_gather_tc.cu", "tc_common.cuh"]


def test_tracked_counters_table_is_readable():
    c = bench.load_counters()
    assert {"gather_contract", "build_states", "walk_merge"} <= set(c)
    for row in c.values():
        assert all(os.path.exists(os.path.join(bench.CSRC, f)) for f in row["sources"])


def test_algorithmic_bytes_of_the_bench_workload():
    w = configs.point_cloud_32768()
    N, nnz = 32768, 3_130_000
    a = bench.algorithmic_bytes(w, N, nnz, nnz, 399038)
    S = w.G * N * w.m * w.d * 2
    assert S == 1_073_741_824
    # gather: S, z (fp32), phi(Q), Phi, out -- each once
    assert a["gather_contract"] == S + w.G * N * w.m * 4 + w.G * N * w.m * 2 + nnz * 8 + (N + 1) * 4 + w.G * N * w.d * 2
    # per token-head: about 4.5 KB, the figure the roofline line quotes
    assert 4400 < a["gather_contract"] / (w.G * N) < 4600
    assert a["build_states"] > S and a["walk_merge"] < 0.2e9


def test_binding_report_arithmetic():
    w = configs.point_cloud_32768()
    pk = {"hbm_gbs": 6500.0, "bf16_tflops": 1600.0}
    ktimes = {"gather_contract": (1.0 * 4, 4), "build_states": (0.5 * 4, 4), "walk_merge": (0.25 * 4, 4)}   # ms, launches
    rep = bench.binding_report(w, 32768, 3_000_000, 3_000_000, ktimes, 4, pk, {}, plan_entries=350_000, mask_entries=None)
    g = rep["gather_contract"]
    assert np.isclose(g["tensor_issued_tflops"], 350_000 * 8 * 2 * 128 * 32 * 64 / 1e-3 / 1e12)
    assert np.isclose(g["tensor_useful_tflops"], 2 * 3_000_000 * 32 * 64 * 8 / 1e-3 / 1e12)
    assert np.isclose(g["smem_fill_gbs"], 350_000 * 8 * 32 * 64 * 2 / 1e-3 / 1e9)
    assert g["binds"] in ("smem_fill", "tensor_issue") and 0 < g["fraction_of_binding_peak"] < 3
    assert rep["walk_merge"]["binds"] == "hbm"            # no profiler row given: only the HBM fraction is known
    assert np.isclose(rep["walk_merge"]["walks_per_s"], 2 * 32768 * 32 / 0.25e-3)


def test_loglog_slope():
    xs = [2 ** k for k in range(14, 21)]
    assert np.isclose(bench.loglog_slope(xs, [3e-6 * x for x in xs]), 1.0)
    assert np.isclose(bench.loglog_slope(xs, [1e-9 * x * x for x in xs]), 2.0)
