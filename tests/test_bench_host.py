"""CPU-side checks of bench.py's bookkeeping: the roofline arithmetic, and that the ncu counter tables
it carries were captured on the kernel sources as they stand (otherwise the line reports no traffic)."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_counter_tables_belong_to_the_current_kernel_sources():
    assert bench.kernel_source_hash() == bench.NCU_HASH, "re-capture the ncu counters (profiles/) and refresh bench.NCU_*"
    for (tag, kernel), (bytes_per_element, inst, captured_on) in bench.NCU_COUNTERS.items():
        assert captured_on and (bytes_per_element is None or 2.0 < bytes_per_element < 13.0), (tag, kernel)
        assert inst is None or 0.5 < inst < 4.0, (tag, kernel)
    for cfg in ("cfg2_M8_resnet18", "cfg3_M16_vgg19scale", "cfg4_M64_resnet18"):
        assert (cfg, "round_kernel") in bench.NCU_COUNTERS


def test_source_hash_sees_code_and_not_comments(tmp_path):
    a, b, c = tmp_path / "a.cuh", tmp_path / "b.cuh", tmp_path / "c.cuh"
    a.write_text("// header\nint f(int x) {  // doubles\n  return 2 * x;\n}\n")
    b.write_text("// another header\n\nint f(int x) {\n  return 2 * x;  // twice x\n}\n")
    c.write_text("int f(int x) {\n  return 3 * x;\n}\n")
    assert bench.hash_sources([a]) == bench.hash_sources([b]) != bench.hash_sources([c])
    assert bench.hash_sources([a, c]) != bench.hash_sources([c, a])


def test_hbm_roofline_counts_the_bytes_that_must_cross_the_pins():
    elements, ms = 89_391_696, 0.19
    r = bench.hbm_roofline("cfg2_M8_resnet18", "round_kernel", ms, elements, 16, 6537.0, "measured")
    assert r["bound"] == "hbm" and r["unit"] == "GB/s"
    assert r["achieved"] == pytest.approx(12 * elements / (ms / 1e3) / 1e9)
    assert r["frac"] == pytest.approx(r["achieved"] / 6537.0) and r["frac"] < 1.0
    assert r["replica_GBs"] == pytest.approx(16 * elements / (ms / 1e3) / 1e9)
    assert r["traffic"] == pytest.approx(1_041_843_000)
    assert r["dram_GBs"] == pytest.approx(r["traffic"] / (ms / 1e3) / 1e9)
    assert r["dram_frac_of_8TBs"] == pytest.approx(r["dram_GBs"] / 8000.0)
    unknown = bench.hbm_roofline("some other workload", "round_kernel", ms, elements, 16, 6537.0, "measured")
    assert unknown["traffic"] is None and "dram_GBs" not in unknown


def test_issue_roofline_counts_warp_instructions():
    elements, ms = 89_391_696, 0.1134
    r = bench.issue_roofline("cfg2_M8_resnet18", "fused_rounds_kernel", ms, elements, 16, 4.0, 1965, 6537.0, "measured")
    assert r["bound"] == "alu" and r["peak"] == pytest.approx(148 * 4 * 1.965)
    ipe = bench.NCU_COUNTERS[("cfg2_M8_resnet18", "fused_rounds_kernel")][1]
    assert r["achieved"] == pytest.approx(ipe * elements / (ms / 1e3) / 1e9)
    assert 0.4 < r["frac"] < 0.8
    assert r["dram_GBs"] == pytest.approx(r["traffic"] / (4 * ms / 1e3) / 1e9)      # a launch covers four rounds
    assert r["pipes_busy"]["fmaheavy"] > r["pipes_busy"]["issue"]


def test_shard_plan_offsets_are_counter_aligned():
    for world in (1, 2, 4, 8):
        plans = [bench.shard_plan(11_173_962, world, rank) for rank in range(world)]
        assert all(p["element_offset"] % 4 == 0 for p in plans)
        assert [p["element_offset"] for p in plans] == [rank * 11_173_964 for rank in range(world)]
        assert plans[0]["global_d"] == world * 11_173_964
    assert bench.shard_plan(10, 2, 1, align=8)["element_offset"] == 16
