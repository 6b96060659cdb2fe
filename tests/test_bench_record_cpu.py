"""The parts of bench.py that shape the record, on CPU: the per-config roofline lines and the bounded
oracle samples (shapes, scale factors, core counts) that go into the one JSON line."""
import os

import pytest

import bench


def test_roofline_configs_projection():
    per = [{"transform": "P(sum)->B", "bytes": 1000, "ms": 0.5, "gbs": 2.0, "frac_measured": 0.25,
            "ms_back_to_back": 0.4, "frac_measured_back_to_back": 0.3}]
    ops = [{"op": "MLP GEMM1 (B,S(1))->S(1) + GeLU", "config": 3, "kernel": "matmul_tc_kernel", "bound": "tensor",
            "flops": 2e12, "ms": 1.0, "achieved": 2000.0, "unit": "TFLOP/s", "frac_measured": 0.8, "traffic": None},
           {"op": "embedding fused gather -> B (replicas aliased, 1 write)", "config": 5, "kernel": "embedding_kernel<fused>",
            "bound": "hbm", "bytes": 10, "ms": 2.0, "achieved": 5.0, "unit": "GB/s", "frac_measured": 0.1,
            "traffic": 8.0, "achieved_dram": 4.0, "frac_dram": 0.05},
           {"op": "beyond the configs", "config": None, "bound": "hbm", "ms": 1.0, "achieved": 1.0, "unit": "GB/s",
            "frac_measured": 0.1},
           {"op": "section_x", "error": "refused"}]
    cfgs = bench.roofline_configs(per, ops)
    assert [c["config"] for c in cfgs] == [2, 3, 5]
    assert cfgs[0]["line"] == "P(sum)->B" and cfgs[0]["work"] == 1000 and cfgs[0]["frac"] == 0.25
    assert cfgs[0]["traffic"] == bench.ncu_traffic("P(sum)->B")
    assert cfgs[0]["achieved_dram"] == pytest.approx(cfgs[0]["traffic"] / 0.5e-3 / 1e9)
    assert cfgs[1]["work"] == 2e12 and cfgs[1]["frac"] == 0.8 and "frac_dram" not in cfgs[1]
    assert cfgs[2]["frac_dram"] == 0.05 and cfgs[2]["achieved_dram"] == 4.0
    for c in cfgs:                     # a frac can be recomputed from ms and work
        assert {"kernel", "bound", "ms", "work", "achieved", "unit", "frac"} <= set(c)


def test_every_traffic_constant_names_a_bench_line():
    src = open(bench.__file__).read()
    for name in bench.NCU_TRAFFIC:
        assert src.count('"' + name + '"') >= 1 or name in [t[0] for t in bench.TRANSFORMS], name
    for t in bench.TRANSFORMS:
        assert bench.ncu_traffic(t[0]) is not None
    assert len(bench.NCU_TRAFFIC_CAPTURED_AT) >= 7


def test_host_cores_and_blas_threads_are_positive():
    assert 1 <= bench.host_cores() <= (os.cpu_count() or 1)
    assert bench.blas_threads() >= 1


def test_oracle_config_samples_cover_configs_3_4_5():
    """The bounded oracle samples as the benchmark runs them (inputs drawn on the CPU here)."""
    out = bench.oracle_config_samples("cpu")
    assert sorted({e["config"] for e in out}) == [3, 4, 5]
    assert len(out) == 4
    for e in out:
        assert e["seconds"] > 0 and e["value"] > 0 and e["scale"] >= 1
        assert e["cores"] >= e["threads_used"] >= 1
        assert e["full_s_extrapolated"] == pytest.approx(e["seconds"] * e["scale"])
        assert e["unit"] in ("GB/s", "GFLOP/s") and e["sample"]
