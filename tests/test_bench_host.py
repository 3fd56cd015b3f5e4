"""Host logic of bench.py: how profile records become the per-kernel table, which roofline a kernel is
held against, and when a stored DRAM-traffic figure may be reported."""
import json

import bench

PEAKS = dict(hbm=6500.0, tc_sustained=1400.0, source="test")


def rec(launches, ms, bytes_, flops):
    return dict(launches=launches, ms=ms, bytes=bytes_, flops=flops)


def test_records_are_merged_per_device_kernel():
    prof = {"conv_fprop_tc|1000|2000": rec(2, 1.0, 2000.0, 4000.0), "conv_dgrad_tc|500|100": rec(1, 0.5, 500.0, 100.0),
            "conv_fprop_tc2|9|9": rec(3, 3.0, 27.0, 27.0), "conv_wgrad_tc2|1|1": rec(1, 1.0, 1.0, 1.0), "sgd|7|0": rec(1, 0.25, 7.0, 0.0)}
    out = bench.by_device_kernel(prof)
    assert set(out) == {"conv_tc_kernel", "conv_tc2_kernel", "wgrad_tc2_kernel", "sgd"}
    assert out["conv_tc_kernel"] == rec(3, 1.5, 2500.0, 4100.0)
    assert sum(v["launches"] for v in out.values()) == sum(v["launches"] for v in prof.values())


def test_convolution_launch_shapes_are_split_by_what_binds_them():
    # 1 GB and 1 GFLOP per launch: memory needs 154 us, the tensor cores 0.7 us -> hbm; 1 MB and 1 TFLOP -> tensor
    prof = {"conv_fprop_tc|1e9|1e9": rec(1, 0.2, 1e9, 1e9), "conv_fprop_tc|1e6|1e12": rec(1, 1.0, 1e6, 1e12), "bn_relu_apply|5|0": rec(1, 0.1, 5.0, 0.0)}
    out = bench.by_device_kernel(prof, PEAKS)
    assert out["conv_tc_kernel [hbm-bound layers]"]["ms"] == 0.2 and out["conv_tc_kernel [tensor-bound layers]"]["ms"] == 1.0
    assert "bn_relu_apply" in out                      # kernels that are not convolutions keep their name


def test_roofline_that_binds_a_kernel():
    assert bench.binding_roofline("conv_tc_kernel", rec(1, 1.0, 1e9, 1e9), PEAKS) == "hbm"
    assert bench.binding_roofline("conv_tc_kernel", rec(1, 1.0, 1e6, 1e12), PEAKS) == "tensor"
    assert bench.binding_roofline("gemm_simt_kernel", rec(1, 1.0, 1e6, 1e12), PEAKS) == "alu"


def test_stored_traffic_is_reported_only_for_unchanged_kernel_sources(tmp_path, monkeypatch):
    prof_dir = tmp_path / "profiles"
    prof_dir.mkdir()
    (prof_dir / "dram_traffic.txt").write_text(json.dumps({"w": {"conv_tc_kernel": dict(dram_bytes_per_launch=123, source_digest="abc")}}))
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    monkeypatch.setattr(bench, "source_digest", lambda k: "abc")
    assert bench.measured_traffic("conv_tc_kernel", "w") == 123
    assert bench.measured_traffic("conv_tc_kernel", "other workload") is None
    assert bench.measured_traffic("wgrad_tc_kernel", "w") is None
    monkeypatch.setattr(bench, "source_digest", lambda k: "changed")
    assert bench.measured_traffic("conv_tc_kernel", "w") is None


def test_committed_traffic_file_names_kernels_the_bench_knows():
    d = json.load(open(bench.os.path.join(bench.ROOT, "profiles", "dram_traffic.txt")))
    for workload, kernels in d.items():
        for k, v in kernels.items():
            assert k in bench.KERNEL_SOURCES, (workload, k)
            assert v["dram_bytes_per_launch"] > 0 and len(v["source_digest"]) == 16
