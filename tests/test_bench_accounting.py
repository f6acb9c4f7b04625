"""The benchmark's byte accounting (no GPU): algorithmic bytes per node-parameter of every recipe and the traffic
figure scaled from the small-case captures, which must never fall below the algorithmic bytes."""
import sys

import pytest

from conftest import ROOT

sys.path.insert(0, ROOT)


@pytest.fixture(scope="module")
def bench():
    import bench as b
    return b


@pytest.fixture(scope="module")
def workloads():
    from paper_1811_10792_b200 import inputs
    return inputs.WORKLOADS


@pytest.mark.parametrize("name,read,write", [("resnet50", 12, 12), ("transformer", 8, 8), ("resnet50_osgp1", 16, 16),
                                            ("transformer_adam", 16, 16)])
def test_algorithmic_bytes_per_update(bench, workloads, name, read, write):
    """x, g (+ u, + both Adam moments, + one ring slot) read; x, z (+ the same extras) written: fp32, in place."""
    w = workloads[name]
    assert bench.read_write_bytes_per_update(w) == (read, write)
    assert bench.bytes_per_update(w) == read + write
    assert bench.read_write_bytes_per_update(w, write_z=False) == (read, write - 4)


@pytest.mark.parametrize("name", ["resnet50", "transformer", "resnet50_osgp1", "transformer_adam"])
def test_scaled_traffic_is_never_below_the_algorithmic_bytes(bench, workloads, name):
    w = workloads[name]
    traffic, detail = bench.scaled_traffic(w)
    algorithmic = bench.bytes_per_update(w) * w.n * w.d
    assert traffic >= algorithmic and traffic <= 1.03 * algorithmic           # the contract's "at most 1.03 x"
    assert detail["l2_dirty_tail_bytes"] >= 0
    assert abs(detail["dram_read_bytes"] + detail["dram_write_bytes_in_kernel"] + detail["l2_dirty_tail_bytes"] - traffic) < 1.0


def test_roofline_fraction_arithmetic(bench, workloads):
    w = workloads["resnet50"]
    r = bench.roofline_of(w, 3.0, 6559.7, "measured")
    assert r["algorithmic_bytes_per_launch"] == 24 * 32 * 25_557_032
    assert abs(r["achieved"] - 24 * 32 * 25_557_032 / 3.0e-3 / 1e9) < 1e-6
    assert abs(r["frac"] - r["achieved"] / 6559.7) < 1e-12 and r["bound"] == "hbm" and r["peak_kind"] == "of measured"
