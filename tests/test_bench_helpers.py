"""Host logic of bench.py that needs no GPU: the recorded ncu traffic is only reported for the
exact kernel sources it was captured on."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_traffic_is_null_when_the_kernels_changed(monkeypatch):
    shapes = [(2048, 2048, 2048), (2048, 2048, 8192), (2048, 8192, 2048)]
    monkeypatch.setattr(bench, "kernel_sources_digest", lambda: bench.NCU_TRAFFIC["sources"])
    assert bench.ncu_traffic("cfg2", shapes) == float(sum(bench.NCU_TRAFFIC["cfg2"].values()))
    assert bench.ncu_traffic("cfg3", [(4096, 4096, 4096)]) is None
    monkeypatch.setattr(bench, "kernel_sources_digest", lambda: "something else")
    assert bench.ncu_traffic("cfg2", shapes) is None


def test_digest_covers_the_kernel_sources():
    d = bench.kernel_sources_digest()
    assert len(d) == 64 and d == bench.kernel_sources_digest()
