"""Host logic of bench.py that needs no GPU: the recorded ncu traffic is only reported for the
exact kernel sources it was captured on."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_traffic_is_null_when_the_kernels_changed(monkeypatch):
    big = [(1024, 8192, 28672), (8192, 8192, 28672), (32768, 8192, 28672)]
    captured = bench.NCU_TRAFFIC["cfg5"]
    monkeypatch.setattr(bench, "kernel_sources_digest", lambda files=None: captured["digest"])
    assert captured["per_row_of"] == (8192, 8192, 28672)
    # the captured shape itself, and the record over all tensor-bound shapes: scaled by the rows processed
    assert bench.ncu_traffic("cfg5", [(8192, 8192, 28672)]) == float(captured["bytes"])
    assert bench.ncu_traffic("cfg5", big) == float(captured["bytes"]) * (1024 + 8192 + 32768) / 8192
    assert bench.ncu_traffic("cfg5", [(8192, 4096, 28672)]) is None          # another weight matrix: no figure
    assert bench.ncu_traffic("cfg3", [(4096, 4096, 14336)]) == float(bench.NCU_TRAFFIC["cfg3"]["shapes"][(4096, 4096, 14336)])
    assert bench.ncu_traffic("cfg3", [(4096, 4096, 4096)]) is None
    assert bench.ncu_traffic("cfg2", [(2048, 2048, 2048)]) is None
    monkeypatch.setattr(bench, "kernel_sources_digest", lambda files=None: "something else")
    assert bench.ncu_traffic("cfg5", big) is None


def test_kernel_label_follows_the_dispatch_rule():
    assert bench.gemm_kernel_name(128, 8192, 28672) == "gemm_mxfp4_kernel"           # one tile row
    assert bench.gemm_kernel_name(1024, 8192, 28672) == "gemm_mxfp4_pair_kernel"
    assert bench.gemm_kernel_name(2048, 2048, 8192) == "gemm_mxfp4_kernel"           # K < 4096
    assert bench.gemm_kernel_name(4096, 4096, 1024) == "gemm_mxfp4_kernel"           # fewer than two rounds of pairs


def test_digest_covers_the_kernel_sources():
    d = bench.kernel_sources_digest()
    assert len(d) == 64 and d == bench.kernel_sources_digest()
    g = bench.kernel_sources_digest(bench.GEMM_SOURCES)
    assert g != d and g != bench.kernel_sources_digest(bench.RQ_SOURCES)
