"""Host-side logic of bench.py that needs no GPU: the DRAM-traffic figure of the roofline object is taken from
an ncu summary only while the kernel sources still are the ones that capture ran."""
import importlib.util
import os

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_traffic_is_dropped_when_the_summary_is_stale_or_missing(tmp_path, monkeypatch):
    bench = _bench()
    digest = bench.kernel_source_digest()
    assert len(digest) == 16 and int(digest, 16) >= 0
    prof = tmp_path / "profiles"
    prof.mkdir()
    (prof / "fresh.md").write_text("notes\ntraffic_bytes_per_launch: 123456\nkernel_source_digest: %s\n" % digest)
    (prof / "stale.md").write_text("traffic_bytes_per_launch: 123456\nkernel_source_digest: 0123456789abcdef\n")
    (prof / "bare.md").write_text("kernel_source_digest: %s\n" % digest)
    real_join = os.path.join
    monkeypatch.setattr(bench.os.path, "join",
                        lambda *a: real_join(str(tmp_path), *a[1:]) if len(a) > 1 and a[1] == "profiles" else real_join(*a))
    assert bench.ncu_traffic("fresh.md") == (123456, "profiles/fresh.md")
    assert bench.ncu_traffic("stale.md")[0] is None and "predates" in bench.ncu_traffic("stale.md")[1]
    assert bench.ncu_traffic("bare.md")[0] is None
    assert bench.ncu_traffic("absent.md") == (None, "no ncu summary")


def test_the_committed_summary_names_its_traffic_and_digest():
    text = open(os.path.join(ROOT, "profiles", "gemm_kernel_moe_prefill_ncu_full.md")).read()
    assert "traffic_bytes_per_launch:" in text and "kernel_source_digest:" in text
