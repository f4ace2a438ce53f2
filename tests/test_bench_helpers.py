"""Host-side pieces of bench.py that need no GPU: the ncu traffic record under profiles/ and how the
benchmark line uses it (a figure taken with another library version must not be printed)."""
import importlib.util
import os

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
bench = importlib.util.module_from_spec(spec)
spec.loader.exec_module(bench)


def test_traffic_record_parses_and_matches_the_library_version():
    from paper_2201_13096_b200 import binding, build as build_mod

    rec = bench.load_ncu_traffic()
    assert {"library_version", "workload_prefix", "budget", "candidates_captured", "row_f32_bytes", "arg_u8_bytes"} <= set(rec)
    build_mod.build_host()
    lib = binding.open_library(binding.HOST_LIB_PATH, host_only=True)
    assert int(rec["library_version"]) == lib.spdy_version(), "re-capture the ncu traffic after changing the kernels"
    per_launch, note = bench.ncu_traffic_per_launch(rec, lib.spdy_version(), "bert-base-L72-K42-N4096-B10000", 10000, 1,
                                                    "row_f32", 4096)
    # algorithmic bytes of the launch: 4096 x (335 644 band cells x 4 B + 12 096 B of errors) = 5.55 GB
    assert 0.85 * 5.55e9 < per_launch < 1.05 * 5.55e9 and "profiles/" in note


def test_stale_or_foreign_traffic_records_give_null_and_say_why(tmp_path):
    rec = {"library_version": "1", "workload_prefix": "bert-base-L72-K42", "budget": "10000",
           "candidates_captured": "592", "row_f32_bytes": "7.5e8", "arg_u8_bytes": "1.5e8"}
    value, note = bench.ncu_traffic_per_launch(rec, 2, "bert-base-L72-K42-N4096-B10000", 10000, 1, "row_f32", 4096)
    assert value is None and "version" in note
    value, note = bench.ncu_traffic_per_launch(rec, 1, "resnet50-L53-K42-N1024-B10000", 10000, 1, "row_f32", 1024)
    assert value is None and "another workload" in note
    value, note = bench.ncu_traffic_per_launch({}, 1, "x", 1, 1, "row_f32", 1)
    assert value is None
    path = tmp_path / "t.txt"
    path.write_text("# comment\nlibrary_version = 7  # trailing\nrow_f32_bytes=12\n")
    assert bench.load_ncu_traffic(str(path)) == {"library_version": "7", "row_f32_bytes": "12"}
    assert bench.load_ncu_traffic(str(tmp_path / "missing.txt")) == {}
