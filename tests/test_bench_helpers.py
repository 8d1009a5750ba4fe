"""Host-side arithmetic of bench.py: the algorithmic work it divides the measured times by, and the workload tables."""
import importlib.util
import os

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
spec = importlib.util.spec_from_file_location("bench", os.path.join(ROOT, "bench.py"))
bench = importlib.util.module_from_spec(spec)
spec.loader.exec_module(bench)


def test_workload_tables_match_the_configurations():
    assert sum(m * n for m, n in bench.spectral_shapes("c5")) == 402_653_184
    assert sum(m * n for m, n in bench.spectral_shapes("c2")) == 10_992_320
    assert sum(m * n for m, n in bench.spectral_shapes("c3")) == 42_813_120
    assert bench.spectral_shapes("c1a") == [(64, 64)]
    assert bench.ENTRYWISE["c4"]["n"] == 25_600_000 and bench.ENTRYWISE["c4"]["budgets"] == [0.01, 0.001, 0.1]
    assert bench.SPECTRAL["c5"]["budgets"][0] == 4.0 and set(bench.SPECTRAL["c5"]["budgets"]) == {2.0, 4.0, 8.0}
    assert set(bench.SPECTRAL["c3"]["budgets"]) == {1.0, 2.0, 3.0}


def test_algorithmic_work_of_the_reductions():
    # blocked reduction: one triangle of the trailing block per Householder step, 4-byte entries: about (2/3) r^3 bytes
    r = 1024
    b = bench.tridiag_big_bytes([(r, 4096)])
    exact = sum(2.0 * (r - c - 1) ** 2 for c in range(r - 2))
    assert b == exact and abs(b / (2.0 / 3.0 * r ** 3) - 1) < 2e-3
    assert bench.tridiag_big_bytes([(512, 4608), (64, 27)]) == 0.0          # small layers take the other kernel
    # register-resident reduction: 4 r^3 / 3 fp64 flop per layer, small layers only
    assert bench.tridiag_small_flops([(512, 4608), (1024, 4096)]) == 4.0 / 3.0 * 512 ** 3
    # config 5: 96 layers -> 68.7 GB
    assert abs(bench.tridiag_big_bytes(bench.spectral_shapes("c5")) / 1e9 - 68.6) < 0.2


def test_workload_text_names_the_config_and_budget():
    assert "c5" in bench.workload_text("c5", 4.0) and "s=4" in bench.workload_text("c5", 4.0)
    assert "1 % of the length" in bench.workload_text("c4", 0.01)
