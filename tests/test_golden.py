"""The paper's printed context numbers (tests/golden/): internally consistent, and quoted by the benchmark."""
import os

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def load():
    vals = {}
    for ln in open(os.path.join(ROOT, "tests", "golden", "paper_context_numbers.txt")):
        ln = ln.strip()
        if ln and not ln.startswith("#"):
            k, v = [x.strip() for x in ln.split("=", 1)]
            vals[k] = v
    return vals


def test_abstract_average_is_the_mean_of_the_table_row():
    v = load()
    row = [float(v[k]) for k in v if k.startswith("table2_flexdraft_qwen3_8b_speedup_")]
    assert len(row) == 5
    assert abs(sum(row) / 5 - float(v["abstract_avg_speedup_qwen3_8b"])) < 0.005


def test_benchmark_quotes_the_same_context():
    import sys
    sys.path.insert(0, ROOT)
    import bench
    ctx = bench.paper_context()
    v = load()
    assert ctx["speedup_over_autoregressive"] == float(v["abstract_avg_speedup_qwen3_8b"])
    assert ctx["hardware"] == v["hardware"] and "context only" in ctx["note"]
