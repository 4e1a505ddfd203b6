"""Host-side pieces of the benchmark (no GPU): byte accounting and the run specification."""
import importlib.util
import os

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
spec = importlib.util.spec_from_file_location("bench", os.path.join(ROOT, "bench.py"))
bench = importlib.util.module_from_spec(spec)
spec.loader.exec_module(bench)


def test_algorithmic_bytes_by_hand():
    cfg = dict(cache_width=4, fanouts=[2], feat_dtype="bf16", feat_dim=8)
    # one step: 3 frontier nodes, 5 picks, 2 new ids, 1 refreshed node, r = 1
    n, m = [3, 5], [5]
    total, feat = bench.algorithmic_bytes(cfg, n, m, [1], 1)
    step = 16 * 3 + 4 * 4 * 3 + 8 * 1 * 1 + 4 * 5 + 8 * (3 + 5) + 8 * 2 + 8 * 5 + 4 * (3 + 1) + 4 * 2
    assert feat == 5 * (4 + 2 * 8 * 2)
    assert total == step + feat


def test_run_spec_prefers_the_otf_run():
    from workloads import get_config
    assert bench.run_spec(get_config("mid")) == ("otf", 0.1)
    assert bench.run_spec(get_config("scale")) == ("otf", 0.1)
