"""The counting rules behind the benchmark's throughput and roofline figures (CPU)."""
import importlib.util
import os

from paper_2505_07239_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_algorithmic_macs_and_bytes_of_the_headline_configuration():
    b = _bench()
    cfg = wl.CONFIGS["opt1.3b"]
    n = cfg.n_active_blocks(0.9) * cfg.block
    assert n == 832
    T, d = cfg.tokens, cfg.d_model
    # 2 T K N per party per product, both parties, both projections
    assert b.ffn_macs(cfg, T, n) == 2 * 2 * T * d * n + 2 * 2 * T * n * d == 6_979_321_856
    # 8 (6 K N + 6 T K + 2 T N) bytes per party per product
    up = 8 * (6 * d * n + 6 * T * d + 2 * T * n)
    dn = 8 * (6 * n * d + 6 * T * n + 2 * T * d)
    assert b.ffn_bytes(cfg, T, n) == 2 * (up + dn) == 515_899_392


def test_gated_configuration_counts_both_stacked_matrices():
    b = _bench()
    cfg = wl.CONFIGS["llama7b"]
    n = 26 * cfg.block
    T, d = cfg.tokens, cfg.d_model
    assert cfg.groups == 2
    assert b.ffn_macs(cfg, T, n) == 2 * (2 * T * d * 2 * n) + 2 * (2 * T * n * d)


def test_workload_name_states_the_shape():
    b = _bench()
    name = b.workload_name(wl.CONFIGS["opt1.3b"], 0.9)
    for piece in ("tokens=512", "d_model=2048", "d_ff=8192", "sparsity=0.90", "n_active=832"):
        assert piece in name
