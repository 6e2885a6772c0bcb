"""KV-cache manager's request planning (Section 6): the oracle pinned by the paper's closed form, and the library's
host routine against the oracle."""
import numpy as np
import pytest

from oracle import kv_rule


def test_oracle_threshold_is_128_for_opt_6_7b():
    """Section 6.2: with x = 4096 and one head's weights 4096 x 128, a not-activated head needs MORE than
    w / x = 128 absent entries before prefetching pays (given at least as many tokens in the batch already)."""
    x, w, tokens, heads = 4096, 4096 * 128, 300, 2
    for L2, want in ((127, 0), (128, 0), (129, 1), (200, 1)):
        present = np.ones((tokens, heads), np.uint8)
        present[:250, 0] = 0                  # activated head 0: 250 tokens to refill -> L1 = 250
        present[:L2, 1] = 0
        _, prefetch, L1 = kv_rule.plan(present, np.array([1, 0], np.uint8), x, w)
        assert L1 == 250 and prefetch[1] == want, L2


def test_oracle_rule_equals_the_cost_comparison_and_its_two_cases():
    rng = np.random.default_rng(0)
    for _ in range(200):
        x, w = int(rng.integers(1, 50)), int(rng.integers(1, 2000))
        L1, L2 = int(rng.integers(0, 80)), int(rng.integers(0, 80))
        tokens = 100
        present = np.ones((tokens, 2), np.uint8)
        present[:L1, 0] = 0
        present[tokens - L2:, 1] = 0
        _, prefetch, l1 = kv_rule.plan(present, np.array([1, 0], np.uint8), x, w)
        assert l1 == L1
        # the inequality as printed: L2 > w/x + max(0, L2 - L1)
        assert bool(prefetch[1]) == (L2 > w / x + max(0, L2 - L1))
        # ... which is L2 > w/x when the batch already holds enough tokens, and L1 > w/x otherwise
        assert bool(prefetch[1]) == ((L2 > w / x) if L2 <= L1 else (L1 > w / x))


def test_oracle_merges_every_miss_of_an_activated_head_once():
    present = np.array([[1, 0, 1], [0, 0, 1], [1, 1, 0]], np.uint8)
    request, prefetch, L1 = kv_rule.plan(present, np.array([1, 1, 0], np.uint8), x=4, w=1000)
    assert request.tolist() == [[0, 1, 0], [1, 1, 0], [0, 0, 0]] and prefetch.tolist() == [0, 0, 0] and L1 == 2


@pytest.mark.parametrize("seed", range(6))
def test_library_routine_matches_the_oracle(seed):
    from paper_2505_07239_b200 import binding as cb

    rng = np.random.default_rng(seed)
    tokens, heads = int(rng.integers(1, 400)), int(rng.integers(1, 40))
    present = (rng.random((tokens, heads)) < rng.random()).astype(np.uint8)
    active = (rng.random(heads) < 0.5).astype(np.uint8)
    x, w = int(rng.integers(1, 64)), int(rng.integers(1, 64 * 200))
    want = kv_rule.plan(present, active, x, w)
    got = cb.kv_plan(present, active, x, w)
    assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1]) and got[2] == want[2]


def test_library_routine_rejects_bad_arguments():
    from paper_2505_07239_b200 import binding as cb

    lib = cb.library()
    p = np.ones((2, 2), np.uint8)
    a = np.ones(2, np.uint8)
    assert lib.comet_kv_plan(None, a.ctypes.data, 2, 2, 1, 1, p.ctypes.data, a.ctypes.data, None) == -1
    assert lib.comet_kv_plan(p.ctypes.data, a.ctypes.data, 0, 2, 1, 1, p.ctypes.data, a.ctypes.data, None) == -2
