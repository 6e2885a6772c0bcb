"""The seeded input generators: determinism, mask structure, sharing."""
import numpy as np
import pytest

from paper_2505_07239_b200 import workloads as wl


def test_generator_is_counter_based_and_seeded():
    a = wl.random_u64(1, "s", 1000)
    assert np.array_equal(a[100:200], wl.random_u64(1, "s", 100, offset=100))
    assert not np.array_equal(a, wl.random_u64(2, "s", 1000))
    assert not np.array_equal(a, wl.random_u64(1, "t", 1000))
    bits = np.unpackbits(a.view(np.uint8)).mean()
    assert 0.49 < bits < 0.51
    u = wl.random_unit(3, "u", 20000)
    assert 0.0 <= u.min() and u.max() < 1.0 and abs(u.mean() - 0.5) < 0.01
    g = wl.random_normal(3, "g", 20000, 0.02)
    assert abs(g.std() - 0.02) < 0.001 and abs(g.mean()) < 0.001


def test_encode_decode_and_shares():
    v = np.array([-1.0, -0.5, 0.0, 0.25, 0.99993], dtype=np.float64)
    r = wl.encode(v, 12)
    assert r.view(np.int64).tolist() == [-4096, -2048, 0, 1024, 4096]
    assert np.allclose(wl.decode(r, 12), [-1, -0.5, 0, 0.25, 1.0])
    s0, s1 = wl.split_shares(r, 5, "x")
    assert np.array_equal(s0 + s1, r) and not np.array_equal(s0, r)


@pytest.mark.parametrize("name,expect", [("tiny", 3), ("opt125m", 10), ("llama7b", 26), ("opt6.7b-decode", 41)])
def test_active_block_counts(name, expect):
    cfg = wl.CONFIGS[name]
    assert cfg.n_active_blocks() == expect
    m = wl.block_mask(cfg, 11)
    assert m.dtype == np.uint8 and m.size == cfg.n_blocks
    if cfg.mask_kind == "pool_union":
        assert 0 < m.sum() <= expect and m.sum() >= expect - 3    # union of per-token masks ~ the pool
    else:
        assert m.sum() == expect


def test_sweep_counts_and_fresh_masks_per_step():
    cfg = wl.CONFIGS["opt1.3b"]
    assert [cfg.n_active_blocks(s) for s in wl.SWEEP_SPARSITIES] == [256, 128, 51, 26, 13]
    assert wl.block_mask(cfg, 1, 0.0).all()
    dec = wl.CONFIGS["opt6.7b-decode"]
    assert not np.array_equal(wl.block_mask(dec, 1, step=0), wl.block_mask(dec, 1, step=1))


def test_runs_mask_is_clustered():
    cfg = wl.CONFIGS["opt125m"]
    runs = []
    for seed in range(40):
        m = wl.block_mask(cfg, seed)
        edges = np.diff(np.concatenate([[0], m, [0]]).astype(int))
        runs.append(m.sum() / (edges == 1).sum())
    assert np.mean(runs) > 1.8      # uniform placement of 10 in 96 would give about 1.1


def test_dealer_triple_is_a_product():
    t = wl.dealer_triple(9, "t", 3, 5, 4)
    A, B, C = t["A"][0], t["B"][0], t["C"][0]
    want = np.array([[sum(int(A[r, k]) * int(B[k, c]) for k in range(5)) % (1 << 64) for c in range(4)]
                     for r in range(3)], dtype=object).astype(np.uint64)
    assert np.array_equal(C, want)
    for key in "ABC":
        assert np.array_equal(t[key][1] + t[key][2], t[key][0])


def test_clustered_token_masks_fall_into_the_requested_groups():
    tm = wl.token_block_masks_clustered(3, "x", 200, 40, 5, 0.3, dead_tokens=3, dead_blocks=2)
    assert tm.shape == (200, 40) and tm.dtype == np.uint8
    rl, cl = wl.bipartite_components(tm)
    assert len(set(rl[rl >= 0].tolist())) >= 5                      # at least one component per group
    assert int((cl < 0).sum()) >= 2 and int((rl < 0).sum()) >= 3    # the blocks and tokens without any entry
    # no edge joins two groups: every component's tokens use only that component's blocks
    for r in range(200):
        for b in np.nonzero(tm[r])[0]:
            assert rl[r] == cl[b]
    # same seed, same mask; another stream, another mask
    assert np.array_equal(tm, wl.token_block_masks_clustered(3, "x", 200, 40, 5, 0.3, dead_tokens=3, dead_blocks=2))
    assert not np.array_equal(tm, wl.token_block_masks_clustered(3, "y", 200, 40, 5, 0.3, dead_tokens=3, dead_blocks=2))


def test_plain_token_masks_leave_no_token_and_no_block_empty():
    tm = wl.token_block_masks(4, "t", 64, 26, 0.05)
    assert tm.sum(axis=0).min() >= 1 and tm.sum(axis=1).min() >= 1
