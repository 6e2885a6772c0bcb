"""Pins of the oracle's SOMM over connected components (Protocol 2 in general)."""
import numpy as np
import pytest

import oracle
from paper_2505_07239_b200 import workloads as wl

U64 = np.uint64


def _same_partition(rc, cc, rl, cl):
    """Two labelings describe the same partition (labels may differ)."""
    a = np.concatenate([rc, cc]).astype(np.int64)
    b = np.concatenate([rl, cl]).astype(np.int64)
    if not np.array_equal(a < 0, b < 0):
        return False
    pairs = set(zip(a[a >= 0].tolist(), b[b >= 0].tolist()))
    return len(pairs) == len({p[0] for p in pairs}) == len({p[1] for p in pairs})


def test_components_of_hand_made_graphs():
    # two blocks that do not touch, one isolated row and one isolated column
    S = np.array([[1, 1, 0, 0, 0],
                  [0, 1, 0, 0, 0],
                  [0, 0, 1, 0, 0],
                  [0, 0, 0, 0, 0],
                  [0, 0, 1, 1, 0]], dtype=np.uint8)
    rc, cc, L = oracle.components_dfs(S)
    assert L == 2 and rc.tolist() == [0, 0, 1, -1, 1] and cc.tolist() == [0, 0, 1, 1, -1]
    # a chain r0-c0-r1-c1-r2-c2: one component although no row shares a column with every other
    S = np.array([[1, 0, 0], [1, 1, 0], [0, 1, 1]], dtype=np.uint8)
    rc, cc, L = oracle.components_dfs(S)
    assert L == 1 and rc.tolist() == [0, 0, 0] and cc.tolist() == [0, 0, 0]
    # a diagonal: every non-zero on its own
    rc, cc, L = oracle.components_dfs(np.eye(4, dtype=np.uint8))
    assert L == 4 and rc.tolist() == [0, 1, 2, 3] and cc.tolist() == [0, 1, 2, 3]


@pytest.mark.parametrize("T,n,density", [(1, 1, 1.0), (7, 9, 0.15), (40, 33, 0.04), (64, 64, 0.02), (30, 50, 0.5)])
def test_components_against_a_library_routine(T, n, density):
    rng = np.random.default_rng(T * 100 + n)
    S = (rng.random((T, n)) < density).astype(np.uint8)
    rc, cc, L = oracle.components_dfs(S)
    rl, cl = wl.bipartite_components(S)
    assert _same_partition(rc, cc, rl, cl)
    assert L == len(set(rl[rl >= 0].tolist()))
    # numbered by the smallest row of each component
    firsts = [int(np.nonzero(rc == t)[0][0]) for t in range(L)]
    assert firsts == sorted(firsts)


def _problem(seed, T, K, n, D, S):
    rng = np.random.default_rng(seed)
    I = np.sort(rng.choice(D, n, replace=False)).astype(np.int32)
    X = wl.random_u64(seed, "X", T * K).reshape(T, K)
    Y = wl.random_u64(seed, "Y", K * D).reshape(K, D)
    tri = wl.dealer_triple_components(seed, "tri", S, K)
    return I, X, Y, tri


@pytest.mark.parametrize("T,K,n,density", [(6, 5, 8, 0.2), (24, 16, 30, 0.05), (16, 8, 12, 0.6)])
def test_reconstructs_the_product_on_the_component_blocks(T, K, n, density):
    seed, D = 40 + T, 3 * n
    rng = np.random.default_rng(seed)
    S = (rng.random((T, n)) < density).astype(np.uint8)
    I, X, Y, tri = _problem(seed, T, K, n, D, S)
    r = oracle.somm_components(wl.split_shares(X, seed, "X"), wl.split_shares(Y, seed, "Y"), I, S,
                               tri["A"][1:], tri["B"][1:], tri["C"][1:])
    same = tri["same_component"]
    want = np.where(same, wl.ring_matmul(X, Y[:, I]), U64(0))
    Z = r["Z"][0] + r["Z"][1]
    assert np.array_equal(Z, want)
    assert np.array_equal(Z[S != 0], wl.ring_matmul(X, Y[:, I])[S != 0])        # every wanted output is there
    assert not r["Z"][0][~same].any() and not r["Z"][1][~same].any()           # Merge: zero in BOTH shares elsewhere
    # Theorem 1: every row / column of a component is masked and sent exactly once, the others never
    live_r, live_c = S.any(axis=1), S.any(axis=0)
    assert r["masked_nodes"] == int(live_r.sum() + live_c.sum())
    E, F = r["E"][0] + r["E"][1], r["F"][0] + r["F"][1]
    assert np.array_equal(E[live_r], (X - tri["A"][0])[live_r]) and not E[~live_r].any()
    assert np.array_equal(F[:, live_c], (Y[:, I] - tri["B"][0])[:, live_c]) and not F[:, ~live_c].any()
    # ... and the dot products are those of the component blocks, no more
    assert r["dot_products"] == int(same.sum())


def test_single_component_is_the_token_shared_protocol():
    seed, T, K, n, D = 51, 9, 12, 10, 25
    S = np.ones((T, n), np.uint8)
    I, X, Y, tri = _problem(seed, T, K, n, D, S)
    xs, ys = wl.split_shares(X, seed, "X"), wl.split_shares(Y, seed, "Y")
    a = oracle.somm_components(xs, ys, I, S, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    b = oracle.somm(xs, ys, I, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    assert a["L"] == 1
    for k in ("E", "F", "Z"):
        for i in (0, 1):
            assert np.array_equal(a[k][i], b[k][i])


def test_splitting_components_saves_dot_products_but_not_messages():
    """The second requirement of Section 5.1: two components in one subgraph cost extra dot products only."""
    S = np.zeros((8, 8), np.uint8)
    S[:4, :4] = 1
    S[4:, 4:] = 1
    seed = 52
    I, X, Y, tri = _problem(seed, 8, 6, 8, 20, S)
    r = oracle.somm_components(wl.split_shares(X, seed, "X"), wl.split_shares(Y, seed, "Y"), I, S,
                               tri["A"][1:], tri["B"][1:], tri["C"][1:])
    assert r["L"] == 2 and r["masked_nodes"] == 16 and r["dot_products"] == 32       # one subgraph would need 64


def test_words_outside_the_blocks_are_ignored():
    seed, T, K, n, D = 53, 12, 7, 14, 40
    rng = np.random.default_rng(seed)
    S = (rng.random((T, n)) < 0.08).astype(np.uint8)
    I, X, Y, tri = _problem(seed, T, K, n, D, S)
    xs, ys = wl.split_shares(X, seed, "X"), wl.split_shares(Y, seed, "Y")
    base = oracle.somm_components(xs, ys, I, S, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    same = tri["same_component"]
    junkC = tuple(np.where(same, c, rng.integers(0, 1 << 63, c.shape, dtype=np.uint64)) for c in tri["C"][1:])
    dead = ~S.any(axis=1)
    junkX = tuple(np.where(dead[:, None], rng.integers(0, 1 << 63, x.shape, dtype=np.uint64), x) for x in xs)
    other = oracle.somm_components(junkX, ys, I, S, tri["A"][1:], tri["B"][1:], junkC)
    for k in ("E", "F", "Z"):
        for i in (0, 1):
            assert np.array_equal(base[k][i], other[k][i])
