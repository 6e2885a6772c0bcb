"""Pins of the oracle's SIMM with per-column row sets R_j (Protocol 3 in general)."""
import numpy as np
import pytest

import oracle
from paper_2505_07239_b200 import workloads as wl

U64 = np.uint64


def _problem(seed, T, n, N, D, density):
    rng = np.random.default_rng(seed)
    I = np.sort(rng.choice(D, n, replace=False)).astype(np.int32)
    S = (rng.random((T, n)) < density).astype(np.uint8)
    X = wl.random_u64(seed, "X", T * n).reshape(T, n)
    Y = wl.random_u64(seed, "Y", D * N).reshape(D, N)
    tri = wl.dealer_triple_rowsets(seed, "tri", S, N)
    return I, S, X, Y, tri


@pytest.mark.parametrize("T,n,N,density", [(1, 1, 1, 1.0), (5, 7, 3, 0.4), (33, 40, 17, 0.15), (64, 96, 8, 0.05)])
def test_reconstructs_the_masked_plaintext_product(T, n, N, density):
    seed, D = 900 + T, 2 * n + 3
    I, S, X, Y, tri = _problem(seed, T, n, N, D, density)
    r = oracle.simm_rowsets(wl.split_shares(X, seed, "X"), wl.split_shares(Y, seed, "Y"), I, S,
                            tri["A"][1:], tri["B"][1:], tri["C"][1:])
    want = wl.ring_matmul(np.where(S != 0, X, U64(0)), Y[I, :])          # (S * X) Y[I], the definition
    assert np.array_equal(r["Z"][0] + r["Z"][1], want)
    # only the entries on the support are masked and sent; everything else of E is zero
    E = r["E"][0] + r["E"][1]
    assert np.array_equal(E, np.where(S != 0, X - tri["A"][0], U64(0)))
    assert not r["E"][0][S == 0].any() and not r["E"][1][S == 0].any()
    # Theorem 2: each non-zero of X is masked exactly once, each row of Y of a non-zero column exactly once
    assert r["masked"] == int(S.sum())
    live = S.any(axis=0)
    F = r["F"][0] + r["F"][1]
    assert np.array_equal(F[live], (Y[I, :] - tri["B"][0])[live]) and not F[~live].any()


def test_all_ones_distribution_is_the_token_shared_protocol():
    seed, T, n, N, D = 31, 12, 20, 9, 50
    I, _, X, Y, _ = _problem(seed, T, n, N, D, 1.0)
    S = np.ones((T, n), np.uint8)
    tri = wl.dealer_triple_rowsets(seed, "tri", S, N)
    xs, ys = wl.split_shares(X, seed, "X"), wl.split_shares(Y, seed, "Y")
    a = oracle.simm_rowsets(xs, ys, I, S, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    b = oracle.simm(xs, ys, I, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    for k in ("E", "F", "Z"):
        for i in (0, 1):
            assert np.array_equal(a[k][i], b[k][i])


def test_words_off_the_support_are_ignored():
    seed, T, n, N, D = 32, 9, 14, 6, 40
    I, S, X, Y, tri = _problem(seed, T, n, N, D, 0.3)
    xs, ys = wl.split_shares(X, seed, "X"), wl.split_shares(Y, seed, "Y")
    base = oracle.simm_rowsets(xs, ys, I, S, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    rng = np.random.default_rng(1)
    junk = lambda a: np.where(S != 0, a, rng.integers(0, 1 << 63, a.shape, dtype=np.uint64))   # noqa: E731
    other = oracle.simm_rowsets((junk(xs[0]), junk(xs[1])), ys, I, S, (junk(tri["A"][1]), junk(tri["A"][2])),
                                tri["B"][1:], tri["C"][1:])
    for k in ("E", "F", "Z"):
        for i in (0, 1):
            assert np.array_equal(base[k][i], other[k][i])


def test_bruteforce_with_python_integers():
    seed, T, n, N, D = 33, 3, 4, 2, 6
    I, S, X, Y, tri = _problem(seed, T, n, N, D, 0.5)
    S[0, 0] = 1
    S[:, 1] = 0                                   # an empty column: not a nonzero column
    tri = wl.dealer_triple_rowsets(seed, "tri", S, N)
    r = oracle.simm_rowsets(wl.split_shares(X, seed, "X"), wl.split_shares(Y, seed, "Y"), I, S,
                            tri["A"][1:], tri["B"][1:], tri["C"][1:])
    M = (1 << 64) - 1
    for t in range(T):
        for q in range(N):
            want = sum(int(X[t, c]) * int(Y[I[c], q]) for c in range(n) if S[t, c]) & M
            assert (int(r["Z"][0][t, q]) + int(r["Z"][1][t, q])) & M == want
    assert not r["F"][0][1].any() and not r["F"][1][1].any()


def test_planted_mistake_is_caught():
    """Handing the protocol a C' built from the unmasked A' (as the token-shared dealer would) breaks it."""
    seed, T, n, N, D = 34, 8, 10, 4, 30
    I, S, X, Y, tri = _problem(seed, T, n, N, D, 0.4)
    wrong = wl.split_shares(wl.ring_matmul(tri["A"][0], tri["B"][0]), seed, "wrongC")
    r = oracle.simm_rowsets(wl.split_shares(X, seed, "X"), wl.split_shares(Y, seed, "Y"), I, S,
                            tri["A"][1:], tri["B"][1:], wrong)
    assert not np.array_equal(r["Z"][0] + r["Z"][1], wl.ring_matmul(np.where(S != 0, X, U64(0)), Y[I, :]))


def test_token_block_masks_generator():
    m = wl.token_block_masks(5, "tm", 64, 26, 0.05)
    assert m.shape == (64, 26) and m.dtype == np.uint8
    assert m.sum(axis=0).min() >= 1 and m.sum(axis=1).min() >= 1 and m.mean() < 0.2
