"""Pins of the oracle's oblivious shuffle (Protocol 1) against things other than itself."""
import itertools

import numpy as np
import pytest

import oracle
from paper_2505_07239_b200 import workloads as wl

U64 = np.uint64


def test_permutation_acts_as_the_paper_example(golden_dir):
    import os

    for line in open(os.path.join(golden_dir, "shuffle_paper_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        pi, x, want = (np.array(f.split(), dtype=np.int64) for f in line.split("|"))
        got = oracle.apply_permutation(pi.astype(np.int32), x.astype(U64))
        assert got.tolist() == want.tolist()


def test_compose_and_invert_against_numpy():
    rng = np.random.default_rng(0)
    n = 37
    p, q = rng.permutation(n).astype(np.int32), rng.permutation(n).astype(np.int32)
    x = rng.integers(0, 1 << 63, n, dtype=np.uint64)
    # (p o q)(x) = p(q(x)) with numpy fancy indexing as the definition of applying a permutation
    assert np.array_equal(x[oracle.compose_permutations(p, q)], (x[q])[p])
    inv = oracle.invert_permutation(p)
    assert np.array_equal(x[p][inv], x) and np.array_equal(x[inv][p], x)


@pytest.mark.parametrize("rows,cols", [(1, 1), (3, 1), (5, 4), (64, 7), (130, 16)])
def test_shuffle_reconstructs_pi_of_x(rows, cols):
    seed = 100 + rows
    x = wl.random_u64(seed, "x", rows * cols).reshape(rows, cols)
    x0, x1 = wl.split_shares(x, seed, "x")
    m = wl.dealer_shuffle(seed, "sh", rows, cols)
    y, z = oracle.shuffle_online((x0, x1), m["tau"], m["rho"], m["a"], m["b"])
    assert np.array_equal(z[0] + z[1], x[m["pi"]])                 # z = pi(x), exactly
    # the message a party sends is its permuted share under a one-time mask
    assert np.array_equal(y[0] - m["a"][0], x0[m["tau"][0]])
    assert np.array_equal(y[1] - m["a"][1], x1[m["tau"][1]])
    # neither share of z is the permuted share itself (masks do not cancel per party)
    if rows * cols > 4:
        assert not np.array_equal(z[0], x0[m["pi"]])


def test_offline_stage_matches_the_dealer_and_its_identities():
    rows, cols, seed = 41, 3, 7
    m = wl.dealer_shuffle(seed, "sh", rows, cols)
    rho, b = oracle.shuffle_offline(m["pi"], m["tau"], m["a"], m["c"])
    for i in (0, 1):
        assert np.array_equal(rho[i], m["rho"][i]) and np.array_equal(b[i], m["b"][i])
    # pi = rho_0 o tau_1 = rho_1 o tau_0, as operators on a test vector
    x = wl.random_u64(seed, "probe", rows)
    assert np.array_equal(x[m["tau"][1]][rho[0]], x[m["pi"]])
    assert np.array_equal(x[m["tau"][0]][rho[1]], x[m["pi"]])
    # the masks cancel: rho_0(a_1) - b_0 + rho_1(a_0) - b_1 = 0
    zero = m["a"][1][rho[0]] - b[0] + m["a"][0][rho[1]] - b[1]
    assert not zero.any()


def test_all_permutations_of_three_elements_bruteforce():
    x = np.array([[11], [22], [33]], dtype=U64)
    x0 = np.array([[5], [1 << 63], [2 ** 64 - 1]], dtype=U64)
    x1 = x - x0
    perms = [np.array(p, dtype=np.int32) for p in itertools.permutations(range(3))]
    a = (np.array([[1], [2], [3]], dtype=U64), np.array([[2 ** 64 - 4], [9], [0]], dtype=U64))
    c = np.array([[17], [2 ** 63], [3]], dtype=U64)
    for pi in perms:
        for t0 in perms:
            for t1 in perms:
                rho, b = oracle.shuffle_offline(pi, (t0, t1), a, c)
                _, z = oracle.shuffle_online((x0, x1), (t0, t1), rho, a, b)
                want = [int(x[pi[j], 0]) for j in range(3)]
                assert [int(v) for v in (z[0] + z[1])[:, 0]] == want


def test_unshuffle_restores_the_original_order():
    rows, cols, seed = 96, 8, 11
    x = wl.random_u64(seed, "x", rows * cols).reshape(rows, cols)
    xs = wl.split_shares(x, seed, "x")
    m = wl.dealer_shuffle(seed, "sh", rows, cols)
    _, z = oracle.shuffle_online(xs, m["tau"], m["rho"], m["a"], m["b"])
    u = wl.dealer_shuffle(seed, "unsh", rows, cols, inverse_of=m)
    # each party derives its inverse sub-permutations locally
    for i in (0, 1):
        assert np.array_equal(u["tau"][i], oracle.invert_permutation(m["rho"][i]))
        assert np.array_equal(u["rho"][i], oracle.invert_permutation(m["tau"][i]))
    _, w = oracle.shuffle_online(z, u["tau"], u["rho"], u["a"], u["b"])
    assert np.array_equal(w[0] + w[1], x)


def test_same_sub_permutations_align_two_vectors():
    """Shuffling the sparsity vector and the target with the same (rho_i, tau_i) but fresh masks puts them in
    the same secret order, so indexing by the revealed shuffled sparsity is correct."""
    n, seed = 64, 13
    s = (wl.random_u64(seed, "s", n) % np.uint64(2)).reshape(n, 1)
    t = wl.random_u64(seed, "t", n).reshape(n, 1)
    m1 = wl.dealer_shuffle(seed, "sh", n, 1)
    m2 = dict(m1)
    a = tuple(wl.random_u64(seed, f"fresh/a{i}", n).reshape(n, 1) for i in (0, 1))
    c = wl.random_u64(seed, "fresh/c", n).reshape(n, 1)
    _, b = oracle.shuffle_offline(m1["pi"], m1["tau"], a, c)
    m2.update(a=a, b=b)
    _, zs = oracle.shuffle_online(wl.split_shares(s, seed, "s"), m1["tau"], m1["rho"], m1["a"], m1["b"])
    _, zt = oracle.shuffle_online(wl.split_shares(t, seed, "t"), m2["tau"], m2["rho"], m2["a"], m2["b"])
    s_sh, t_sh = (zs[0] + zs[1])[:, 0], (zt[0] + zt[1])[:, 0]
    assert sorted(t_sh[s_sh != 0].tolist()) == sorted(t[:, 0][s[:, 0] != 0].tolist())


def test_planted_mistakes_are_caught():
    """A wrong sign on b, or rho applied to the party's own message, breaks reconstruction."""
    rows, cols, seed = 33, 2, 17
    x = wl.random_u64(seed, "x", rows * cols).reshape(rows, cols)
    xs = wl.split_shares(x, seed, "x")
    m = wl.dealer_shuffle(seed, "sh", rows, cols)
    bad_b = (m["b"][0], np.zeros_like(m["b"][1]) - m["b"][1])
    _, z = oracle.shuffle_online(xs, m["tau"], m["rho"], m["a"], bad_b)
    assert not np.array_equal(z[0] + z[1], x[m["pi"]])
    _, z = oracle.shuffle_online(xs, m["tau"], (m["rho"][1], m["rho"][0]), m["a"], m["b"])
    assert not np.array_equal(z[0] + z[1], x[m["pi"]])
