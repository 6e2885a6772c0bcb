"""Pins for the CPU oracle: everything here checks `oracle/` against something
other than itself -- hand-computed fixtures, Python big-integer brute force,
numpy's integer matmul on plaintexts, and identities the paper fixes."""
import os

import numpy as np
import pytest

import oracle
from oracle import functionality
from paper_2505_07239_b200 import workloads as wl

U64 = np.uint64
M = 1 << 64


def _to_u64(vals, shape):
    return np.array([v % M for v in vals], dtype=object).astype(U64).reshape(shape)


def _parse_cases(path):
    cases, cur = {}, None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "case":
            cur = {"dims": tuple(int(t) for t in tok[2:5])}
            cases[tok[1]] = cur
        else:
            cur[tok[0]] = [int(t) for t in tok[1:]]
    return cases


# ---------------------------------------------------------------- Eq. 1, hand examples
@pytest.mark.parametrize("name", ["scalar", "dot", "outer"])
def test_eq1_hand_examples(golden_dir, name):
    c = _parse_cases(os.path.join(golden_dir, "eq1_hand_examples.txt"))[name]
    T, K, N = c["dims"]
    sh = {"X": (T, K), "A": (T, K), "E": (T, K), "Y": (K, N), "B": (K, N), "F": (K, N), "C": (T, N), "Z": (T, N)}
    t = {k: (_to_u64(c[k + "0"], s), _to_u64(c[k + "1"], s)) for k, s in sh.items()}
    out = oracle.pi_matmul(t["X"], t["Y"], t["A"], t["B"], t["C"])
    for key in ("E", "F", "Z"):
        for i in (0, 1):
            assert np.array_equal(out[key][i], t[key][i]), (name, key, i)
    # the same through the two-step interface
    E = oracle.reconstruct(*out["E"])
    F = oracle.reconstruct(*out["F"])
    for i in (0, 1):
        assert np.array_equal(oracle.beaver_combine(i, E, F, t["A"][i], t["B"][i], t["C"][i]), t["Z"][i])


# ---------------------------------------------------------------- brute force, big integers
def _bigint_matmul(X, Y):
    T, K = X.shape
    N = Y.shape[1]
    out = np.empty((T, N), dtype=object)
    for r in range(T):
        for c in range(N):
            out[r, c] = sum(int(X[r, k]) * int(Y[k, c]) for k in range(K)) % M
    return out.astype(U64)


def _edge_values(rng, shape):
    """Random words mixed with values at the ring's edges (near 0, 2^63, 2^64)."""
    v = rng.integers(0, M, size=shape, dtype=U64)
    edges = np.array([0, 1, M - 1, (1 << 63) - 1, 1 << 63, (1 << 63) + 1, M - 2, 1 << 32, (1 << 32) - 1],
                     dtype=object).astype(U64)
    pick = rng.random(shape) < 0.5
    v[pick] = edges[rng.integers(0, len(edges), size=int(pick.sum()))]
    return v


def _share(rng, v):
    s0 = rng.integers(0, M, size=v.shape, dtype=U64)
    return s0, v - s0


@pytest.mark.parametrize("T,K,N", [(1, 1, 1), (2, 3, 4), (4, 2, 3), (3, 4, 1), (4, 4, 4)])
def test_pi_matmul_reconstructs_plaintext_bruteforce(T, K, N):
    rng = np.random.default_rng(1000 + 100 * T + 10 * K + N)
    for _ in range(8):
        X, Y = _edge_values(rng, (T, K)), _edge_values(rng, (K, N))
        A, B = _edge_values(rng, (T, K)), _edge_values(rng, (K, N))
        C = _bigint_matmul(A, B)
        out = oracle.pi_matmul(_share(rng, X), _share(rng, Y), _share(rng, A), _share(rng, B), _share(rng, C))
        assert np.array_equal(out["Z"][0] + out["Z"][1], _bigint_matmul(X, Y))
        assert np.array_equal(out["E"][0] + out["E"][1], X - A)
        assert np.array_equal(out["F"][0] + out["F"][1], Y - B)


def test_party_one_carries_the_open_product():
    """With all-zero shares of A, B, C for party 1 and zero E*B, A*F terms, the
    only thing that can make Z_1 non-zero is the i*E*F term of Eq. 1."""
    X = np.array([[3]], dtype=U64)
    Y = np.array([[5]], dtype=U64)
    z = np.zeros((1, 1), dtype=U64)
    out = oracle.pi_matmul((X, z), (Y, z), (z, z), (z, z), (z, z))
    assert out["Z"][0][0, 0] == 0 and out["Z"][1][0, 0] == 15


# ---------------------------------------------------------------- SOMM / SIMM against plaintext
def _setup(T, d, D, bs, active_blocks, groups, seed):
    rng = np.random.default_rng(seed)
    mask = np.zeros(D // bs, dtype=np.uint8)
    mask[list(active_blocks)] = 1
    X = rng.integers(0, M, size=(T, d), dtype=U64)
    Y = rng.integers(0, M, size=(d, groups * D), dtype=U64)
    return rng, mask, X, Y


def test_index_set_bruteforce():
    rng = np.random.default_rng(5)
    for nb, bs, g in [(1, 32, 1), (7, 4, 1), (16, 32, 2), (5, 64, 2)]:
        for _ in range(5):
            mask = (rng.random(nb) < 0.4).astype(np.uint8)
            D = nb * bs
            expect = [gg * D + j for gg in range(g) for j in range(D) if mask[j // bs]]
            got = oracle.index_set(mask, bs, g)
            assert got.tolist() == expect
            assert len(got) == g * bs * int(mask.sum())
    assert oracle.index_set(np.zeros(4, np.uint8), 8).size == 0


@pytest.mark.parametrize("groups", [1, 2])
def test_somm_reconstructs_masked_product(groups):
    T, d, D, bs = 5, 24, 64, 8
    rng, mask, X, Y = _setup(T, d, D, bs, [1, 2, 6], groups, 11)
    I = oracle.index_set(mask, bs, groups)
    n = I.size
    tri = wl.dealer_triple(3, "t", T, d, n)
    out = oracle.somm(_share(rng, X), _share(rng, Y), I, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    assert np.array_equal(out["Z"][0] + out["Z"][1], X @ Y[:, I])          # numpy integer matmul on plaintext
    assert np.array_equal(out["F"][0] + out["F"][1], Y[:, I] - tri["B"][0])
    # message volume of Section "Optimality proof": |X| rows and |Y| columns once each
    assert out["E"][0].size == T * d and out["F"][0].size == d * n


def test_somm_all_ones_equals_dense_and_masked_neurons_are_ignored():
    T, d, D, bs = 4, 16, 32, 8
    rng, mask, X, Y = _setup(T, d, D, bs, [0, 1, 2, 3], 1, 12)
    I = oracle.index_set(mask, bs)
    assert I.tolist() == list(range(D))
    tri = wl.dealer_triple(4, "t", T, d, D)
    Xs, Ys = _share(rng, X), _share(rng, Y)
    sparse = oracle.somm(Xs, Ys, I, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    dense = oracle.pi_matmul(Xs, Ys, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    for key in ("E", "F", "Z"):
        for i in (0, 1):
            assert np.array_equal(sparse[key][i], dense[key][i])
    # now a real mask: garbage in the masked columns of both weight shares changes nothing
    mask[:] = [1, 0, 1, 0]
    I = oracle.index_set(mask, bs)
    tri = wl.dealer_triple(5, "t", T, d, I.size)
    ref = oracle.somm(Xs, Ys, I, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    dead = np.setdiff1d(np.arange(D), I)
    Yg = (Ys[0].copy(), Ys[1].copy())
    Yg[0][:, dead] = rng.integers(0, M, size=(d, dead.size), dtype=U64)
    Yg[1][:, dead] = rng.integers(0, M, size=(d, dead.size), dtype=U64)
    got = oracle.somm(Xs, Yg, I, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    for key in ("E", "F", "Z"):
        for i in (0, 1):
            assert np.array_equal(ref[key][i], got[key][i])
    # Merge: dense layout, exact zeros (in each share) at masked positions
    Zd = oracle.merge_cols(ref["Z"][0], I, D)
    assert np.array_equal(Zd[:, I], ref["Z"][0]) and not Zd[:, dead].any()


def test_simm_reconstructs_and_equals_gathered_matmul():
    T, D, N, bs = 6, 40, 9, 4
    rng = np.random.default_rng(13)
    mask = np.zeros(D // bs, dtype=np.uint8)
    mask[[0, 3, 4, 9]] = 1
    I = oracle.index_set(mask, bs)
    n = I.size
    H = rng.integers(0, M, size=(T, n), dtype=U64)
    W2 = rng.integers(0, M, size=(D, N), dtype=U64)
    tri = wl.dealer_triple(6, "t", T, n, N)
    Hs, Ws = _share(rng, H), _share(rng, W2)
    out = oracle.simm(Hs, Ws, I, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    assert np.array_equal(out["Z"][0] + out["Z"][1], H @ W2[I, :])
    # column-by-row with summed per-column triples == one gathered Pi_MatMul, share by share
    Wg = (oracle.index_rows(Ws[0], I), oracle.index_rows(Ws[1], I))
    assert np.array_equal(Wg[0], Ws[0][I, :])
    one = oracle.pi_matmul(Hs, Wg, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    for key in ("E", "F", "Z"):
        for i in (0, 1):
            assert np.array_equal(out[key][i], one[key][i])
    # rows of W2 outside I do not matter
    dead = np.setdiff1d(np.arange(D), I)
    Wj = (Ws[0].copy(), Ws[1].copy())
    Wj[0][dead] += U64(12345)
    Wj[1][dead] = rng.integers(0, M, size=(dead.size, N), dtype=U64)
    again = oracle.simm(Hs, Wj, I, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    assert np.array_equal(again["Z"][0], out["Z"][0]) and np.array_equal(again["Z"][1], out["Z"][1])


def test_combine_at_matches_full_combine():
    rng = np.random.default_rng(14)
    T, K, N = 7, 19, 11
    E, A = rng.integers(0, M, (T, K), dtype=U64), rng.integers(0, M, (T, K), dtype=U64)
    F, B = rng.integers(0, M, (K, N), dtype=U64), rng.integers(0, M, (K, N), dtype=U64)
    C = rng.integers(0, M, (T, N), dtype=U64)
    rows, cols = rng.integers(0, T, 30), rng.integers(0, N, 30)
    for party in (0, 1):
        full = oracle.beaver_combine(party, E, F, A, B, C)
        # independent statement of Eq. 1 with numpy's integer matmul
        assert np.array_equal(full, C + E @ B + A @ F + U64(party) * (E @ F))
        assert np.array_equal(oracle.beaver_combine_at(party, E, F, A, B, C, rows, cols), full[rows, cols])


# ---------------------------------------------------------------- truncation
def test_truncate_hand_words(golden_dir):
    for line in open(os.path.join(golden_dir, "truncate_hand_words.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        party, f, inp, exp = line.split()
        got = oracle.truncate(int(party), _to_u64([eval(inp)], (1,)), int(f))
        assert int(got[0]) == eval(exp) % M, line


@pytest.mark.parametrize("f", [12, 13, 16])
def test_truncate_invariant_off_by_at_most_one(f):
    rng = np.random.default_rng(f)
    z = rng.integers(-(1 << 40), 1 << 40, size=20000, dtype=np.int64)
    zu = z.view(U64)
    s0 = rng.integers(0, M, size=z.shape, dtype=U64)
    s1 = zu - s0
    t = (oracle.truncate(0, s0, f) + oracle.truncate(1, s1, f)).view(np.int64)
    diff = t - (z >> f)          # floor
    assert set(np.unique(diff).tolist()) <= {0, 1}
    # shares (z, 0) of a non-negative z: exactly the logical shift, and party 1 contributes 0
    zp = np.abs(z).view(U64)
    assert np.array_equal(oracle.truncate(0, zp, f), zp >> U64(f))
    assert not oracle.truncate(1, np.zeros(4, U64), f).any()


# ---------------------------------------------------------------- whole FFN vs float64
@pytest.mark.parametrize("name", ["tiny", "opt125m"])
def test_oracle_ffn_matches_float64(name):
    cfg = wl.CONFIGS[name]
    seed = 7
    T = min(cfg.tokens, 16)
    mask = wl.block_mask(cfg, seed)
    I = oracle.index_set(mask, cfg.block)
    assert np.array_equal(I, wl.active_neurons(mask, cfg.block))
    n, f = I.size, cfg.frac_bits
    W = wl.model_shares(cfg, seed)
    Xr, X0, X1 = wl.activation_shares(cfg, seed, tokens=T)
    up = wl.dealer_triple(seed, "up", T, cfg.d_model, n)
    r = oracle.somm((X0, X1), W["W1"][1:], I, up["A"][1:], up["B"][1:], up["C"][1:])
    H = [oracle.truncate(i, r["Z"][i], f) for i in (0, 1)]
    act = functionality.activation(H[0], H[1], False, f)
    Hs = wl.reshare(act, seed, "act")
    dn = wl.dealer_triple(seed, "dn", T, n, cfg.d_model)
    y = oracle.simm(Hs, W["W2"][1:], I, dn["A"][1:], dn["B"][1:], dn["C"][1:])
    O = [oracle.truncate(i, y["Z"][i], f) for i in (0, 1)]
    got = wl.decode(O[0] + O[1], f)
    ref = functionality.plain_ffn_float64(wl.decode(Xr, f), wl.decode(W["W1"][0], f), wl.decode(W["W2"][0], f), I)
    integer = functionality.plain_ffn_integer(Xr, W["W1"][0], W["W2"][0], I, f)
    err = np.abs(got - ref).max()
    # shared vs unshared integer pipeline: +{0,1} ulp after the up-projection
    # propagates through W2, +{0,1} ulp after the down-projection
    w2abs = np.abs(wl.decode(W["W2"][0], f)[I, :]).sum(axis=0).max()
    assert np.abs(got - wl.decode(integer, f)).max() <= (w2abs + 2.0) * 2.0 ** -f
    if name == "opt125m":
        assert err < 2.0 ** -10
    else:
        # 12 fractional bits with |w| up to 1 over 96 active neurons: a priori
        # bound n * 2^-f on the propagated rounding, above 2^-10 by arithmetic
        assert err < n * 2.0 ** -f
