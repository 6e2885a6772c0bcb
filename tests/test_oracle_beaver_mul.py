"""Pins of the oracle's element-wise Beaver product (Eq. 1 element by element)."""
import numpy as np

import oracle
from paper_2505_07239_b200 import workloads as wl

U64 = np.uint64
MASK = (1 << 64) - 1


def _case(golden_dir, name):
    import os

    vals, on = {}, False
    for line in open(os.path.join(golden_dir, "eq1_hand_examples.txt")):
        if line.startswith("case "):
            on = line.split()[1] == name
            continue
        if on and line.strip() and not line.startswith("#"):
            k, *v = line.split()
            vals[k] = np.array([int(t) & MASK for t in v], dtype=object).astype(U64)
    return vals


def test_scalar_hand_example_of_eq1(golden_dir):
    v = _case(golden_dir, "scalar")              # a 1x1x1 matrix product is the scalar product of Eq. 1
    r = oracle.beaver_mul((v["X0"], v["X1"]), (v["Y0"], v["Y1"]), (v["A0"], v["A1"]), (v["B0"], v["B1"]),
                          (v["C0"], v["C1"]))
    for i in (0, 1):
        assert r["D"][i].tolist() == v[f"E{i}"].tolist()       # the fixture names the messages E (of x) and F (of y)
        assert r["E"][i].tolist() == v[f"F{i}"].tolist()
        assert r["Z"][i].tolist() == v[f"Z{i}"].tolist()


def test_reconstructs_the_product_against_python_integers():
    seed, shape = 5, (7, 9)
    x = wl.random_u64(seed, "x", 63).reshape(shape)
    y = wl.random_u64(seed, "y", 63).reshape(shape)
    x[0, 0], y[0, 0] = U64(MASK), U64(MASK)            # (-1) * (-1) = 1
    x[0, 1], y[0, 1] = U64(1 << 63), U64(3)
    x[0, 2], y[0, 2] = U64(0), U64(12345)
    t = wl.dealer_triple_elementwise(seed, "tri", shape)
    r = oracle.beaver_mul(wl.split_shares(x, seed, "x"), wl.split_shares(y, seed, "y"), t["a"][1:], t["b"][1:],
                          t["c"][1:])
    got = r["Z"][0] + r["Z"][1]
    want = [[(int(x[i, j]) * int(y[i, j])) & MASK for j in range(9)] for i in range(7)]
    assert [[int(v) for v in row] for row in got] == want
    # the opened values are x - a and y - b
    assert np.array_equal(r["D"][0] + r["D"][1], x - t["a"][0])
    assert np.array_equal(r["E"][0] + r["E"][1], y - t["b"][0])


def test_agrees_with_pi_matmul_on_one_by_one_products():
    seed = 6
    n = 12
    x, y = wl.random_u64(seed, "x", n), wl.random_u64(seed, "y", n)
    xs, ys = wl.split_shares(x, seed, "x"), wl.split_shares(y, seed, "y")
    t = wl.dealer_triple_elementwise(seed, "tri", (n,))
    r = oracle.beaver_mul(xs, ys, t["a"][1:], t["b"][1:], t["c"][1:])
    for k in range(n):
        one = lambda pair: tuple(np.array([[v[k]]], dtype=U64) for v in pair)   # noqa: E731
        m = oracle.pi_matmul(one(xs), one(ys), one(t["a"][1:]), one(t["b"][1:]), one(t["c"][1:]))
        for i in (0, 1):
            assert int(m["Z"][i][0, 0]) == int(r["Z"][i][k])


def test_planted_mistakes_are_caught():
    seed, n = 7, 32
    x, y = wl.random_u64(seed, "x", n), wl.random_u64(seed, "y", n)
    xs, ys = wl.split_shares(x, seed, "x"), wl.split_shares(y, seed, "y")
    t = wl.dealer_triple_elementwise(seed, "tri", (n,))
    with np.errstate(over="ignore"):
        want = x * y
    good = oracle.beaver_mul(xs, ys, t["a"][1:], t["b"][1:], t["c"][1:])
    assert np.array_equal(good["Z"][0] + good["Z"][1], want)
    same = oracle.beaver_mul(xs, ys, t["b"][1:], t["b"][1:], t["c"][1:])         # b used as the mask of x too
    assert not np.array_equal(same["Z"][0] + same["Z"][1], want)
    both = oracle.beaver_mul(xs, ys, t["a"][1:], t["b"][1:], (t["c"][1], t["c"][1]))   # not a sharing of c
    assert not np.array_equal(both["Z"][0] + both["Z"][1], want)


def test_bias_addition_is_local_and_reconstructs():
    seed, T, N = 8, 5, 7
    z = wl.random_u64(seed, "z", T * N).reshape(T, N)
    b = wl.random_u64(seed, "b", N)
    zs, bs = wl.split_shares(z, seed, "z"), wl.split_shares(b, seed, "b")
    out = [oracle.add_bias(zs[i], bs[i]) for i in (0, 1)]
    assert np.array_equal(out[0] + out[1], z + b[None, :])        # Section 2.1: z = x + y share by share
    assert np.array_equal(out[0], zs[0] + bs[0][None, :])
