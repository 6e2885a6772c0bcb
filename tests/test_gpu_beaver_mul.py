"""GPU parity of the element-wise Beaver product (comet_beaver_mul, through the C ABI) against the CPU oracle."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2505_07239_b200 import workloads as wl  # noqa: E402


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int64)).cuda()


def _host(t):
    return t.cpu().numpy().view(np.uint64)


@pytest.mark.parametrize("shape", [(1,), (2,), (7, 9), (256, 1664), (1025, 333)])
def test_beaver_mul_matches_oracle(shape):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb

    seed = 500 + len(shape) + shape[0]
    n = int(np.prod(shape))
    x, y = wl.random_u64(seed, "x", n).reshape(shape), wl.random_u64(seed, "y", n).reshape(shape)
    xs, ys = wl.split_shares(x, seed, "x"), wl.split_shares(y, seed, "y")
    t = wl.dealer_triple_elementwise(seed, "tri", shape)
    ref = oracle.beaver_mul(xs, ys, t["a"][1:], t["b"][1:], t["c"][1:])
    D, E, Z = cb.beaver_mul([_dev(v) for v in xs], [_dev(v) for v in ys], [_dev(v) for v in t["a"][1:]],
                            [_dev(v) for v in t["b"][1:]], [_dev(v) for v in t["c"][1:]])
    torch.cuda.synchronize()
    for i in (0, 1):
        assert np.array_equal(_host(D[i]), ref["D"][i])
        assert np.array_equal(_host(E[i]), ref["E"][i])
        assert np.array_equal(_host(Z[i]), ref["Z"][i])
    with np.errstate(over="ignore"):
        assert np.array_equal(_host(Z[0]) + _host(Z[1]), x * y)


def test_gated_activation_product_end_to_end():
    """ReLU(gate) * up on shares: the comparison is the ideal functionality, the product is the library's, and the
    truncated result equals floor(relu(gate) * up / 2^f) up to the +1 of local truncation."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb

    seed, T, n, f = 77, 40, 128, 16
    gate = wl.encode(wl.random_normal(seed, "gate", T * n, 1.0).reshape(T, n), f)
    up = wl.encode(wl.random_normal(seed, "up", T * n, 1.0).reshape(T, n), f)
    relu = np.maximum(gate.view(np.int64), 0).view(np.uint64)
    rs, us = wl.split_shares(relu, seed, "relu"), wl.split_shares(up, seed, "up")
    t = wl.dealer_triple_elementwise(seed, "tri", (T, n))
    _, _, Z = cb.beaver_mul([_dev(v) for v in rs], [_dev(v) for v in us], [_dev(v) for v in t["a"][1:]],
                            [_dev(v) for v in t["b"][1:]], [_dev(v) for v in t["c"][1:]])
    torch.cuda.synchronize()
    z = [_host(v) for v in Z]
    h = oracle.truncate(0, z[0], f) + oracle.truncate(1, z[1], f)
    want = (relu.view(np.int64) * up.view(np.int64)) >> np.int64(f)
    diff = h.view(np.int64) - want
    assert diff.min() >= 0 and diff.max() <= 1


def test_beaver_mul_argument_errors():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import ctypes

    from paper_2505_07239_b200 import binding as cb

    t = torch.zeros(4, dtype=torch.int64, device="cuda")
    ok = (ctypes.c_void_p * 2)(t.data_ptr(), t.data_ptr())
    null = (ctypes.c_void_p * 2)(None, None)
    lib = cb.library()
    assert lib.comet_beaver_mul(None, ok, ok, ok, null, ok, ok, ok, ok, 4) == -1
    assert lib.comet_beaver_mul(None, ok, ok, ok, ok, ok, ok, ok, ok, 0) == -2
    torch.cuda.synchronize()


def test_gated_ffn_chain_with_bias_only_the_comparison_is_ideal():
    """Whole gated FFN on shares with everything but the comparison done by the library: up-projection [gate || up],
    bias, truncation, ReLU(gate) by the ideal functionality, the element-wise Beaver product, truncation, and the
    down-projection.  Bit-exact against the oracle chain, and close to the float64 FFN."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb
    from tests import harness as hz

    cfg = wl.FFNConfig("gated-chain", 40, 128, 512, 64, 16, True, 0.5, "uniform", "normal", "normal0.02")
    seed, T, d, f, bs = 606, cfg.tokens, cfg.d_model, cfg.frac_bits, cfg.block
    W = wl.model_shares(cfg, seed)
    Xr, X0, X1 = wl.activation_shares(cfg, seed)
    mask = wl.block_mask(cfg, seed)
    I1, Ig = oracle.index_set(mask, bs, 1), oracle.index_set(mask, bs, 2)
    n = I1.size
    bias_plain = wl.encode(wl.random_normal(seed, "bias", 2 * n, 0.1), 2 * f)        # at the product's scale 2f
    bias = wl.split_shares(bias_plain, seed, "bias")

    ctx = hz.make_context(cfg, T, cb.PATH_LIMB)
    hz.load_weights(ctx, cfg, W)
    for p, Xs in ((0, X0), (1, X1)):
        ctx.load_shares(p, cb.X, cb.to_device(Xs))
    assert ctx.set_mask(mask) == n
    tri = wl.dealer_triple(seed, "up", T, d, 2 * n)
    hz.load_triple_up(ctx, tri)
    ctx.ffn_up(T)
    ref = oracle.somm((X0, X1), (hz.oracle_up_operand(cfg, W, 1), hz.oracle_up_operand(cfg, W, 2)), Ig,
                      tri["A"][1:], tri["B"][1:], tri["C"][1:])
    # bias and truncation: library on its own copies of Z (stateless calls), oracle beside it
    Zdev = [_dev(ctx.get(p, cb.Z_UP, (T, 2 * n))) for p in (0, 1)]
    cb.add_bias(Zdev, [_dev(b) for b in bias])
    torch.cuda.synchronize()
    Zb_ref = [oracle.add_bias(ref["Z"][p], bias[p]) for p in (0, 1)]
    for p in (0, 1):
        assert np.array_equal(_host(Zdev[p]), Zb_ref[p])
    Hpre = [oracle.truncate(p, Zb_ref[p], f) for p in (0, 1)]
    gate = (Hpre[0][:, :n] + Hpre[1][:, :n]).view(np.int64)
    relu = np.maximum(gate, 0).view(np.uint64)                                       # the only ideal step
    rs = wl.split_shares(relu, seed, "relu")
    us = (np.ascontiguousarray(Hpre[0][:, n:]), np.ascontiguousarray(Hpre[1][:, n:]))
    tm = wl.dealer_triple_elementwise(seed, "mul", (T, n))
    _, _, Zm = cb.beaver_mul([_dev(v) for v in rs], [_dev(v) for v in us], [_dev(v) for v in tm["a"][1:]],
                             [_dev(v) for v in tm["b"][1:]], [_dev(v) for v in tm["c"][1:]])
    torch.cuda.synchronize()
    mref = oracle.beaver_mul(rs, us, tm["a"][1:], tm["b"][1:], tm["c"][1:])
    H = []
    for p in (0, 1):
        assert np.array_equal(_host(Zm[p]), mref["Z"][p])
        H.append(oracle.truncate(p, mref["Z"][p], f))
    for p in (0, 1):
        ctx.load_shares(p, cb.H, cb.to_device(H[p]))
    trd = wl.dealer_triple(seed, "down", T, n, d)
    hz.load_triple_down(ctx, trd)
    ctx.ffn_down(T)
    ctx.truncate(cb.Y)
    refd = oracle.simm((H[0], H[1]), W["W2"][1:], I1, trd["A"][1:], trd["B"][1:], trd["C"][1:])
    O = []
    for p in (0, 1):
        O.append(ctx.get(p, cb.Y, (T, d)))
        assert np.array_equal(O[p], oracle.truncate(p, refd["Z"][p], f))
    ctx.close()
    # against the float64 gated FFN with the same bias (bias decoded at scale 2f)
    x = wl.decode(Xr, f)
    g64 = x @ wl.decode(W["WG"][0], f)[:, I1] + wl.decode(bias_plain[:n], 2 * f)
    u64 = x @ wl.decode(W["W1"][0], f)[:, I1] + wl.decode(bias_plain[n:], 2 * f)
    want = (np.maximum(g64, 0.0) * u64) @ wl.decode(W["W2"][0], f)[I1, :]
    got = wl.decode(O[0] + O[1], f)
    assert np.abs(got - want).max() < 2.0 ** -10
