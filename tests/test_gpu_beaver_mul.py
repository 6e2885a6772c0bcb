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
