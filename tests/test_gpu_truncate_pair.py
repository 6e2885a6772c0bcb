"""GPU parity of the truncation with a dealer's pair (comet_truncate_pair, through the C ABI) against the CPU oracle."""
import ctypes

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


def _case(seed, shape, f, bits):
    n = int(np.prod(shape))
    z = (wl.random_u64(seed, "z", n).view(np.int64) >> np.int64(64 - bits)).view(np.uint64).reshape(shape)
    return z, wl.split_shares(z, seed, "z"), wl.dealer_truncation_pair(seed, "pair", shape, f)


@pytest.mark.parametrize("shape,f", [((1,), 12), ((2,), 16), ((7, 9), 13), ((512, 832), 16), ((1025, 333), 1),
                                     ((32, 4096), 31)])
def test_truncate_pair_matches_oracle(shape, f):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb

    z, zs, pair = _case(900 + f + shape[0], shape, f, 44)
    ref = oracle.truncate_pair(zs, pair["r"][1:], pair["rp"][1:], f)
    Z = [_dev(v) for v in zs]
    M = cb.truncate_pair(Z, [_dev(v) for v in pair["r"][1:]], [_dev(v) for v in pair["rp"][1:]], f)
    torch.cuda.synchronize()
    for i in (0, 1):
        assert np.array_equal(_host(M[i]), ref["M"][i])
        assert np.array_equal(_host(Z[i]), ref["OUT"][i])
    diff = (_host(Z[0]) + _host(Z[1])).view(np.int64) - (z.view(np.int64) >> np.int64(f))
    assert diff.min() >= -1 and diff.max() <= 0


def test_truncate_pair_on_random_ring_words_and_odd_alignment():
    """Shares of arbitrary ring words (where the protocol's result is meaningless but still defined) and buffers
    that start 8 bytes off a 16-byte boundary: the word-wise kernels run and give the oracle's bits."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb

    seed, n, f = 31, 4098, 16
    z = wl.random_u64(seed, "z", n)
    zs = wl.split_shares(z, seed, "z")
    pair = wl.dealer_truncation_pair(seed, "pair", (n,), f)
    ref = oracle.truncate_pair(zs, pair["r"][1:], pair["rp"][1:], f)

    def off(a):                                     # a view that starts one word into a fresh allocation
        buf = torch.empty(n + 1, dtype=torch.int64, device="cuda")
        buf[1:].copy_(_dev(a))
        return buf[1:]

    Z = [off(v) for v in zs]
    assert Z[0].data_ptr() % 16 == 8
    M = cb.truncate_pair(Z, [off(v) for v in pair["r"][1:]], [off(v) for v in pair["rp"][1:]], f)
    torch.cuda.synchronize()
    for i in (0, 1):
        assert np.array_equal(_host(M[i]), ref["M"][i])
        assert np.array_equal(_host(Z[i]), ref["OUT"][i])


def test_truncate_pair_after_the_ffn_up_projection_agrees_with_plaintext():
    """The protocol in its place: Z of the up-projection (scale 2f) truncated to scale f, against the plaintext
    product of the decoded inputs: reconstruction equals floor(x w / 2^f) or one less."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb

    seed, T, n, f = 41, 33, 96, 16
    x = wl.encode(wl.random_normal(seed, "x", T * n, 1.0).reshape(T, n), f)
    w = wl.encode(wl.random_normal(seed, "w", T * n, 0.5).reshape(T, n), f)
    with np.errstate(over="ignore"):
        z = x * w                                    # an element-wise stand-in for a product at scale 2f
    zs = wl.split_shares(z, seed, "z")
    pair = wl.dealer_truncation_pair(seed, "pair", (T, n), f)
    Z = [_dev(v) for v in zs]
    cb.truncate_pair(Z, [_dev(v) for v in pair["r"][1:]], [_dev(v) for v in pair["rp"][1:]], f)
    torch.cuda.synchronize()
    got = (_host(Z[0]) + _host(Z[1])).view(np.int64)
    want = (x.view(np.int64) * w.view(np.int64)) >> np.int64(f)
    assert set(np.unique(got - want).tolist()) <= {-1, 0}


def test_truncate_pair_argument_errors():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb

    lib = cb.library()
    t = [torch.zeros(4, dtype=torch.int64, device="cuda") for _ in range(8)]
    pair = ctypes.c_void_p * 2
    ok = [pair(t[2 * k].data_ptr(), t[2 * k + 1].data_ptr()) for k in range(4)]
    assert lib.comet_truncate_pair(None, ok[0], ok[1], ok[2], ok[3], 4, 16) == 0
    assert lib.comet_truncate_pair(None, ok[0], ok[1], ok[2], ok[3], 0, 16) == -2
    assert lib.comet_truncate_pair(None, ok[0], ok[1], ok[2], ok[3], 4, 0) == -2
    assert lib.comet_truncate_pair(None, ok[0], ok[1], ok[2], ok[3], 4, 32) == -2
    bad = pair(t[0].data_ptr(), None)
    assert lib.comet_truncate_pair(None, bad, ok[1], ok[2], ok[3], 4, 16) == -1
    assert lib.comet_truncate_pair(None, ok[0], ok[1], ok[2], bad, 4, 16) == -1
    torch.cuda.synchronize()
