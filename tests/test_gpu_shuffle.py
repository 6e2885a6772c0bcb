"""GPU parity of the oblivious shuffle (comet_shuffle, through the C ABI) against the CPU oracle, bit for bit."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2505_07239_b200 import workloads as wl  # noqa: E402


@pytest.fixture(scope="module")
def cb():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding

    return binding


def _dev64(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int64)).cuda()


def _dev32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def _host(t):
    return t.cpu().numpy().view(np.uint64)


def _run(cb, xs, m):
    Y, Z = cb.shuffle([_dev64(v) for v in xs], [_dev32(v) for v in m["tau"]], [_dev32(v) for v in m["rho"]],
                      [_dev64(v) for v in m["a"]], [_dev64(v) for v in m["b"]])
    torch.cuda.synchronize()
    return [_host(t) for t in Y], [_host(t) for t in Z]


# rows x cols: single row, scalar (odd / one column) paths, ragged sizes, the activation matrices of the workloads
SHAPES = [(1, 8), (3, 1), (130, 7), (257, 2), (16, 256), (512, 2048), (4097, 34), (8192, 1)]


@pytest.mark.parametrize("rows,cols", SHAPES)
def test_shuffle_matches_oracle(cb, rows, cols):
    seed = 300 + rows + cols
    x = wl.random_u64(seed, "x", rows * cols).reshape(rows, cols)
    xs = wl.split_shares(x, seed, "x")
    m = wl.dealer_shuffle(seed, "sh", rows, cols)
    y_ref, z_ref = oracle.shuffle_online(xs, m["tau"], m["rho"], m["a"], m["b"])
    Y, Z = _run(cb, xs, m)
    for i in (0, 1):
        assert np.array_equal(Y[i], y_ref[i]) and np.array_equal(Z[i], z_ref[i])
    assert np.array_equal(Z[0] + Z[1], x[m["pi"]])


def test_unshuffle_with_device_inverted_permutations(cb):
    rows, cols, seed = 512, 768, 41
    x = wl.random_u64(seed, "x", rows * cols).reshape(rows, cols)
    xs = wl.split_shares(x, seed, "x")
    m = wl.dealer_shuffle(seed, "sh", rows, cols)
    _, Z = _run(cb, xs, m)
    u = wl.dealer_shuffle(seed, "unsh", rows, cols, inverse_of=m)
    # each party inverts its own sub-permutations on the device
    tau_inv = [cb.invert_permutation(_dev32(m["rho"][i])) for i in (0, 1)]
    rho_inv = [cb.invert_permutation(_dev32(m["tau"][i])) for i in (0, 1)]
    for i in (0, 1):
        assert np.array_equal(tau_inv[i].cpu().numpy(), oracle.invert_permutation(m["rho"][i]))
        assert np.array_equal(rho_inv[i].cpu().numpy(), oracle.invert_permutation(m["tau"][i]))
    Y2, W = cb.shuffle([_dev64(v) for v in Z], tau_inv, rho_inv, [_dev64(v) for v in u["a"]],
                       [_dev64(v) for v in u["b"]])
    torch.cuda.synchronize()
    y_ref, w_ref = oracle.shuffle_online(Z, u["tau"], u["rho"], u["a"], u["b"])
    for i in (0, 1):
        assert np.array_equal(_host(W[i]), w_ref[i]) and np.array_equal(_host(Y2[i]), y_ref[i])
    assert np.array_equal(_host(W[0]) + _host(W[1]), x)


def test_unaligned_views_take_the_8_byte_path(cb):
    rows, cols, seed = 64, 6, 43
    x = wl.random_u64(seed, "x", rows * cols).reshape(rows, cols)
    xs = wl.split_shares(x, seed, "x")
    m = wl.dealer_shuffle(seed, "sh", rows, cols)
    _, z_ref = oracle.shuffle_online(xs, m["tau"], m["rho"], m["a"], m["b"])

    def off(a):          # the same words, starting 8 bytes into an allocation
        buf = torch.empty(a.size + 1, dtype=torch.int64, device="cuda")
        buf[1:] = torch.from_numpy(np.ascontiguousarray(a).view(np.int64).reshape(-1)).cuda()
        return buf[1:].view(a.shape)

    Y, Z = cb.shuffle([off(v) for v in xs], [_dev32(v) for v in m["tau"]], [_dev32(v) for v in m["rho"]],
                      [off(v) for v in m["a"]], [off(v) for v in m["b"]])
    torch.cuda.synchronize()
    for i in (0, 1):
        assert np.array_equal(_host(Z[i]), z_ref[i])


def test_bad_permutation_entry_is_flagged_not_followed(cb):
    rows, cols, seed = 32, 4, 47
    x = wl.random_u64(seed, "x", rows * cols).reshape(rows, cols)
    xs = wl.split_shares(x, seed, "x")
    m = wl.dealer_shuffle(seed, "sh", rows, cols)
    tau0 = m["tau"][0].copy()
    tau0[5] = rows + 100            # out of range: the kernel's bounds check must catch it
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y, _ = cb.shuffle([_dev64(v) for v in xs], [_dev32(tau0), _dev32(m["tau"][1])], [_dev32(v) for v in m["rho"]],
                      [_dev64(v) for v in m["a"]], [_dev64(v) for v in m["b"]], bad_index_flag=flag)
    torch.cuda.synchronize()
    assert int(flag.item()) == 1
    y0 = _host(Y[0])
    assert np.array_equal(y0[5], m["a"][0][5])                     # the missing row counted as zero
    keep = np.arange(rows) != 5
    assert np.array_equal(y0[keep], (xs[0][m["tau"][0]] + m["a"][0])[keep])


def test_shuffle_argument_errors(cb):
    import ctypes

    lib = cb.library()
    t = torch.zeros(8, dtype=torch.int64, device="cuda")
    p = torch.zeros(4, dtype=torch.int32, device="cuda")
    ok64 = (ctypes.c_void_p * 2)(t.data_ptr(), t.data_ptr())
    ok32 = (ctypes.c_void_p * 2)(p.data_ptr(), p.data_ptr())
    null = (ctypes.c_void_p * 2)(None, None)
    assert lib.comet_shuffle(None, null, ok32, ok32, ok64, ok64, ok64, ok64, 4, 2, None) == -1
    assert lib.comet_shuffle(None, ok64, ok32, ok32, ok64, ok64, ok64, ok64, 0, 2, None) == -2
    assert lib.comet_shuffle(None, ok64, ok32, ok32, ok64, ok64, ok64, ok64, 4, 0, None) == -2
    assert lib.comet_invert_permutation(None, None, p.data_ptr(), 4, None) == -1
    assert lib.comet_invert_permutation(None, p.data_ptr(), p.data_ptr(), 0, None) == -2
    torch.cuda.synchronize()
