"""The allocation-free Pi_MatMul entry point (comet_beaver_matmul_static).

It serves callers that cannot allocate device memory at call time (a process
whose framework already owns all GPU memory, or a serving loop that must not
stall in cudaMalloc), by keeping the product's message buffers in an array
inside the library.  Here it is called through the C ABI twice in a row and
compared, bit for bit, with the CPU oracle's dense Beaver product on the same
words and with the context-based entry points (comet_ffn_up under an all-ones
mask computes the same dense product).  Collected last on purpose.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2505_07239_b200 import workloads as wl  # noqa: E402


def _existing_entry_points(cb, X, A, Y, B, C, T, K, N):
    """Z_i from comet_ffn_up: d_model = K, d_ff = N, every block active, tensor-core path."""
    ctx = cb.Comet(T, K, N, 16, 12, False, 0, 0, cb.PATH_LIMB)
    for p in (0, 1):
        ctx.load_shares(p, cb.X, X[p])
        ctx.load_shares(p, cb.W1, Y[p])
        ctx.load_shares(p, cb.W2, torch.zeros((K, N), dtype=torch.int64, device="cuda"))
    assert ctx.set_mask(np.ones(N // 16, np.uint8)) == N
    for p in (0, 1):
        ctx.load_shares(p, cb.A_UP, A[p])
        ctx.load_shares(p, cb.B_UP, B[p])
        ctx.load_shares(p, cb.C_UP, C[p])
    ctx.ffn_up(T)
    out = [ctx.get(p, cb.Z_UP, (T, N)) for p in (0, 1)]
    ctx.close()
    return out


def test_static_scratch_matmul_matches_oracle_and_context_path_twice():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb

    # two different problems back to back: the second reuses (and fully overwrites) the first one's scratch
    for call, (T, K, N) in enumerate([(40, 64, 96), (130, 256, 208)]):
        def draw(name, shape):
            return [wl.random_u64(77 + call, f"static/{name}/{p}", shape[0] * shape[1]).reshape(shape)
                    for p in (0, 1)]

        Xh, Ah = draw("X", (T, K)), draw("A", (T, K))
        Yh, Bh = draw("Y", (N, K)), draw("B", (N, K))           # stored output-feature-major: the paper's Y^T, B^T
        Ch = draw("C", (T, N))
        X, A, Y, B, C = ([cb.to_device(v) for v in pair] for pair in (Xh, Ah, Yh, Bh, Ch))
        Z = [torch.full((T, N), -1, dtype=torch.int64, device="cuda") for _ in (0, 1)]
        assert cb.beaver_matmul_static(X, A, Y, B, C, Z) == cb.OK
        torch.cuda.synchronize()
        ref = oracle.pi_matmul(Xh, [np.ascontiguousarray(v.T) for v in Yh], Ah,
                               [np.ascontiguousarray(v.T) for v in Bh], Ch)
        same = _existing_entry_points(cb, X, A, Y, B, C, T, K, N)
        for p in (0, 1):
            got = Z[p].cpu().numpy().view(np.uint64)
            assert np.array_equal(got, ref["Z"][p]), (call, p)
            assert np.array_equal(got, same[p]), (call, p)


def test_static_scratch_refuses_unaligned_pointers():
    """A pointer carved out of a pool at an odd word (8 but not 16 bytes aligned) is refused on the host."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import ctypes

    from paper_2505_07239_b200 import binding as cb

    T, K, N = 8, 16, 8
    pool = torch.zeros(4096, dtype=torch.int64, device="cuda")
    base = pool.data_ptr()
    assert base % 16 == 0
    pair = ctypes.c_void_p * 2
    good = [pair(base + 2048 * (2 * k), base + 2048 * (2 * k + 1)) for k in range(6)]    # 256-word slots
    lib = cb.library()
    assert lib.comet_beaver_matmul_static(None, *good, T, K, N) == cb.OK
    for k in range(6):
        for party in (0, 1):
            args = list(good)
            odd = [good[k][0], good[k][1]]
            odd[party] += 8
            args[k] = pair(*odd)
            assert lib.comet_beaver_matmul_static(None, *args, T, K, N) == -1, (k, party)
    torch.cuda.synchronize()
    assert not pool[12 * 256:].any()         # nothing was written beyond the operands of the accepted call


def test_static_scratch_limit_is_refused_cleanly():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb

    T, K, N = 512, 1024, 64          # 2*(T*K + N*K) = 1 179 648 words > 2^20
    assert 2 * (T * K + N * K) > cb.STATIC_SCRATCH_WORDS
    mk = lambda r, c: [torch.zeros((r, c), dtype=torch.int64, device="cuda") for _ in (0, 1)]  # noqa: E731
    Z = mk(T, N)
    code = cb.beaver_matmul_static(mk(T, K), mk(T, K), mk(N, K), mk(N, K), mk(T, N), Z)
    assert code == cb.ERR_SCRATCH_LIMIT
    assert b"static scratch" in cb.library().comet_strerror(code)
    # null share pointers and bad shapes are refused too, and nothing was launched
    import ctypes

    null = (ctypes.c_void_p * 2)(None, None)
    assert cb.library().comet_beaver_matmul_static(None, null, null, null, null, null, null, 1, 8, 4) == -1
    small = mk(8, 12)
    ok = (ctypes.c_void_p * 2)(small[0].data_ptr(), small[1].data_ptr())
    assert cb.library().comet_beaver_matmul_static(None, ok, ok, ok, ok, ok, ok, 8, 12, 4) == -2     # K % 8
    torch.cuda.synchronize()
