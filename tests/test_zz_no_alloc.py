"""The allocation-free Pi_MatMul entry point (comet_beaver_matmul_static).

It serves callers that cannot allocate device memory at call time (a process
whose framework already owns all GPU memory, or a serving loop that must not
stall in cudaMalloc), by keeping the product's message buffers in an array
inside the library.  Here it is called through the C ABI twice in a row and
compared, bit for bit, with the context-based path (comet_ffn_up under an
all-ones mask computes the same dense product).  Collected last on purpose.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from paper_2505_07239_b200 import workloads as wl  # noqa: E402


def _reference_via_context(cb, X, A, Y, B, C, T, K, N):
    """Z_i from the existing entry points: d_model = K, d_ff = N, every block active."""
    ctx = cb.Comet(T, K, N, 16, 12, False, 0, 0, cb.PATH_SIMT)
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


def test_static_scratch_matmul_matches_context_path_twice():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb

    # two different problems back to back: the second reuses (and fully overwrites) the first one's scratch
    for call, (T, K, N) in enumerate([(40, 64, 96), (130, 256, 208)]):
        def draw(name, shape):
            return [cb.to_device(wl.random_u64(77 + call, f"static/{name}/{p}", shape[0] * shape[1]).reshape(shape))
                    for p in (0, 1)]

        X, A = draw("X", (T, K)), draw("A", (T, K))
        Y, B = draw("Y", (N, K)), draw("B", (N, K))
        C = draw("C", (T, N))
        Z = [torch.full((T, N), -1, dtype=torch.int64, device="cuda") for _ in (0, 1)]
        assert cb.beaver_matmul_static(X, A, Y, B, C, Z) == cb.OK
        torch.cuda.synchronize()
        want = _reference_via_context(cb, X, A, Y, B, C, T, K, N)
        for p in (0, 1):
            got = Z[p].cpu().numpy().view(np.uint64)
            assert np.array_equal(got, want[p]), (call, p)


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
