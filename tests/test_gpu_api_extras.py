"""GPU tests of the entry points around the path: the two ways a block mask reaches the compaction kernel, the
in-place view of a result buffer, and the probe of the multiply pipes."""
import ctypes

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2505_07239_b200 import workloads as wl  # noqa: E402


def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")


@pytest.mark.parametrize("n_blocks", [96, 3584, 3600, 8192])
def test_host_and_device_masks_compact_to_the_same_index_list(n_blocks):
    """A HOST mask is counted on the host and travels in the kernel's parameter block (up to 3584 blocks) or through
    a pinned staging slot (beyond); a DEVICE mask is read in place and its count comes back through mapped memory.
    All three must give the oracle's index set."""
    _need_gpu()
    from paper_2505_07239_b200 import binding as cb

    block, d = 16, 16
    ctx = cb.Comet(4, d, n_blocks * block, block, 12, False, 0, 0, cb.PATH_LIMB)
    rng = np.random.default_rng(n_blocks)
    for trial in range(6):          # more calls than staging slots
        mask = (rng.random(n_blocks) < 0.3).astype(np.uint8)
        if trial == 0:
            mask[:] = 0
        if trial == 1:
            mask[:] = 1
        want = oracle.index_set(mask, block, 1)
        for where in ("host", "device"):
            m = mask.copy() if where == "host" else torch.from_numpy(mask).cuda()
            n = ctx.set_mask(m)
            if where == "host":
                m[:] = 0xFF          # the caller's buffer is free again on return
            assert n == want.size
            ids = ctx.get_index()
            got = (ids[:, None] * block + np.arange(block)[None, :]).reshape(-1).astype(np.int32)
            assert np.array_equal(got, want), (n_blocks, trial, where)
    ctx.close()


def test_result_view_aliases_the_library_buffer():
    _need_gpu()
    from paper_2505_07239_b200 import binding as cb
    from tests import harness as hz

    cfg = wl.CONFIGS["tiny"]
    T, d = cfg.tokens, cfg.d_model
    ctx = hz.make_context(cfg, T)
    hz.load_weights(ctx, cfg, wl.model_shares(cfg, 3, plain=False))
    assert ctx.set_mask(np.zeros(cfg.n_blocks, np.uint8)) == 0
    C = [wl.random_u64(3, f"view/C{p}", T * d).reshape(T, d) for p in (0, 1)]
    for p in (0, 1):
        ctx.load_shares(p, cb.C_DN, cb.to_device(C[p]))
    ctx.ffn_down(T)                          # no active neuron: Y_i = 0
    views = [ctx.result_view(p, cb.Y, (T, d)) for p in (0, 1)]
    ctx.synchronize()
    for p in (0, 1):
        assert not views[p].any()
        views[p].add_(cb.to_device(C[p]))    # what an in-place all-reduce does: the library's buffer changes
    torch.cuda.synchronize()
    for p in (0, 1):
        assert np.array_equal(ctx.get(p, cb.Y, (T, d)), C[p])
    bad = ctypes.c_void_p()
    assert cb.library().comet_device_pointer(ctx._h, 0, cb.X, ctypes.byref(bad)) == -1     # results only
    assert cb.library().comet_device_pointer(ctx._h, 2, cb.Y, ctypes.byref(bad)) == -1
    ctx.close()


def test_pipe_probe_reports_plausible_rates():
    _need_gpu()
    from paper_2505_07239_b200 import binding as cb

    ms, macs = cb.pipe_probe(cb.PIPE_TENSOR_I8, 3, 400)
    assert len(ms) == 3 and all(m > 0 for m in ms)
    rate = macs / (min(ms) * 1e-3)
    assert 0.5e15 < rate < 3.0e15            # nominal 148 SMs x 8192 per clock x 1.965 GHz = 2.38e15
    ms, macs = cb.pipe_probe(cb.PIPE_ALU_U64, 2, 2000)
    rate = macs / (min(ms) * 1e-3)
    assert 1.0e12 < rate < 2.0e13
    lib = cb.library()
    out, m = (ctypes.c_float * 1)(), ctypes.c_double()
    assert lib.comet_pipe_probe(None, 7, 1, 1, out, ctypes.byref(m)) == -1
    assert lib.comet_pipe_probe(None, 0, 0, 1, out, ctypes.byref(m)) == -2
    assert lib.comet_pipe_probe(None, 0, 1, 1, None, ctypes.byref(m)) == -1
