"""GPU parity of the down-projection under a per-token mask (Protocol 3 with per-column row sets R_j,
comet_set_token_mask + comet_ffn_down through the C ABI) against the CPU oracle, bit for bit."""
import ctypes

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2505_07239_b200 import workloads as wl  # noqa: E402


_LAST = {}


def _run(cfg, seed, tokens, sparsity, p_token, path, clear_after=False, token_mask=None):
    from paper_2505_07239_b200 import binding as cb
    from tests import harness as hz

    T, d, f = tokens, cfg.d_model, cfg.frac_bits
    W = wl.model_shares(cfg, seed, plain=False)
    mask = wl.block_mask(cfg, seed, sparsity)
    I = oracle.index_set(mask, cfg.block, 1)
    n, nab = I.size, int(mask.sum())
    tm = token_mask if token_mask is not None else wl.token_block_masks(seed, "tm", T, nab, p_token)
    S = np.repeat(tm, cfg.block, axis=1)                       # element-level distribution over the compact columns
    _, H0, H1 = wl.hidden_shares(cfg, seed, n, tokens=T)       # uniform words everywhere, also off the support
    tri = wl.dealer_triple_rowsets(seed, "down", S, d)

    ctx = hz.make_context(cfg, T, path)
    hz.load_weights(ctx, cfg, W)
    assert ctx.set_mask(mask) == n
    masked = ctx.set_token_mask(tm)
    assert masked == int(S.sum())
    for p, Hs in ((0, H0), (1, H1)):
        ctx.load_shares(p, cb.H, cb.to_device(Hs))
    hz.load_triple_down(ctx, tri)
    ctx.ffn_down(T)
    st = ctx.stats()
    assert st.matmul_path == path
    used = int((tm.sum(axis=0) > 0).sum()) * cfg.block         # columns of X with a non-zero
    assert st.message_bytes == 2 * 8 * (masked + used * d)     # only the non-zeros of X and those rows of Y are sent
    assert st.ring_macs == 2 * 2 * masked * d                  # Theorem 2: one row of Y per non-zero of X
    _LAST.update(tile_macs=st.tensor_tile_macs,
                 dense_tile_macs=2 * 2 * (-(-T // 128) * 128) * (-(-d // 64) * 64) * (-(-n // 32) * 32))
    ref = oracle.simm_rowsets((H0, H1), W["W2"][1:], I, S, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    assert ref["masked"] == masked
    bad = 0
    for p in (0, 1):
        bad += int((ctx.get(p, cb.E_DN, (T, n)) != ref["E"][p]).sum())
        bad += int((ctx.get(p, cb.F_DN, (d, n)).T != ref["F"][p]).sum())
        bad += int((ctx.get(p, cb.Y, (T, d)) != ref["Z"][p]).sum())
    ctx.truncate(cb.Y)
    for p in (0, 1):
        bad += int((ctx.get(p, cb.Y, (T, d)) != oracle.truncate(p, ref["Z"][p], f)).sum())
    if clear_after:
        # cleared: the next product is the token-shared one again
        assert ctx.set_token_mask(None) == 0
        full = wl.dealer_triple(seed, "down/full", T, n, d, valid=False)
        for p, Hs in ((0, H0), (1, H1)):
            ctx.load_shares(p, cb.H, cb.to_device(Hs))
        hz.load_triple_down(ctx, full)
        ctx.ffn_down(T)
        ref2 = oracle.simm((H0, H1), W["W2"][1:], I, full["A"][1:], full["B"][1:], full["C"][1:])
        for p in (0, 1):
            bad += int((ctx.get(p, cb.Y, (T, d)) != ref2["Z"][p]).sum())
            bad += int((ctx.get(p, cb.E_DN, (T, n)) != ref2["E"][p]).sum())
    ctx.close()
    return bad


@pytest.mark.parametrize("path", [1, 2])
@pytest.mark.parametrize("tokens", [16, 40, 130])          # few-token kernel, one ragged tile, two tiles
def test_token_masked_down_projection_small(path, tokens):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("rowsets-small", tokens, 128, 512, 32, 16, False, 0.5, "uniform", "normal", "normal0.02")
    assert _run(cfg, 61 + tokens, tokens, 0.5, 0.3, path, clear_after=True) == 0


@pytest.mark.parametrize("path", [1, 2])
def test_token_masked_down_projection_opt125m(path):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    assert _run(wl.CONFIGS["opt125m"], 71, 128, None, 0.25, path) == 0


def test_token_masked_down_projection_llama_shape_blocks_of_64():
    """Config 4's structure: 64-neuron blocks, block mask = union of sparse per-token masks."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("rowsets-b64", 96, 256, 2048, 64, 16, True, 0.25, "uniform", "normal", "normal0.02")
    assert _run(cfg, 73, 96, 0.75, 0.05, 2) == 0


# ---- per-column row sets that fall into several components (tensor-core path, more than 32 tokens): rows and the
#      contraction index are taken in component order and a row tile runs over its components' blocks only

@pytest.mark.parametrize("tokens,block,clusters,dead", [(200, 32, 4, 2), (130, 16, 3, 1), (300, 64, 6, 3), (40, 16, 5, 0)])
def test_grouped_down_projection_scattered_components(tokens, block, clusters, dead):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("rowsets-grouped", tokens, 128, 2048, block, 16, False, 0.5, "uniform", "normal", "normal0.02")
    nab = int(wl.block_mask(cfg, 500 + tokens, 0.5).sum())
    tm = wl.token_block_masks_clustered(500 + tokens, "tmc", tokens, nab, clusters, 0.3, dead, dead)
    assert _run(cfg, 500 + tokens, tokens, 0.5, None, 2, token_mask=tm, clear_after=True) == 0
    assert 0 < _LAST["tile_macs"] <= _LAST["dense_tile_macs"]
    if tokens > 128:                                            # several row tiles: each skips the others' blocks
        assert _LAST["tile_macs"] < _LAST["dense_tile_macs"]


def test_down_projection_token_mask_without_any_entry():
    """No non-zero in the hidden state at all: nothing is opened and Y_i = C'_i."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("rowsets-empty", 140, 128, 512, 32, 16, False, 0.5, "uniform", "normal", "normal0.02")
    nab = int(wl.block_mask(cfg, 89, 0.5).sum())
    for path in (1, 2):
        assert _run(cfg, 89, 140, 0.5, None, path, token_mask=np.zeros((140, nab), np.uint8)) == 0


def test_grouped_down_projection_token_mask_too_large_for_shared_memory():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("rowsets-large-mask", 1400, 128, 8192, 16, 16, False, 0.5, "uniform", "normal", "normal0.02")
    nab = int(wl.block_mask(cfg, 432, 0.5).sum())
    tm = wl.token_block_masks_clustered(432, "tmc", 1400, nab, 5, 0.05, 3, 2)
    assert _run(cfg, 432, 1400, 0.5, None, 2, token_mask=tm) == 0
    assert 0 < _LAST["tile_macs"] < _LAST["dense_tile_macs"]


def test_grouped_down_projection_opt13b_at_90_percent():
    """The graded FFN shape with the batch dealt to four groups of requests: full comparison against the oracle."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.CONFIGS["opt1.3b"]
    nab = int(wl.block_mask(cfg, 556, 0.9).sum())
    tm = wl.token_block_masks_clustered(556, "tmc", 512, nab, 4, 0.6)
    assert _run(cfg, 556, 512, 0.9, None, 2, token_mask=tm) == 0
    assert _LAST["tile_macs"] < _LAST["dense_tile_macs"]


@pytest.mark.parametrize("path", [1, 2])
@pytest.mark.parametrize("tokens", [12, 70])
def test_active_block_without_any_token_is_not_opened(path, tokens):
    """A block of the block mask that no token uses holds no non-zero column of X: its rows of the weight matrix
    are not masked and not sent (zero message words), on both paths and in the few-token kernel."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("rowsets-dead", tokens, 128, 512, 32, 16, False, 0.5, "uniform", "normal", "normal0.02")
    nab = int(wl.block_mask(cfg, 640, 0.5).sum())
    tm = wl.token_block_masks(640, "tm", tokens, nab, 0.4)
    tm[:, 2] = 0
    tm[:, nab - 1] = 0
    assert _run(cfg, 640, tokens, 0.5, None, path, token_mask=tm) == 0


def test_token_mask_errors():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb
    from tests import harness as hz

    cfg = wl.CONFIGS["tiny"]
    ctx = hz.make_context(cfg, cfg.tokens)
    lib, h = cb.library(), ctx._h
    m = torch.ones((cfg.tokens, 3), dtype=torch.uint8, device="cuda")
    out = ctypes.c_int64(0)
    assert lib.comet_set_token_mask(h, m.data_ptr(), 0, cfg.tokens, 3, ctypes.byref(out)) == -3     # no block mask yet
    assert ctx.set_mask(wl.block_mask(cfg, 1)) == 96
    assert lib.comet_set_token_mask(h, m.data_ptr(), 0, cfg.tokens, 4, ctypes.byref(out)) == -2     # 3 active blocks
    assert lib.comet_set_token_mask(h, m.data_ptr(), 0, cfg.tokens + 1, 3, ctypes.byref(out)) == -2
    assert lib.comet_set_token_mask(h, None, 0, 5, 3, ctypes.byref(out)) == -1
    assert lib.comet_set_token_mask(h, m.data_ptr(), 0, cfg.tokens, 3, ctypes.byref(out)) == 0
    assert out.value == cfg.tokens * 96
    ctx.close()


@pytest.mark.parametrize("tokens", [16, 70])
def test_token_mask_cleared_between_the_projections(tokens):
    """The up-projection runs under a token mask in which one active block is used by no token and, since W2 and
    B' are already loaded, opens the down-projection's weight side early with that block's rows zeroed; the mask
    is then cleared, so the down-projection is the token-shared one and must open those rows after all."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb
    from tests import harness as hz

    cfg = wl.FFNConfig("rowsets-clear", tokens, 128, 512, 32, 16, False, 0.5, "uniform", "normal", "normal0.02")
    seed, T, d = 910 + tokens, tokens, cfg.d_model
    W = wl.model_shares(cfg, seed, plain=False)
    mask = wl.block_mask(cfg, seed, 0.5)
    I = oracle.index_set(mask, cfg.block, 1)
    n, nab = I.size, int(mask.sum())
    tm = wl.token_block_masks(seed, "tm", T, nab, 0.4)
    tm[:, 1] = 0
    S = np.repeat(tm, cfg.block, axis=1)
    _, X0, X1 = wl.activation_shares(cfg, seed, tokens=T)
    _, H0, H1 = wl.hidden_shares(cfg, seed, n, tokens=T)
    tri = wl.dealer_triple_components(seed, "up", S, d)
    full = wl.dealer_triple(seed, "down/full", T, n, d, valid=False)

    ctx = hz.make_context(cfg, T, cb.PATH_LIMB)
    hz.load_weights(ctx, cfg, W)
    assert ctx.set_mask(mask) == n
    ctx.set_token_mask(tm)
    for p, Xs in ((0, X0), (1, X1)):
        ctx.load_shares(p, cb.X, cb.to_device(Xs))
    hz.load_triple_up(ctx, tri)
    hz.load_triple_down(ctx, full)                  # W2 and B' are there: the weight side is opened during ffn_up
    ctx.ffn_up(T)
    assert ctx.set_token_mask(None) == 0
    for p, Hs in ((0, H0), (1, H1)):
        ctx.load_shares(p, cb.H, cb.to_device(Hs))
    ctx.ffn_down(T)
    ref = oracle.simm((H0, H1), W["W2"][1:], I, full["A"][1:], full["B"][1:], full["C"][1:])
    bad = 0
    for p in (0, 1):
        bad += int((ctx.get(p, cb.E_DN, (T, n)) != ref["E"][p]).sum())
        bad += int((ctx.get(p, cb.F_DN, (d, n)).T != ref["F"][p]).sum())
        bad += int((ctx.get(p, cb.Y, (T, d)) != ref["Z"][p]).sum())
    ctx.close()
    assert bad == 0
