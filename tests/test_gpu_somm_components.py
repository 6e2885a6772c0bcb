"""GPU parity of the up-projection under a per-token mask (Protocol 2 over connected components,
comet_set_token_mask + comet_ffn_up through the C ABI) against the CPU oracle, bit for bit."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2505_07239_b200 import workloads as wl  # noqa: E402


def _canonical(row_comp, col_comp):
    """Component ids -> smallest row index of the component (what the library reports)."""
    rc, cc = row_comp.astype(np.int64), col_comp.astype(np.int64)
    first = {}
    for r, t in enumerate(rc.tolist()):
        if t >= 0 and t not in first:
            first[t] = r
    f = np.vectorize(lambda t: first[t] if t >= 0 else -1, otypes=[np.int64])
    return f(rc), f(cc)


_LAST = {}


def _run(cfg, seed, tokens, sparsity, path, p_token=None, token_mask=None):
    from paper_2505_07239_b200 import binding as cb
    from tests import harness as hz

    T, d, f, g, bs = tokens, cfg.d_model, cfg.frac_bits, cfg.groups, cfg.block
    W = wl.model_shares(cfg, seed, plain=False)
    mask = wl.block_mask(cfg, seed, sparsity)
    Ig = oracle.index_set(mask, bs, g)
    n, nab = Ig.size // g, int(mask.sum())
    tm = token_mask if token_mask is not None else wl.token_block_masks(seed, "tm", T, nab, p_token)
    S = np.tile(np.repeat(tm, bs, axis=1), (1, g))                # [T, g*n]: gate and up columns share the mask
    _, X0, X1 = wl.activation_shares(cfg, seed, tokens=T)
    tri = wl.dealer_triple_components(seed, "up", S, d)
    Wup = (hz.oracle_up_operand(cfg, W, 1), hz.oracle_up_operand(cfg, W, 2))
    ref = oracle.somm_components((X0, X1), Wup, Ig, S, tri["A"][1:], tri["B"][1:], tri["C"][1:])

    ctx = hz.make_context(cfg, T, path)
    hz.load_weights(ctx, cfg, W)
    for p, Xs in ((0, X0), (1, X1)):
        ctx.load_shares(p, cb.X, cb.to_device(Xs))
    assert ctx.set_mask(mask) == n
    ctx.set_token_mask(tm)
    hz.load_triple_up(ctx, tri)
    ctx.ffn_up(T)
    st = ctx.stats()
    assert st.matmul_path == path and st.n_components == ref["L"]
    _LAST.update(ring_macs=st.ring_macs, tile_macs=st.tensor_tile_macs, dot_products=ref["dot_products"],
                 dense_tile_macs=2 * 2 * (-(-T // 128) * 128) * (-(-(g * n) // 64) * 64) * (-(-d // 32) * 32), d=d)
    rl, bl, L = ctx.get_components(T, nab)
    want_r, want_c = _canonical(ref["row_comp"], ref["col_comp"][:n])
    assert L == ref["L"] and np.array_equal(rl, want_r) and np.array_equal(np.repeat(bl, bs), want_c)
    live_rows, live_cols = int((rl >= 0).sum()), int((bl >= 0).sum()) * bs * g
    assert live_rows + live_cols == ref["masked_nodes"]
    assert st.message_bytes == 2 * 8 * (live_rows * d + live_cols * d)      # Theorem 1: each row / column once
    bad = 0
    for p in (0, 1):
        bad += int((ctx.get(p, cb.E_UP, (T, d)) != ref["E"][p]).sum())
        bad += int((ctx.get(p, cb.F_UP, (g * n, d)).T != ref["F"][p]).sum())
        bad += int((ctx.get(p, cb.Z_UP, (T, g * n)) != ref["Z"][p]).sum())
    ctx.truncate(cb.Z_UP)
    for p in (0, 1):
        bad += int((ctx.get(p, cb.Z_UP, (T, g * n)) != oracle.truncate(p, ref["Z"][p], f)).sum())
    ctx.close()
    return bad, ref["L"]


@pytest.mark.parametrize("path", [1, 2])
@pytest.mark.parametrize("tokens", [16, 40, 130])
def test_component_partitioned_up_projection_small(path, tokens):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("comp-small", tokens, 128, 512, 32, 16, False, 0.5, "uniform", "normal", "normal0.02")
    bad, L = _run(cfg, 81 + tokens, tokens, 0.5, path, p_token=0.12)
    assert bad == 0 and L >= 1


@pytest.mark.parametrize("path", [1, 2])
def test_component_partitioned_up_projection_gated(path):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("comp-gated", 48, 128, 1024, 64, 16, True, 0.5, "uniform", "normal", "normal0.02")
    bad, _ = _run(cfg, 91, 48, 0.5, path, p_token=0.1)
    assert bad == 0


def test_several_components_dead_token_and_dead_block():
    """Hand-made distribution: two components, one token without any block, one active block without any token."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("comp-hand", 8, 128, 256, 32, 16, False, 0.5, "uniform", "normal", "normal0.02")
    tm = np.zeros((8, 4), np.uint8)
    tm[0:3, 0] = 1
    tm[2, 1] = 1              # tokens 0-2 with blocks 0-1
    tm[4:8, 3] = 1            # tokens 4-7 with block 3; token 3 and block 2 have no edge
    for path in (1, 2):
        bad, L = _run(cfg, 95, 8, 0.5, path, token_mask=tm)
        assert bad == 0 and L == 2


def test_opt125m_one_giant_component():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    bad, L = _run(wl.CONFIGS["opt125m"], 97, 128, None, 2, p_token=0.3)
    assert bad == 0 and L == 1


# ---- one multiplication per component on the tensor-core path (more than 32 tokens): component-sorted operands,
#      only the tiles that meet a component are computed, results scattered back to the compact layout

def _clustered(cfg, seed, tokens, sparsity, clusters, p, dead_tokens=0, dead_blocks=0):
    mask = wl.block_mask(cfg, seed, sparsity)
    return wl.token_block_masks_clustered(seed, "tmc", tokens, int(mask.sum()), clusters, p, dead_tokens, dead_blocks)


@pytest.mark.parametrize("tokens,block,clusters,dead", [(200, 32, 4, 2), (130, 16, 3, 0), (300, 64, 6, 3), (33, 32, 2, 1)])
def test_grouped_launch_scattered_components(tokens, block, clusters, dead):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("comp-grouped", tokens, 128, 2048, block, 16, False, 0.5, "uniform", "normal", "normal0.02")
    tm = _clustered(cfg, 300 + tokens, tokens, 0.5, clusters, 0.3, dead, dead)
    bad, L = _run(cfg, 300 + tokens, tokens, 0.5, 2, token_mask=tm)
    assert bad == 0 and L >= clusters
    assert _LAST["ring_macs"] == 2 * 2 * _LAST["d"] * _LAST["dot_products"]      # Theorem 1: one product per component
    assert 0 < _LAST["tile_macs"] <= _LAST["dense_tile_macs"]
    if tokens > 128:                                                               # several row tiles: fewer tiles
        assert _LAST["tile_macs"] < _LAST["dense_tile_macs"]                       # than the union needs


def test_grouped_launch_token_mask_too_large_for_shared_memory():
    """1400 tokens x 256 active blocks: the planning kernel's bit matrix and labels (52 KB) work in global memory."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("comp-large-mask", 1400, 128, 8192, 16, 16, False, 0.5, "uniform", "normal", "normal0.02")
    tm = _clustered(cfg, 431, 1400, 0.5, 5, 0.05, 3, 2)
    bad, L = _run(cfg, 431, 1400, 0.5, 2, token_mask=tm)
    assert bad == 0 and L >= 5
    assert _LAST["ring_macs"] == 2 * 2 * _LAST["d"] * _LAST["dot_products"]
    assert 0 < _LAST["tile_macs"] < _LAST["dense_tile_macs"]


def test_token_mask_without_any_entry_and_with_a_single_one():
    """Degenerate distributions on the tensor-core path with more than 32 tokens: no entry at all (nothing is opened,
    every result share is zero) and a single (token, block) entry."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("comp-degenerate", 140, 128, 512, 32, 16, False, 0.5, "uniform", "normal", "normal0.02")
    nab = int(wl.block_mask(cfg, 88, 0.5).sum())
    tm = np.zeros((140, nab), np.uint8)
    bad, L = _run(cfg, 88, 140, 0.5, 2, token_mask=tm)
    assert bad == 0 and L == 0 and _LAST["ring_macs"] == 0
    tm[137, nab - 1] = 1
    bad, L = _run(cfg, 88, 140, 0.5, 2, token_mask=tm)
    assert bad == 0 and L == 1 and _LAST["ring_macs"] == 2 * 2 * 128 * 32
    assert _LAST["tile_macs"] == 2 * 2 * 128 * 64 * 128            # one output tile per party and operand pair


@pytest.mark.parametrize("live", [127, 128, 129])
def test_grouped_launch_row_tile_boundaries(live):
    """Exactly 127 / 128 / 129 tokens lie in a component (of 200): the sorted rows fill one tile, or one and one row."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("comp-boundary", 200, 128, 1024, 32, 16, False, 0.5, "uniform", "normal", "normal0.02")
    nab = int(wl.block_mask(cfg, 90 + live, 0.5).sum())
    tm = wl.token_block_masks_clustered(90 + live, "tmc", 200, nab, 3, 0.4)
    order = np.argsort(wl.random_u64(90 + live, "kill", 200), kind="stable")
    tm[order[:200 - live], :] = 0
    tm[:, tm.sum(axis=0) == 0] = 0
    rows_alive = int((tm.sum(axis=1) > 0).sum())
    assert rows_alive == live
    bad, L = _run(cfg, 90 + live, 200, 0.5, 2, token_mask=tm)
    assert bad == 0 and L >= 1


def test_grouped_launch_gated_two_matrices():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("comp-grouped-gated", 260, 128, 2048, 64, 16, True, 0.5, "uniform", "normal", "normal0.02")
    tm = _clustered(cfg, 411, 260, 0.5, 4, 0.4, 1, 1)
    bad, L = _run(cfg, 411, 260, 0.5, 2, token_mask=tm)
    assert bad == 0 and L >= 4
    assert _LAST["ring_macs"] == 2 * 2 * _LAST["d"] * _LAST["dot_products"]
    assert 0 < _LAST["tile_macs"] < _LAST["dense_tile_macs"]


def test_grouped_launch_contiguous_components_and_single_rows():
    """Hand-made: components that are already contiguous, one of a single token and a single block, tokens and
    blocks in no component between them."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("comp-hand-grouped", 140, 128, 512, 32, 16, False, 0.5, "uniform", "normal", "normal0.02")
    nab = int(wl.block_mask(cfg, 77, 0.5).sum())
    assert nab == 8
    tm = np.zeros((140, nab), np.uint8)
    tm[0:60, 0:3] = 1
    tm[60, 5] = 1                       # a component of one token and one block
    tm[70:139, 6:8] = 1                 # tokens 61-69 and 139, blocks 3-4 in no component
    bad, L = _run(cfg, 77, 140, 0.5, 2, token_mask=tm)
    assert bad == 0 and L == 3
    assert _LAST["ring_macs"] == 2 * 2 * 128 * (60 * 96 + 1 * 32 + 69 * 64)


def test_grouped_launch_opt13b_at_90_percent():
    """The graded FFN shape (512 tokens, d = 2048, 26 of 256 blocks active) with the batch split into four groups
    of requests: full comparison against the oracle."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.CONFIGS["opt1.3b"]
    tm = _clustered(cfg, 555, 512, 0.9, 4, 0.6)
    bad, L = _run(cfg, 555, 512, 0.9, 2, token_mask=tm)
    assert bad == 0 and L >= 4
    assert _LAST["ring_macs"] == 2 * 2 * _LAST["d"] * _LAST["dot_products"]
    assert _LAST["tile_macs"] < _LAST["dense_tile_macs"]


def test_grouped_chain_up_then_down_with_three_stacked_matrices():
    """Both products of one layer under one clustered token mask, the down-projection's weight side opened early
    (on the side stream, in component order) during the up-projection: three stacked matrices, then the
    row-gathered product, each against the oracle."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb
    from tests import harness as hz

    cfg = wl.FFNConfig("comp-chain", 150, 256, 1024, 64, 16, False, 0.5, "uniform", "normal", "normal0.02", stacked=3)
    seed, T, d, g, bs = 620, 150, cfg.d_model, cfg.groups, cfg.block
    W = wl.model_shares(cfg, seed, plain=False)
    mask = wl.block_mask(cfg, seed, 0.5)
    I1, Ig = oracle.index_set(mask, bs, 1), oracle.index_set(mask, bs, g)
    n, nab = I1.size, int(mask.sum())
    tm = wl.token_block_masks_clustered(seed, "tmc", T, nab, 3, 0.5, 2, 1)
    S1 = np.repeat(tm, bs, axis=1)
    Sg = np.tile(S1, (1, g))
    _, X0, X1 = wl.activation_shares(cfg, seed, tokens=T)
    tri = wl.dealer_triple_components(seed, "up", Sg, d)
    trd = wl.dealer_triple_rowsets(seed, "down", S1, d)
    _, H0, H1 = wl.hidden_shares(cfg, seed, n, tokens=T)
    Wup = (hz.oracle_up_operand(cfg, W, 1), hz.oracle_up_operand(cfg, W, 2))
    ref = oracle.somm_components((X0, X1), Wup, Ig, Sg, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    refd = oracle.simm_rowsets((H0, H1), W["W2"][1:], I1, S1, trd["A"][1:], trd["B"][1:], trd["C"][1:])

    ctx = hz.make_context(cfg, T, 2)
    hz.load_weights(ctx, cfg, W)
    for p, Xs in ((0, X0), (1, X1)):
        ctx.load_shares(p, cb.X, cb.to_device(Xs))
    assert ctx.set_mask(mask) == n
    ctx.set_token_mask(tm)
    hz.load_triple_up(ctx, tri)
    hz.load_triple_down(ctx, trd)                 # B' is there before ffn_up: the weight side is opened early
    ctx.ffn_up(T)
    assert ctx.stats().n_components == ref["L"] >= 3
    bad = 0
    for p in (0, 1):
        bad += int((ctx.get(p, cb.Z_UP, (T, g * n)) != ref["Z"][p]).sum())
        bad += int((ctx.get(p, cb.F_UP, (g * n, d)).T != ref["F"][p]).sum())
    for p, Hs in ((0, H0), (1, H1)):
        ctx.load_shares(p, cb.H, cb.to_device(Hs))
    ctx.ffn_down(T)
    for p in (0, 1):
        bad += int((ctx.get(p, cb.Y, (T, d)) != refd["Z"][p]).sum())
        bad += int((ctx.get(p, cb.E_DN, (T, n)) != refd["E"][p]).sum())
        bad += int((ctx.get(p, cb.F_DN, (d, n)).T != refd["F"][p]).sum())
    ctx.close()
    assert bad == 0


def test_one_context_through_grouped_cleared_and_regrouped_masks():
    """State carried by a context across calls: a clustered token mask (grouped launches, the down-projection's
    weight side opened early in component order), the mask cleared (products over the union again), a token mask
    with one component, then a new block mask with another clustered token mask.  Every product is compared with
    the oracle, so nothing of an earlier plan may leak into a later call."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb
    from tests import harness as hz

    cfg = wl.FFNConfig("comp-states", 160, 128, 1024, 32, 16, False, 0.5, "uniform", "normal", "normal0.02")
    T, d, bs = 160, cfg.d_model, cfg.block
    seed = 700
    W = wl.model_shares(cfg, seed, plain=False)
    Wup = (hz.oracle_up_operand(cfg, W, 1), hz.oracle_up_operand(cfg, W, 2))
    ctx = hz.make_context(cfg, T, 2)
    hz.load_weights(ctx, cfg, W)
    bad = 0

    def both(step, mask, tm):
        """One up- and one down-projection under (mask, tm); tm None = no token mask."""
        nonlocal bad
        I = oracle.index_set(mask, bs, 1)
        n, nab = I.size, int(mask.sum())
        _, X0, X1 = wl.activation_shares(cfg, seed, step=step, tokens=T)
        _, H0, H1 = wl.hidden_shares(cfg, seed, n, step=step, tokens=T)
        assert ctx.set_mask(mask) == n
        if tm is None:
            tri = wl.dealer_triple(seed, f"up/{step}", T, d, n, valid=False)
            trd = wl.dealer_triple(seed, f"dn/{step}", T, n, d, valid=False)
            ref = oracle.somm((X0, X1), Wup, I, tri["A"][1:], tri["B"][1:], tri["C"][1:])
            refd = oracle.simm((H0, H1), W["W2"][1:], I, trd["A"][1:], trd["B"][1:], trd["C"][1:])
        else:
            S = np.repeat(tm, bs, axis=1)
            tri = wl.dealer_triple_components(seed, f"up/{step}", S, d)
            trd = wl.dealer_triple_rowsets(seed, f"dn/{step}", S, d)
            ref = oracle.somm_components((X0, X1), Wup, I, S, tri["A"][1:], tri["B"][1:], tri["C"][1:])
            refd = oracle.simm_rowsets((H0, H1), W["W2"][1:], I, S, trd["A"][1:], trd["B"][1:], trd["C"][1:])
            ctx.set_token_mask(tm)
        for p, Xs in ((0, X0), (1, X1)):
            ctx.load_shares(p, cb.X, cb.to_device(Xs))
        hz.load_triple_up(ctx, tri)
        hz.load_triple_down(ctx, trd)
        ctx.ffn_up(T)
        for p, Hs in ((0, H0), (1, H1)):
            ctx.load_shares(p, cb.H, cb.to_device(Hs))
        ctx.ffn_down(T)
        for p in (0, 1):
            bad += int((ctx.get(p, cb.Z_UP, (T, n)) != ref["Z"][p]).sum())
            bad += int((ctx.get(p, cb.F_UP, (n, d)).T != ref["F"][p]).sum())
            bad += int((ctx.get(p, cb.Y, (T, d)) != refd["Z"][p]).sum())
            bad += int((ctx.get(p, cb.F_DN, (d, n)).T != refd["F"][p]).sum())
            bad += int((ctx.get(p, cb.E_DN, (T, n)) != refd["E"][p]).sum())
        return nab

    m1 = wl.block_mask(cfg, seed, 0.5, 0)
    nab = int(m1.sum())
    both(0, m1, wl.token_block_masks_clustered(seed, "a", T, nab, 4, 0.5, 2, 1))     # grouped
    assert ctx.stats().n_components >= 4
    assert ctx.set_token_mask(None) == 0
    both(1, m1, None)                                                                 # union, same block mask
    both(2, m1, wl.token_block_masks(seed, "b", T, nab, 0.5))                         # one component: not grouped
    m2 = wl.block_mask(cfg, seed, 0.75, 1)
    both(3, m2, wl.token_block_masks_clustered(seed, "c", T, int(m2.sum()), 3, 0.6))  # new block mask, grouped again
    both(4, m2, None)                                                                 # set_mask alone drops the token mask
    ctx.close()
    assert bad == 0
