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
