"""Second workload of the same kernels: the projections of an attention layer under a head mask (Section 3.3:
sparse QKV is SOMM, the sparse output projection is SIMM).  block = head size, d_ff = heads * head size, three
stacked weight matrices [Wq || Wk || Wv] share the mask and X is opened once; the output projection is the
row-gathered product.  GPU (through the C ABI) against the CPU oracle, bit for bit."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2505_07239_b200 import workloads as wl  # noqa: E402


def _run(cfg, seed, path):
    from paper_2505_07239_b200 import binding as cb
    from tests import harness as hz

    T, d, f, g = cfg.tokens, cfg.d_model, cfg.frac_bits, cfg.groups
    assert g == 3
    W = wl.model_shares(cfg, seed)
    Xr, X0, X1 = wl.activation_shares(cfg, seed)
    mask = wl.block_mask(cfg, seed)                       # active heads
    ctx = hz.make_context(cfg, T, path)
    hz.load_weights(ctx, cfg, W)
    for p, Xs in ((0, X0), (1, X1)):
        ctx.load_shares(p, cb.X, cb.to_device(Xs))
    n = ctx.set_mask(mask)
    I1, Ig = oracle.index_set(mask, cfg.block, 1), oracle.index_set(mask, cfg.block, g)
    tri = wl.dealer_triple(seed, "qkv", T, d, g * n)
    hz.load_triple_up(ctx, tri)
    ctx.ffn_up(T)
    assert ctx.stats().matmul_path == path
    Wup = (hz.oracle_up_operand(cfg, W, 1), hz.oracle_up_operand(cfg, W, 2))
    ref = oracle.somm((X0, X1), Wup, Ig, tri["A"][1:], tri["B"][1:], tri["C"][1:])
    bad = 0
    Z = []
    for p in (0, 1):
        bad += int((ctx.get(p, cb.E_UP, (T, d)) != ref["E"][p]).sum())
        bad += int((ctx.get(p, cb.F_UP, (g * n, d)).T != ref["F"][p]).sum())
        Z.append(ctx.get(p, cb.Z_UP, (T, g * n)))
        bad += int((Z[p] != ref["Z"][p]).sum())
    # Q, K, V of the active heads reconstruct exactly
    Wfull = hz.oracle_up_operand(cfg, W, 0)
    assert np.array_equal(Z[0] + Z[1], wl.ring_matmul(Xr, Wfull[:, Ig]))
    ctx.truncate(cb.Z_UP)
    for p in (0, 1):
        bad += int((ctx.get(p, cb.Z_UP, (T, g * n)) != oracle.truncate(p, ref["Z"][p], f)).sum())
    # output projection over the active heads (the attention itself is outside this path: synthetic context vectors)
    _, H0, H1 = wl.hidden_shares(cfg, seed, n)
    for p, Hs in ((0, H0), (1, H1)):
        ctx.load_shares(p, cb.H, cb.to_device(Hs))
    trd = wl.dealer_triple(seed, "out", T, n, d)
    hz.load_triple_down(ctx, trd)
    ctx.ffn_down(T)
    refd = oracle.simm((H0, H1), W["W2"][1:], I1, trd["A"][1:], trd["B"][1:], trd["C"][1:])
    for p in (0, 1):
        bad += int((ctx.get(p, cb.Y, (T, d)) != refd["Z"][p]).sum())
        bad += int((ctx.get(p, cb.F_DN, (d, n)).T != refd["F"][p]).sum())
    ctx.close()
    return bad, n


@pytest.mark.parametrize("path", [1, 2])
def test_qkv_and_output_projection_under_a_head_mask(path):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    # 8 heads of 64, half of them active (the paper reports about half of the heads inactive)
    cfg = wl.FFNConfig("mha-small", 72, 512, 512, 64, 16, False, 0.5, "uniform", "normal", "normal0.02", stacked=3)
    bad, n = _run(cfg, 101, path)
    assert bad == 0 and n == 4 * 64


def test_qkv_few_tokens_and_head_size_128():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cfg = wl.FFNConfig("mha-decode", 8, 1024, 1024, 128, 16, False, 0.5, "uniform", "normal", "normal0.02", stacked=3)
    bad, n = _run(cfg, 103, 2)
    assert bad == 0 and n == 4 * 128


def test_third_matrix_is_refused_without_three_groups():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_07239_b200 import binding as cb
    from tests import harness as hz

    cfg = wl.CONFIGS["tiny"]
    ctx = hz.make_context(cfg, cfg.tokens)
    buf = torch.zeros(cfg.d_ff * cfg.d_model, dtype=torch.int64, device="cuda")
    assert cb.library().comet_load_shares(ctx._h, 0, cb.W3, buf.data_ptr(), 0, cfg.d_ff, cfg.d_model) == -1
    ctx.close()
