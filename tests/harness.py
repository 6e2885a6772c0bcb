"""Test harness: drives the CUDA library through its C ABI and the CPU oracle on
the same seeded inputs, and compares every exported buffer bit for bit.

The oracle never sees anything the GPU produced: the hidden state fed to the
down-projection is derived from the ORACLE's up-projection, and the GPU is
handed the same shares.
"""
from __future__ import annotations

import numpy as np

import oracle
from oracle import functionality
from paper_2505_07239_b200 import binding as cb
from paper_2505_07239_b200 import workloads as wl

U64 = np.uint64


def _mismatch(name, got, want, report):
    bad = int((got != want).sum())
    report["compared"].append((name, int(got.size), bad))
    report["mismatches"] += bad


def make_context(cfg, tokens, matmul_path=cb.PATH_AUTO, max_active=0):
    return cb.Comet(tokens, cfg.d_model, cfg.d_ff, cfg.block, cfg.frac_bits, cfg.groups - 1, 0, max_active, matmul_path)


def load_weights(ctx, cfg, W):
    for party in (0, 1):
        ctx.load_shares(party, cb.W1, cb.to_device(wl.lib_layout(W["W1"][1 + party])))
        ctx.load_shares(party, cb.W2, cb.to_device(wl.lib_layout(W["W2"][1 + party])))
        if cfg.groups >= 2:
            ctx.load_shares(party, cb.WG, cb.to_device(wl.lib_layout(W["WG"][1 + party])))
        if cfg.groups == 3:
            ctx.load_shares(party, cb.W3, cb.to_device(wl.lib_layout(W["W3"][1 + party])))


def oracle_up_operand(cfg, W, party_slot):
    """The paper-shaped right operand of the up product: W1, [WG || W1] when gated, [WG || W1 || W3] for three
    stacked matrices."""
    if cfg.groups == 3:
        return np.concatenate([W["WG"][party_slot], W["W1"][party_slot], W["W3"][party_slot]], axis=1)
    if cfg.groups == 2:
        return np.concatenate([W["WG"][party_slot], W["W1"][party_slot]], axis=1)
    return W["W1"][party_slot]


def load_triple_up(ctx, tri):
    for party in (0, 1):
        ctx.load_shares(party, cb.A_UP, cb.to_device(tri["A"][1 + party]))
        ctx.load_shares(party, cb.B_UP, cb.to_device(wl.lib_layout(tri["B"][1 + party])))
        ctx.load_shares(party, cb.C_UP, cb.to_device(tri["C"][1 + party]))


def load_triple_down(ctx, tri):
    for party in (0, 1):
        ctx.load_shares(party, cb.A_DN, cb.to_device(tri["A"][1 + party]))
        ctx.load_shares(party, cb.B_DN, cb.to_device(wl.lib_layout(tri["B"][1 + party])))
        ctx.load_shares(party, cb.C_DN, cb.to_device(tri["C"][1 + party]))


def run_and_compare_full(cfg, seed, sparsity=None, tokens=None, step=0, matmul_path=cb.PATH_AUTO,
                         mask=None, float_report=True):
    """Whole FFN (set_mask, ffn_up, truncate, activation functionality, ffn_down,
    truncate) on the GPU and in the oracle; every buffer compared exactly."""
    T = cfg.tokens if tokens is None else tokens
    d, D, f, g = cfg.d_model, cfg.d_ff, cfg.frac_bits, cfg.groups
    report = {"config": cfg.name, "tokens": T, "compared": [], "mismatches": 0}
    W = wl.model_shares(cfg, seed)
    Xr, X0, X1 = wl.activation_shares(cfg, seed, step=step, tokens=T)
    if mask is None:
        mask = wl.block_mask(cfg, seed, sparsity, step)

    ctx = make_context(cfg, T, matmul_path)
    load_weights(ctx, cfg, W)
    for party, Xs in ((0, X0), (1, X1)):
        ctx.load_shares(party, cb.X, cb.to_device(Xs))
    n = ctx.set_mask(mask)
    I1 = oracle.index_set(mask, cfg.block, 1)
    Ig = oracle.index_set(mask, cfg.block, g)
    report["n_active"] = n
    assert n == I1.size, (n, I1.size)
    ids = ctx.get_index()
    _mismatch("index", (ids[:, None] * cfg.block + np.arange(cfg.block)[None, :]).reshape(-1).astype(np.int32),
              I1, report)

    # ---- up projection (Protocol 2)
    tri = wl.dealer_triple(seed, f"{cfg.name}/up/step{step}", T, d, g * n)
    load_triple_up(ctx, tri)
    ctx.ffn_up(T)
    st = ctx.stats()
    report["path"] = st.matmul_path
    assert st.message_bytes == 2 * 8 * (T * d + d * g * n)
    ref = oracle.somm((X0, X1), (oracle_up_operand(cfg, W, 1), oracle_up_operand(cfg, W, 2)), Ig,
                      tri["A"][1:], tri["B"][1:], tri["C"][1:])
    Zg = []
    for party in (0, 1):
        _mismatch(f"E_up[{party}]", ctx.get(party, cb.E_UP, (T, d)), ref["E"][party], report)
        _mismatch(f"F_up[{party}]", ctx.get(party, cb.F_UP, (g * n, d)).T, ref["F"][party], report)
        Zg.append(ctx.get(party, cb.Z_UP, (T, g * n)))
        _mismatch(f"Z_up[{party}]", Zg[party], ref["Z"][party], report)
    ctx.truncate(cb.Z_UP)
    Hpre = [oracle.truncate(party, ref["Z"][party], f) for party in (0, 1)]
    Hgpu = [ctx.get(party, cb.Z_UP, (T, g * n)) for party in (0, 1)]
    for party in (0, 1):
        _mismatch(f"trunc(Z_up)[{party}]", Hgpu[party], Hpre[party], report)

    # ---- activation functionality on the oracle's values, re-shared
    act = functionality.activation(Hpre[0], Hpre[1], cfg.gated, f)
    H0, H1 = wl.reshare(act, seed, f"{cfg.name}/act/step{step}")
    for party, Hs in ((0, H0), (1, H1)):
        ctx.load_shares(party, cb.H, cb.to_device(Hs))

    # ---- down projection (Protocol 3)
    trd = wl.dealer_triple(seed, f"{cfg.name}/down/step{step}", T, n, d)
    load_triple_down(ctx, trd)
    ctx.ffn_down(T)
    refd = oracle.simm((H0, H1), W["W2"][1:], I1, trd["A"][1:], trd["B"][1:], trd["C"][1:])
    for party in (0, 1):
        _mismatch(f"E_dn[{party}]", ctx.get(party, cb.E_DN, (T, n)), refd["E"][party], report)
        _mismatch(f"F_dn[{party}]", ctx.get(party, cb.F_DN, (d, n)).T, refd["F"][party], report)
        _mismatch(f"Y[{party}]", ctx.get(party, cb.Y, (T, d)), refd["Z"][party], report)
    ctx.truncate(cb.Y)
    O = [oracle.truncate(party, refd["Z"][party], f) for party in (0, 1)]
    Og = [ctx.get(party, cb.Y, (T, d)) for party in (0, 1)]
    for party in (0, 1):
        _mismatch(f"trunc(Y)[{party}]", Og[party], O[party], report)

    # ---- reconstruction identities on the GPU's own outputs (Eq. 1 is exact)
    Wup = oracle_up_operand(cfg, W, 0)
    report["up_reconstructs"] = bool(np.array_equal(Zg[0] + Zg[1], wl.ring_matmul(Xr, Wup[:, Ig])))

    if float_report:
        got = wl.decode(Og[0] + Og[1], f)
        want = functionality.plain_ffn_float64(
            wl.decode(Xr, f), wl.decode(W["W1"][0], f), wl.decode(W["W2"][0], f), I1,
            wl.decode(W["WG"][0], f) if cfg.gated else None)
        report["float64_max_abs_err"] = float(np.abs(got - want).max())
    ctx.close()
    return report


def sample_positions(rng, rows, cols, count):
    """Corners, tile edges and random interior positions of a [rows, cols] output."""
    r = [0, 0, rows - 1, rows - 1]
    c = [0, cols - 1, 0, cols - 1]
    for edge in (63, 64, 127, 128, 255, 256):
        if edge < rows:
            r += [edge, edge]
            c += [0, cols - 1]
        if edge < cols:
            r += [0, rows - 1]
            c += [edge, edge]
    r = np.array(r + rng.integers(0, rows, count).tolist(), dtype=np.int32)
    c = np.array(c + rng.integers(0, cols, count).tolist(), dtype=np.int32)
    return r, c


def run_and_compare_sampled(cfg, seed, sparsity=None, tokens=None, step=0, matmul_path=cb.PATH_AUTO,
                            samples=512, ctx=None, weights=None, early_down=True):
    """Full-size check: messages E, F compared in full (they are cheap on the
    CPU), the products compared at sampled output positions computed one by
    one by the oracle from Eq. 1.  Up and down projections are exercised
    independently (the hidden state is synthetic)."""
    T = cfg.tokens if tokens is None else tokens
    d, f, g = cfg.d_model, cfg.frac_bits, cfg.groups
    rng = np.random.default_rng(seed + 17 * step)
    report = {"config": cfg.name, "tokens": T, "compared": [], "mismatches": 0}
    W = weights if weights is not None else wl.model_shares(cfg, seed, plain=False)
    _, X0, X1 = wl.activation_shares(cfg, seed, step=step, tokens=T)
    mask = wl.block_mask(cfg, seed, sparsity, step)
    own_ctx = ctx is None
    if own_ctx:
        ctx = make_context(cfg, T, matmul_path)
        load_weights(ctx, cfg, W)
    for party, Xs in ((0, X0), (1, X1)):
        ctx.load_shares(party, cb.X, cb.to_device(Xs))
    n = ctx.set_mask(mask)
    I1 = oracle.index_set(mask, cfg.block, 1)
    Ig = oracle.index_set(mask, cfg.block, g)
    report["n_active"] = n
    assert n == I1.size

    tri = wl.dealer_triple(seed, f"{cfg.name}/up/step{step}", T, d, g * n, valid=False)
    load_triple_up(ctx, tri)
    trd = wl.dealer_triple(seed, f"{cfg.name}/down/step{step}", T, n, d, valid=False)
    if early_down:
        # the down-projection's triple is already there when ffn_up runs, so the library may open its
        # weight side early (the full-chain tests load it late and cover the other order)
        load_triple_down(ctx, trd)
    ctx.ffn_up(T)
    report["path"] = ctx.stats().matmul_path
    Zg = [ctx.get(party, cb.Z_UP, (T, g * n)) for party in (0, 1)]
    ctx.truncate(cb.Z_UP)
    E = [oracle.mask_operand((X0, X1)[p], tri["A"][1 + p]) for p in (0, 1)]
    F = [oracle.mask_operand(oracle.index_cols(oracle_up_operand(cfg, W, 1 + p), Ig), tri["B"][1 + p]) for p in (0, 1)]
    Eo, Fo = oracle.reconstruct(*E), oracle.reconstruct(*F)
    rows, cols = sample_positions(rng, T, g * n, samples)
    for party in (0, 1):
        _mismatch(f"E_up[{party}]", ctx.get(party, cb.E_UP, (T, d)), E[party], report)
        _mismatch(f"F_up[{party}]", ctx.get(party, cb.F_UP, (g * n, d)).T, F[party], report)
        want = oracle.beaver_combine_at(party, Eo, Fo, tri["A"][1 + party], tri["B"][1 + party],
                                        tri["C"][1 + party], rows, cols)
        _mismatch(f"Z_up[{party}]@samples", Zg[party][rows, cols], want, report)
        Ht = ctx.get(party, cb.Z_UP, (T, g * n))
        _mismatch(f"trunc(Z_up)[{party}]@samples", Ht[rows, cols], oracle.truncate(party, want, f), report)

    _, H0, H1 = wl.hidden_shares(cfg, seed, n, step=step, tokens=T)
    for party, Hs in ((0, H0), (1, H1)):
        ctx.load_shares(party, cb.H, cb.to_device(Hs))
    if not early_down:
        load_triple_down(ctx, trd)
    ctx.ffn_down(T)
    Yg = [ctx.get(party, cb.Y, (T, d)) for party in (0, 1)]
    ctx.truncate(cb.Y)
    E = [oracle.mask_operand((H0, H1)[p], trd["A"][1 + p]) for p in (0, 1)]
    F = [oracle.mask_operand(oracle.index_rows(W["W2"][1 + p], I1), trd["B"][1 + p]) for p in (0, 1)]
    Eo, Fo = oracle.reconstruct(*E), oracle.reconstruct(*F)
    rows, cols = sample_positions(rng, T, d, samples)
    for party in (0, 1):
        _mismatch(f"E_dn[{party}]", ctx.get(party, cb.E_DN, (T, n)), E[party], report)
        _mismatch(f"F_dn[{party}]", ctx.get(party, cb.F_DN, (d, n)).T, F[party], report)
        want = oracle.beaver_combine_at(party, Eo, Fo, trd["A"][1 + party], trd["B"][1 + party],
                                        trd["C"][1 + party], rows, cols)
        _mismatch(f"Y[{party}]@samples", Yg[party][rows, cols], want, report)
        Yt = ctx.get(party, cb.Y, (T, d))
        _mismatch(f"trunc(Y)[{party}]@samples", Yt[rows, cols], oracle.truncate(party, want, f), report)
    if own_ctx:
        ctx.close()
    return report


def run_and_compare_products(cfg, seed, sparsity=None, tokens=None, step=0, matmul_path=cb.PATH_AUTO, ctx=None,
                             weights=None, early_down=True):
    """Full-size check, element by element: both projections under the configuration's mask on uniformly random
    shares (what the kernels see whatever the plaintext distribution), with the messages, the products and the
    truncated products of both parties compared in full with `oracle.somm` / `oracle.simm` / `oracle.truncate`.
    The two projections are exercised independently (the hidden state is synthetic), so no reconstruction or
    float64 report is made here; `run_and_compare_full` does that on real plaintexts."""
    T = cfg.tokens if tokens is None else tokens
    d, f, g = cfg.d_model, cfg.frac_bits, cfg.groups
    report = {"config": cfg.name, "tokens": T, "compared": [], "mismatches": 0}
    W = weights if weights is not None else wl.model_shares(cfg, seed, plain=False)
    _, X0, X1 = wl.activation_shares(cfg, seed, step=step, tokens=T)
    mask = wl.block_mask(cfg, seed, sparsity, step)
    own_ctx = ctx is None
    if own_ctx:
        ctx = make_context(cfg, T, matmul_path)
        load_weights(ctx, cfg, W)
    for party, Xs in ((0, X0), (1, X1)):
        ctx.load_shares(party, cb.X, cb.to_device(Xs))
    n = ctx.set_mask(mask)
    I1 = oracle.index_set(mask, cfg.block, 1)
    Ig = oracle.index_set(mask, cfg.block, g)
    report["n_active"] = n
    assert n == I1.size

    tri = wl.dealer_triple(seed, f"{cfg.name}/up/step{step}", T, d, g * n, valid=False)
    load_triple_up(ctx, tri)
    trd = wl.dealer_triple(seed, f"{cfg.name}/down/step{step}", T, n, d, valid=False)
    if early_down:
        load_triple_down(ctx, trd)
    ctx.ffn_up(T)
    report["path"] = ctx.stats().matmul_path
    Zg = [ctx.get(party, cb.Z_UP, (T, g * n)) for party in (0, 1)]
    ctx.truncate(cb.Z_UP)
    ref = oracle.somm((X0, X1), (oracle_up_operand(cfg, W, 1), oracle_up_operand(cfg, W, 2)), Ig,
                      tri["A"][1:], tri["B"][1:], tri["C"][1:])
    for party in (0, 1):
        _mismatch(f"E_up[{party}]", ctx.get(party, cb.E_UP, (T, d)), ref["E"][party], report)
        _mismatch(f"F_up[{party}]", ctx.get(party, cb.F_UP, (g * n, d)).T, ref["F"][party], report)
        _mismatch(f"Z_up[{party}]", Zg[party], ref["Z"][party], report)
        _mismatch(f"trunc(Z_up)[{party}]", ctx.get(party, cb.Z_UP, (T, g * n)),
                  oracle.truncate(party, ref["Z"][party], f), report)

    _, H0, H1 = wl.hidden_shares(cfg, seed, n, step=step, tokens=T)
    for party, Hs in ((0, H0), (1, H1)):
        ctx.load_shares(party, cb.H, cb.to_device(Hs))
    if not early_down:
        load_triple_down(ctx, trd)
    ctx.ffn_down(T)
    Yg = [ctx.get(party, cb.Y, (T, d)) for party in (0, 1)]
    ctx.truncate(cb.Y)
    refd = oracle.simm((H0, H1), W["W2"][1:], I1, trd["A"][1:], trd["B"][1:], trd["C"][1:])
    for party in (0, 1):
        _mismatch(f"E_dn[{party}]", ctx.get(party, cb.E_DN, (T, n)), refd["E"][party], report)
        _mismatch(f"F_dn[{party}]", ctx.get(party, cb.F_DN, (d, n)).T, refd["F"][party], report)
        _mismatch(f"Y[{party}]", Yg[party], refd["Z"][party], report)
        _mismatch(f"trunc(Y)[{party}]", ctx.get(party, cb.Y, (T, d)), oracle.truncate(party, refd["Z"][party], f),
                  report)
    if own_ctx:
        ctx.close()
    return report
