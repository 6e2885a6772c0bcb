"""GPU parity on extreme ring words.

Uniformly random shares never push a 32-bit limb accumulator of the tensor-core path near its limits, so these
cases choose the shares such that every operand the kernels multiply -- the opened E and F, the triple shares
A_i (hence V_i = A_i + i*E) and B_i -- consists of hand-picked words: all-ones, the sign bit alone, one, and
alternating 0xFF / 0x00 bytes.  The all-ones region fills whole output tiles over the full depth a segment may
accumulate (16384 contraction indices: limb sums with s <= 3 reach 4 * 16384 * 255^2, just below 2^32; the
sums with s >= 4 pass 2^32 and wrap, which Eq. 1 mod 2^64 allows because only their low 64 - 8s bits count).
Expected values come from the oracle (Eq. 1 position by position) and, for the all-ones tile, from the closed
form Z_i = C_i + 2K.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2505_07239_b200 import workloads as wl  # noqa: E402

U64 = np.uint64
ONES, SIGN, ONE = U64(0xFFFFFFFFFFFFFFFF), U64(0x8000000000000000), U64(1)
ALT_HI, ALT_LO, MAXPOS = U64(0xFF00FF00FF00FF00), U64(0x00FF00FF00FF00FF), U64(0x7FFFFFFFFFFFFFFF)
CYCLE = np.array([ONES, SIGN, ONE, ALT_HI, ALT_LO, MAXPOS], dtype=U64)


def _left_pattern(T, K, band):
    """[T, K]: rows [0, band) all-ones, then a band of sign bits, a band cycling through all six words along
    the contraction index, and seeded random words for the rest."""
    E = wl.random_u64(7, "extreme/left", T * K).reshape(T, K)
    E[:band] = ONES
    E[band:2 * band] = SIGN
    E[2 * band:3 * band] = CYCLE[np.arange(K) % 6][None, :]
    return E


def _right_pattern(K, N, band):
    """[K, N]: columns [0, band) all-ones, then bands of the sign bit, of ones, of alternating bytes, a band
    cycling with the contraction index, and seeded random words for the rest."""
    F = wl.random_u64(7, "extreme/right", K * N).reshape(K, N)
    F[:, :band] = ONES
    F[:, band:2 * band] = SIGN
    F[:, 2 * band:3 * band] = ONE
    F[:, 3 * band:4 * band] = ALT_HI
    F[:, 4 * band:5 * band] = CYCLE[(np.arange(K) + 1) % 6][:, None]
    return F


def _run_down(hz, T, d, D, left_band, right_band, samples):
    """Down-projection with every block active (contraction depth D) on the chosen words; returns the report."""
    from paper_2505_07239_b200 import binding as cb

    cfg = wl.FFNConfig("extreme", T, d, D, 32, 16, False, 1.0, "uniform", "normal", "normal0.02")
    E, F = _left_pattern(T, D, left_band), _right_pattern(D, d, right_band)
    zero_l, zero_r = np.zeros((T, D), U64), np.zeros((D, d), U64)
    # party 0 opens E_0 = E and F_0 = F, party 1 opens zeros; A_0 = E, A_1 = 0 (so V_0 = V_1 = E); B_0 = B_1 = F
    A = (E, zero_l)
    B = (F, F)
    H = (E + E, zero_l)                     # H_i = E_i + A_i
    W2 = (F + F, F)                         # W2_i = F_i + B_i
    C = tuple(wl.random_u64(7, f"extreme/C{p}", T * d).reshape(T, d) for p in (0, 1))

    ctx = cb.Comet(T, d, D, cfg.block, cfg.frac_bits, 0, 0, 0, cb.PATH_LIMB)
    for p in (0, 1):
        ctx.load_shares(p, cb.W2, cb.to_device(wl.lib_layout(W2[p])))
    assert ctx.set_mask(np.ones(D // cfg.block, np.uint8)) == D
    for p in (0, 1):
        ctx.load_shares(p, cb.H, cb.to_device(H[p]))
        ctx.load_shares(p, cb.A_DN, cb.to_device(A[p]))
        ctx.load_shares(p, cb.B_DN, cb.to_device(wl.lib_layout(B[p])))
        ctx.load_shares(p, cb.C_DN, cb.to_device(C[p]))
    ctx.ffn_down(T)
    assert ctx.stats().matmul_path == cb.PATH_LIMB
    Y = [ctx.get(p, cb.Y, (T, d)) for p in (0, 1)]
    Eg = [ctx.get(p, cb.E_DN, (T, D)) for p in (0, 1)]
    Fg = [ctx.get(p, cb.F_DN, (d, D)).T for p in (0, 1)]
    ctx.truncate(cb.Y)
    Yt = [ctx.get(p, cb.Y, (T, d)) for p in (0, 1)]
    ctx.close()

    I = np.arange(D, dtype=np.int32)
    Eo = [oracle.mask_operand(H[p], A[p]) for p in (0, 1)]
    Fo = [oracle.mask_operand(oracle.index_rows(W2[p], I), B[p]) for p in (0, 1)]
    Er, Fr = oracle.reconstruct(*Eo), oracle.reconstruct(*Fo)
    assert np.array_equal(Er, E) and np.array_equal(Fr, F)           # the kernels multiply exactly the chosen words
    bad = 0
    for p in (0, 1):
        bad += int((Eg[p] != Eo[p]).sum()) + int((Fg[p] != Fo[p]).sum())
    rng = np.random.default_rng(3)
    rows, cols = hz.sample_positions(rng, T, d, samples)
    # every pairing of a left band with a right band, at a few positions each
    lb = [min(T - 1, k * left_band + o) for k in range(4) for o in (0, left_band - 1)]
    rb = [min(d - 1, k * right_band + o) for k in range(6) for o in (0, right_band - 1)]
    rows = np.concatenate([rows, np.repeat(lb, len(rb))]).astype(np.int32)
    cols = np.concatenate([cols, np.tile(rb, len(lb))]).astype(np.int32)
    for p in (0, 1):
        want = oracle.beaver_combine_at(p, Er, Fr, A[p], B[p], C[p], rows, cols)
        bad += int((Y[p][rows, cols] != want).sum())
        bad += int((Yt[p][rows, cols] != oracle.truncate(p, want, cfg.frac_bits)).sum())
        # closed form on the all-ones tile: (-1)(-1) summed over both products = 2K
        tile = Y[p][:min(left_band, T), :right_band]
        bad += int((tile != C[p][:min(left_band, T), :right_band] + U64(2 * D)).sum())
    return bad


def test_extreme_words_full_depth_segments_many_tokens():
    """OPT-1.3B shape, all 8192 neurons active: a down-projection tile is 512 steps of 32 deep, the most a
    segment accumulates, and the first tile of the launch (all-ones operands) lies inside one CTA's share."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from tests import harness

    assert _run_down(harness, 512, 2048, 8192, 128, 64, 1024) == 0


def test_extreme_words_few_token_kernel_deep_contraction():
    """At most 32 token rows (operand roles exchanged) over 51200 contraction indices: every CTA's share of the
    launch exceeds the 512-step cap of a segment, so full-depth segments of all-ones operands occur."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from tests import harness

    assert _run_down(harness, 32, 1024, 51200, 8, 128, 512) == 0
