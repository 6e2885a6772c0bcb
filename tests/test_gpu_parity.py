"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle,
bit for bit, on the same seeded inputs."""
import ctypes

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2505_07239_b200 import workloads as wl  # noqa: E402


@pytest.fixture(scope="module")
def hz():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from tests import harness

    return harness


def _ok(report, path=None):
    assert report["mismatches"] == 0, [c for c in report["compared"] if c[2]]
    if path is not None:
        assert report["path"] == path, "the requested matmul path did not run"
    return report


PATHS = [1, 2]   # COMET_PATH_SIMT, COMET_PATH_LIMB


@pytest.mark.parametrize("path", PATHS)
def test_tiny_full(hz, path):
    r = _ok(hz.run_and_compare_full(wl.CONFIGS["tiny"], seed=1, matmul_path=path), path)
    assert r["n_active"] == 96 and r["up_reconstructs"]
    # 12 fractional bits, |w| <= 1, 96 active neurons: bounded by n * 2^-f, not by 2^-10
    assert r["float64_max_abs_err"] < 96 * 2.0 ** -12


@pytest.mark.parametrize("path", PATHS)
def test_opt125m_full(hz, path):
    r = _ok(hz.run_and_compare_full(wl.CONFIGS["opt125m"], seed=2, matmul_path=path), path)
    assert r["n_active"] == 320 and r["up_reconstructs"]
    assert r["float64_max_abs_err"] < 2.0 ** -10


@pytest.mark.parametrize("path", PATHS)
def test_opt13b_95_full(hz, path):
    r = _ok(hz.run_and_compare_full(wl.CONFIGS["opt1.3b"], seed=3, sparsity=0.95, matmul_path=path), path)
    assert r["n_active"] == 416 and r["up_reconstructs"]
    assert r["float64_max_abs_err"] < 2.0 ** -10


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("tokens", [1, 17, 130])
def test_ragged_token_counts(hz, path, tokens):
    _ok(hz.run_and_compare_full(wl.CONFIGS["opt125m"], seed=4, tokens=tokens, matmul_path=path, float_report=False), path)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("tokens", [5, 40, 140])
def test_contraction_depths_that_end_inside_a_k_block(hz, path, tokens):
    """d_model = 48 and n = 48 (three 16-neuron blocks): both projections contract over one and a half 32-deep
    blocks, and 48 weight rows end inside a 64-row plane tile; with 5, 40 and 140 token rows the few-token kernel,
    one ragged row tile and two row tiles are covered."""
    cfg = wl.FFNConfig("ragged-k", tokens, 48, 160, 16, 14, False, 0.3, "uniform", "normal", "normal0.02")
    m = np.zeros(cfg.n_blocks, np.uint8)
    m[[1, 4, 9]] = 1
    r = _ok(hz.run_and_compare_full(cfg, seed=41 + tokens, mask=m, matmul_path=path), path)
    assert r["n_active"] == 48 and r["up_reconstructs"]
    assert r["float64_max_abs_err"] < 2.0 ** -10


@pytest.mark.parametrize("path", PATHS)
def test_gated_small(hz, path):
    cfg = wl.FFNConfig("gated-small", 40, 128, 512, 64, 16, True, 0.25, "uniform", "normal", "normal0.02")
    r = _ok(hz.run_and_compare_full(cfg, seed=5, matmul_path=path), path)
    assert r["n_active"] == 128 and r["up_reconstructs"]
    assert r["float64_max_abs_err"] < 2.0 ** -10


@pytest.mark.parametrize("path", PATHS)
def test_all_ones_mask_is_the_dense_product(hz, path):
    cfg = wl.CONFIGS["tiny"]
    r = _ok(hz.run_and_compare_full(cfg, seed=6, sparsity=0.0, matmul_path=path), path)
    assert r["n_active"] == cfg.d_ff and r["up_reconstructs"]


@pytest.mark.parametrize("path", PATHS)
def test_single_block_first_and_last(hz, path):
    cfg = wl.CONFIGS["tiny"]
    for b in (0, cfg.n_blocks - 1):
        m = np.zeros(cfg.n_blocks, np.uint8)
        m[b] = 1
        r = _ok(hz.run_and_compare_full(cfg, seed=7, mask=m, matmul_path=path, float_report=False), path)
        assert r["n_active"] == cfg.block


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("sparsity", [0.0, 0.5, 0.8, 0.9])
def test_opt13b_sweep_sampled(hz, path, sparsity):
    _ok(hz.run_and_compare_sampled(wl.CONFIGS["opt1.3b"], seed=8, sparsity=sparsity, matmul_path=path), path)


@pytest.mark.parametrize("path", PATHS)
def test_llama7b_sampled(hz, path):
    r = _ok(hz.run_and_compare_sampled(wl.CONFIGS["llama7b"], seed=9, matmul_path=path), path)
    assert 23 * 64 <= r["n_active"] <= 26 * 64


@pytest.mark.parametrize("path", PATHS)
def test_opt67b_decode_steps_sampled(hz, path):
    cfg = wl.CONFIGS["opt6.7b-decode"]
    W = wl.model_shares(cfg, 10, plain=False)
    ctx = hz.make_context(cfg, cfg.tokens, path, max_active=2048)
    hz.load_weights(ctx, cfg, W)
    for step in (0, 1, 63):       # fresh mask, X and triples per step, weights loaded once
        r = _ok(hz.run_and_compare_sampled(cfg, seed=10, step=step, matmul_path=path, ctx=ctx, weights=W,
                                           samples=256), path)
        assert r["n_active"] == 1312
    ctx.close()


# ---- every benchmark configuration at full size, products compared element by element (not at samples)

@pytest.mark.parametrize("path", PATHS)
def test_opt13b_90_products_in_full(hz, path):
    """The headline configuration: OPT-1.3B shape at 90 % block sparsity."""
    r = _ok(hz.run_and_compare_products(wl.CONFIGS["opt1.3b"], seed=21, sparsity=0.9, matmul_path=path), path)
    assert r["n_active"] == 832


@pytest.mark.parametrize("sparsity,n", [(0.8, 1632), (0.5, 4096), (0.0, 8192)])
def test_opt13b_sweep_products_in_full(hz, sparsity, n):
    """The rest of the sparsity sweep on the default (tensor-core) path; n = 1632 leaves a ragged column tile."""
    r = _ok(hz.run_and_compare_products(wl.CONFIGS["opt1.3b"], seed=22, sparsity=sparsity), 2)
    assert r["n_active"] == n


def test_llama7b_products_in_full(hz):
    r = _ok(hz.run_and_compare_products(wl.CONFIGS["llama7b"], seed=23), 2)
    assert 23 * 64 <= r["n_active"] <= 26 * 64


def test_opt67b_decode_steps_products_in_full(hz):
    cfg = wl.CONFIGS["opt6.7b-decode"]
    W = wl.model_shares(cfg, 24, plain=False)
    ctx = hz.make_context(cfg, cfg.tokens, 2, max_active=2048)
    hz.load_weights(ctx, cfg, W)
    for step in (0, 1, 63):       # fresh mask, X and triples per step, weights loaded once
        r = _ok(hz.run_and_compare_products(cfg, seed=24, step=step, ctx=ctx, weights=W), 2)
        assert r["n_active"] == 1312
    ctx.close()


def test_timeout_status_reaches_the_caller(hz):
    """COMET_ERR_TIMEOUT is handed out by the calls that hand results out.  No kernel waits here: the error
    words a timed-out kernel would write are set through the library's test hook."""
    from paper_2505_07239_b200 import binding as cb

    cfg = wl.CONFIGS["tiny"]
    r = hz.run_and_compare_full(cfg, seed=25, float_report=False)
    assert r["mismatches"] == 0
    ctx = hz.make_context(cfg, cfg.tokens)
    lib, h = cb.library(), ctx._h
    W = wl.model_shares(cfg, 25, plain=False)
    hz.load_weights(ctx, cfg, W)
    assert lib.comet_synchronize(h) == cb.OK
    assert lib.comet_inject_timeout(h) == cb.OK
    assert lib.comet_synchronize(h) == cb.ERR_TIMEOUT
    out = torch.zeros(cfg.d_ff * cfg.d_model, dtype=torch.int64, device="cuda")
    assert lib.comet_get(h, 0, cb.W1, out.data_ptr(), 0, out.numel(), None) == cb.ERR_TIMEOUT
    n = ctypes.c_int32(0)
    m = torch.ones(cfg.n_blocks, dtype=torch.uint8, device="cuda")
    assert lib.comet_set_mask(h, m.data_ptr(), 0, cfg.n_blocks, ctypes.byref(n)) == cb.ERR_TIMEOUT
    assert b"bounded" in lib.comet_strerror(cb.ERR_TIMEOUT)
    ctx.close()
    # another context is unaffected
    assert hz.run_and_compare_full(cfg, seed=26, float_report=False)["mismatches"] == 0


def test_masked_neurons_contribute_exactly_zero(hz):
    """Garbage in the weight shares of inactive neurons leaves every output bit unchanged."""
    from paper_2505_07239_b200 import binding as cb

    cfg = wl.CONFIGS["tiny"]
    T, d, f = cfg.tokens, cfg.d_model, cfg.frac_bits
    seed = 11
    W = wl.model_shares(cfg, seed, plain=False)
    mask = wl.block_mask(cfg, seed)
    I = wl.active_neurons(mask, cfg.block)
    dead = np.setdiff1d(np.arange(cfg.d_ff), I)
    _, X0, X1 = wl.activation_shares(cfg, seed)
    outs = []
    for garble in (False, True):
        Wv = {k: tuple(a.copy() for a in v) for k, v in W.items()}
        if garble:
            rng = np.random.default_rng(0)
            for slot in (1, 2):
                Wv["W1"][slot][:, dead] = rng.integers(0, 1 << 64, (d, dead.size), dtype=np.uint64)
                Wv["W2"][slot][dead, :] = rng.integers(0, 1 << 64, (dead.size, d), dtype=np.uint64)
        ctx = hz.make_context(cfg, T)
        hz.load_weights(ctx, cfg, Wv)
        for p, Xs in ((0, X0), (1, X1)):
            ctx.load_shares(p, cb.X, cb.to_device(Xs))
        n = ctx.set_mask(mask)
        hz.load_triple_up(ctx, wl.dealer_triple(seed, "u", T, d, n, valid=False))
        ctx.ffn_up(T)
        ctx.truncate(cb.Z_UP)
        _, H0, H1 = wl.hidden_shares(cfg, seed, n)
        for p, Hs in ((0, H0), (1, H1)):
            ctx.load_shares(p, cb.H, cb.to_device(Hs))
        hz.load_triple_down(ctx, wl.dealer_triple(seed, "d", T, n, d, valid=False))
        ctx.ffn_down(T)
        ctx.truncate(cb.Y)
        outs.append([ctx.get(p, t, s) for p in (0, 1) for t, s in ((cb.Z_UP, (T, n)), (cb.Y, (T, d)),
                                                                    (cb.F_UP, (n, d)), (cb.F_DN, (d, n)))])
        ctx.close()
    for a, b in zip(*outs):
        assert np.array_equal(a, b)


def test_no_active_neuron(hz):
    from paper_2505_07239_b200 import binding as cb

    cfg = wl.CONFIGS["tiny"]
    T, d = cfg.tokens, cfg.d_model
    W = wl.model_shares(cfg, 12, plain=False)
    ctx = hz.make_context(cfg, T)
    hz.load_weights(ctx, cfg, W)
    _, X0, X1 = wl.activation_shares(cfg, 12)
    for p, Xs in ((0, X0), (1, X1)):
        ctx.load_shares(p, cb.X, cb.to_device(Xs))
    assert ctx.set_mask(np.zeros(cfg.n_blocks, np.uint8)) == 0
    assert ctx.get_index().size == 0
    tri = wl.dealer_triple(12, "u", T, d, 0, valid=False)
    hz.load_triple_up(ctx, tri)
    ctx.ffn_up(T)                       # nothing to do
    ctx.truncate(cb.Z_UP)
    for p in (0, 1):
        ctx.load_shares(p, cb.C_DN, cb.to_device(np.ones((T, d), np.uint64)))
    ctx.ffn_down(T)
    ctx.truncate(cb.Y)
    for p in (0, 1):
        assert not ctx.get(p, cb.Y, (T, d)).any()
    ctx.close()


def test_run_to_run_determinism(hz):
    a = hz.run_and_compare_sampled(wl.CONFIGS["opt125m"], seed=13, samples=64)
    b = hz.run_and_compare_sampled(wl.CONFIGS["opt125m"], seed=13, samples=64)
    assert a["mismatches"] == 0 and b["mismatches"] == 0


def test_errors_are_status_codes(hz):
    from paper_2505_07239_b200 import binding as cb

    cfg = wl.CONFIGS["tiny"]
    T, d, D = cfg.tokens, cfg.d_model, cfg.d_ff
    ctx = hz.make_context(cfg, T)
    lib = cb.library()
    h = ctx._h
    buf = torch.zeros(D * d, dtype=torch.int64, device="cuda")
    n = ctypes.c_int32(-5)
    # wrong order
    assert lib.comet_ffn_up(h, T) == -3
    assert lib.comet_truncate(h, cb.Z_UP) == -3
    assert lib.comet_load_shares(h, 0, cb.B_UP, buf.data_ptr(), 0, 96, d) == -3      # needs the mask first
    # bad arguments
    assert lib.comet_load_shares(h, 2, cb.X, buf.data_ptr(), 0, T, d) == -1
    assert lib.comet_load_shares(h, 0, cb.Z_UP, buf.data_ptr(), 0, T, d) == -1       # not an input
    assert lib.comet_load_shares(h, 0, cb.WG, buf.data_ptr(), 0, D, d) == -1         # not gated
    assert lib.comet_load_shares(h, 0, cb.X, None, 0, T, d) == -1
    assert lib.comet_load_shares(h, 0, cb.X, buf.data_ptr(), 5, T, d) == -1
    # bad shapes
    assert lib.comet_load_shares(h, 0, cb.X, buf.data_ptr(), 0, T + 1, d) == -2
    assert lib.comet_load_shares(h, 0, cb.X, buf.data_ptr(), 0, T, d + 16) == -2
    assert lib.comet_load_shares(h, 0, cb.W1, buf.data_ptr(), 0, d, D) == -2         # transposed
    m = torch.ones(cfg.n_blocks, dtype=torch.uint8, device="cuda")
    assert lib.comet_set_mask(h, m.data_ptr(), 0, cfg.n_blocks - 1, ctypes.byref(n)) == -2
    assert lib.comet_set_mask(h, m.data_ptr(), 0, cfg.n_blocks, ctypes.byref(n)) == 0 and n.value == D
    assert lib.comet_load_shares(h, 0, cb.B_UP, buf.data_ptr(), 0, 96, d) == -2      # n is d_ff now
    assert lib.comet_ffn_up(h, T + 1) == -2
    assert lib.comet_ffn_up(h, T) == -3                                              # inputs still missing
    assert lib.comet_truncate(h, cb.X) == -1
    assert lib.comet_get(h, 0, cb.Y, buf.data_ptr(), 0, T * d, None) == -3
    # a context sized for fewer active neurons refuses a denser mask
    small = cb.Comet(T, d, D, cfg.block, cfg.frac_bits, False, 0, 64)
    assert lib.comet_set_mask(small._h, m.data_ptr(), 0, cfg.n_blocks, ctypes.byref(n)) == -2
    small.close()
    # the context is still usable afterwards
    ctx.close()
    hz.run_and_compare_full(cfg, seed=14, float_report=False)


def test_bound_inputs_give_the_same_bits_as_copied_ones(hz):
    """comet_bind_shares: inputs read in place from the caller's device memory."""
    from paper_2505_07239_b200 import binding as cb

    cfg = wl.CONFIGS["opt125m"]
    T, d, seed = cfg.tokens, cfg.d_model, 15
    W = wl.model_shares(cfg, seed, plain=False)
    mask = wl.block_mask(cfg, seed)
    _, X0, X1 = wl.activation_shares(cfg, seed)
    outs = []
    for bind in (False, True):
        ctx = hz.make_context(cfg, T)
        keep = []                                     # bound tensors stay alive until the context is closed

        def put(p, tid, arr):
            t = cb.to_device(arr)
            if bind:
                keep.append(t)
                ctx.bind_shares(p, tid, t)
            else:
                ctx.load_shares(p, tid, t)

        for p in (0, 1):
            put(p, cb.W1, wl.lib_layout(W["W1"][1 + p]))
            put(p, cb.W2, wl.lib_layout(W["W2"][1 + p]))
            put(p, cb.X, (X0, X1)[p])
        n = ctx.set_mask(mask)
        tri = wl.dealer_triple(seed, "u", T, d, n, valid=False)
        trd = wl.dealer_triple(seed, "d", T, n, d, valid=False)
        _, H0, H1 = wl.hidden_shares(cfg, seed, n)
        for p in (0, 1):
            put(p, cb.A_UP, tri["A"][1 + p]); put(p, cb.B_UP, wl.lib_layout(tri["B"][1 + p])); put(p, cb.C_UP, tri["C"][1 + p])
            put(p, cb.A_DN, trd["A"][1 + p]); put(p, cb.B_DN, wl.lib_layout(trd["B"][1 + p])); put(p, cb.C_DN, trd["C"][1 + p])
            put(p, cb.H, (H0, H1)[p])
        ctx.ffn_up(T)
        ctx.truncate(cb.Z_UP)
        ctx.ffn_down(T)
        ctx.truncate(cb.Y)
        outs.append([ctx.get(p, t, s) for p in (0, 1) for t, s in ((cb.Z_UP, (T, n)), (cb.Y, (T, d)), (cb.E_DN, (T, n)))])
        if bind:
            # an unaligned pointer is refused, and a new mask ends the bindings of the triples
            t = torch.zeros(T * d + 1, dtype=torch.int64, device="cuda")
            assert cb.library().comet_bind_shares(ctx._h, 0, cb.X, t.data_ptr() + 8, T, d) == -1
            ctx.set_mask(mask)
            assert cb.library().comet_ffn_up(ctx._h, T) == -3
        ctx.close()
    for a, b in zip(*outs):
        assert np.array_equal(a, b)


def test_four_problems_in_flight_at_full_size(hz):
    """The benchmark's throughput configuration: four contexts on four streams, OPT-1.3B shape at 90 % sparsity,
    inputs bound in place, two steps per context issued round-robin with nothing but each context's own mask
    report between them.  Every context's last step is compared with the oracle: messages in full, products and
    truncated products at sampled positions."""
    from paper_2505_07239_b200 import binding as cb

    cfg = wl.CONFIGS["opt1.3b"]
    T, d, f, seed, C = cfg.tokens, cfg.d_model, cfg.frac_bits, 31, 4
    W = wl.model_shares(cfg, seed, plain=False)
    Wdev = [[cb.to_device(wl.lib_layout(W[k][1 + p])) for k in ("W1", "W2")] for p in (0, 1)]
    n_cap = cfg.n_active_blocks(0.9) * cfg.block
    ctxs, inputs = [], []
    for k in range(C):
        sk = torch.cuda.Stream()
        cx = cb.Comet(T, d, cfg.d_ff, cfg.block, f, 0, 0, n_cap, cb.PATH_AUTO, sk)
        for p in (0, 1):
            cx.bind_shares(p, cb.W1, Wdev[p][0])
            cx.bind_shares(p, cb.W2, Wdev[p][1])
        ctxs.append((cx, sk))
        steps = []
        for j in range(2):
            step = 10 * k + j
            mask = wl.block_mask(cfg, seed, 0.9, step)
            n = int(mask.sum()) * cfg.block
            _, X0, X1 = wl.activation_shares(cfg, seed, step=step, tokens=T)
            _, H0, H1 = wl.hidden_shares(cfg, seed, n, step=step, tokens=T)
            tri = wl.dealer_triple(seed, f"fl/up/{step}", T, d, n, valid=False)
            trd = wl.dealer_triple(seed, f"fl/dn/{step}", T, n, d, valid=False)
            host = {"mask": mask, "n": n, "X": (X0, X1), "H": (H0, H1), "up": tri, "dn": trd}
            dev = [{cb.X: cb.to_device((X0, X1)[p]), cb.H: cb.to_device((H0, H1)[p]),
                    cb.A_UP: cb.to_device(tri["A"][1 + p]), cb.B_UP: cb.to_device(wl.lib_layout(tri["B"][1 + p])),
                    cb.C_UP: cb.to_device(tri["C"][1 + p]), cb.A_DN: cb.to_device(trd["A"][1 + p]),
                    cb.B_DN: cb.to_device(wl.lib_layout(trd["B"][1 + p])), cb.C_DN: cb.to_device(trd["C"][1 + p])}
                   for p in (0, 1)]
            steps.append((host, dev, torch.from_numpy(mask).cuda()))
        inputs.append(steps)
    torch.cuda.synchronize()
    zup = {}
    for j in range(2):
        for k, (cx, sk) in enumerate(ctxs):
            host, dev, mask_dev = inputs[k][j]
            with torch.cuda.stream(sk):
                assert cx.set_mask(mask_dev) == host["n"]
                for p in (0, 1):
                    for tid in (cb.X, cb.A_UP, cb.B_UP, cb.C_UP, cb.A_DN, cb.B_DN, cb.C_DN):
                        cx.bind_shares(p, tid, dev[p][tid])
                cx.ffn_up(T)
                if j == 1:                              # keep the untruncated product of the step that is checked
                    zup[k] = [torch.empty(T * host["n"], dtype=torch.int64, device="cuda") for _ in (0, 1)]
                    for p in (0, 1):
                        cx.get_into(p, cb.Z_UP, zup[k][p])
                cx.truncate(cb.Z_UP)
                for p in (0, 1):
                    cx.bind_shares(p, cb.H, dev[p][cb.H])
                cx.ffn_down(T)
                cx.truncate(cb.Y)
    torch.cuda.synchronize()
    rng = np.random.default_rng(5)
    bad = 0
    for k, (cx, sk) in enumerate(ctxs):
        host, _, _ = inputs[k][1]
        n, tri, trd, mask = host["n"], host["up"], host["dn"], host["mask"]
        I = oracle.index_set(mask, cfg.block, 1)
        E = [oracle.mask_operand(host["X"][p], tri["A"][1 + p]) for p in (0, 1)]
        F = [oracle.mask_operand(oracle.index_cols(W["W1"][1 + p], I), tri["B"][1 + p]) for p in (0, 1)]
        Eo, Fo = oracle.reconstruct(*E), oracle.reconstruct(*F)
        rows, cols = hz.sample_positions(rng, T, n, 256)
        for p in (0, 1):
            bad += int((cx.get(p, cb.E_UP, (T, d)) != E[p]).sum())
            bad += int((cx.get(p, cb.F_UP, (n, d)).T != F[p]).sum())
            want = oracle.beaver_combine_at(p, Eo, Fo, tri["A"][1 + p], tri["B"][1 + p], tri["C"][1 + p], rows, cols)
            got = zup[k][p].cpu().numpy().view(np.uint64).reshape(T, n)
            bad += int((got[rows, cols] != want).sum())
            bad += int((cx.get(p, cb.Z_UP, (T, n))[rows, cols] != oracle.truncate(p, want, f)).sum())
        E = [oracle.mask_operand(host["H"][p], trd["A"][1 + p]) for p in (0, 1)]
        F = [oracle.mask_operand(oracle.index_rows(W["W2"][1 + p], I), trd["B"][1 + p]) for p in (0, 1)]
        Eo, Fo = oracle.reconstruct(*E), oracle.reconstruct(*F)
        rows, cols = hz.sample_positions(rng, T, d, 256)
        for p in (0, 1):
            bad += int((cx.get(p, cb.E_DN, (T, n)) != E[p]).sum())
            bad += int((cx.get(p, cb.F_DN, (d, n)).T != F[p]).sum())
            want = oracle.beaver_combine_at(p, Eo, Fo, trd["A"][1 + p], trd["B"][1 + p], trd["C"][1 + p], rows, cols)
            bad += int((cx.get(p, cb.Y, (T, d))[rows, cols] != oracle.truncate(p, want, f)).sum())
    for cx, _ in ctxs:
        cx.close()
    assert bad == 0
