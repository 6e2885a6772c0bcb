"""Sharding the active neurons over ranks (paper_2505_07239_b200/shard.py), on CPU: two gloo ranks run the oracle
on their shards and the partial down-projection shares, added over the ranks, must equal the whole layer's shares
bit for bit (Eq. 1 is a sum over the contraction index; Section 2.1: shares add locally)."""
import os

import numpy as np
import pytest

torch = pytest.importorskip("torch")

import oracle  # noqa: E402
from paper_2505_07239_b200 import shard  # noqa: E402
from paper_2505_07239_b200 import workloads as wl  # noqa: E402

U64 = np.uint64
CFG = wl.FFNConfig("shard-small", 12, 32, 256, 16, 12, False, 0.5, "uniform", "normal", "normal0.02")
SEED = 404


def _layer():
    """The whole layer's inputs, the same on every rank (same seed)."""
    W = wl.model_shares(CFG, SEED, plain=False)
    mask = wl.block_mask(CFG, SEED, 0.5)
    I = oracle.index_set(mask, CFG.block, 1)
    _, X0, X1 = wl.activation_shares(CFG, SEED)
    _, H0, H1 = wl.hidden_shares(CFG, SEED, I.size)
    up = wl.dealer_triple(SEED, "shard/up", CFG.tokens, CFG.d_model, I.size)
    dn = wl.dealer_triple(SEED, "shard/dn", CFG.tokens, I.size, CFG.d_model)
    return W, mask, I, (X0, X1), (H0, H1), up, dn


def _rank_partials(rank, world):
    """One rank's products on its shard, by the oracle: (its columns of the up result, its partial down result)."""
    W, mask, I, X, H, up, dn = _layer()
    neurons = shard.owned_neurons(CFG.n_blocks, CFG.block, rank, world)
    cols = shard.local_columns(mask, CFG.block, rank, world)
    I_r = oracle.index_set(shard.local_mask(mask, rank, world), CFG.block, 1)
    assert np.array_equal(neurons[I_r], I[cols])                  # local compact order = the rank's part of the global one
    W1_r = [np.ascontiguousarray(W["W1"][s][:, neurons]) for s in (1, 2)]
    W2_r = [np.ascontiguousarray(W["W2"][s][neurons, :]) for s in (1, 2)]
    take_c = lambda a: np.ascontiguousarray(a[:, cols])           # noqa: E731
    take_r = lambda a: np.ascontiguousarray(a[cols, :])           # noqa: E731
    zu = oracle.somm(X, W1_r, I_r, up["A"][1:], [take_c(b) for b in up["B"][1:]],
                     [take_c(c) for c in up["C"][1:]])["Z"]
    c_dn = dn["C"][1:] if rank == 0 else [np.zeros_like(dn["C"][1]), np.zeros_like(dn["C"][2])]
    yd = oracle.simm([take_c(h) for h in H], W2_r, I_r, [take_c(a) for a in dn["A"][1:]],
                     [take_r(b) for b in dn["B"][1:]], c_dn)["Z"]
    return cols, zu, yd


def _worker(rank, world, port, out):
    import torch.distributed as dist

    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cols, zu, yd = _rank_partials(rank, world)
    summed = []
    for p in (0, 1):
        t = torch.from_numpy(yd[p].view(np.int64).copy())
        shard.add_over_ranks(t)                                   # the one exchange step of the sharded layer
        summed.append(t.numpy().view(U64).copy())
    dist.barrier()
    out.put((rank, cols, [z.copy() for z in zu], summed))
    dist.destroy_process_group()


def test_two_ranks_partial_shares_sum_to_the_whole_layer_bit_for_bit():
    import torch.multiprocessing as mp

    W, mask, I, X, H, up, dn = _layer()
    ref_up = oracle.somm(X, W["W1"][1:], I, up["A"][1:], up["B"][1:], up["C"][1:])["Z"]
    ref_dn = oracle.simm(H, W["W2"][1:], I, dn["A"][1:], dn["B"][1:], dn["C"][1:])["Z"]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted((q.get(timeout=180) for _ in procs), key=lambda g: g[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    seen = np.zeros(I.size, bool)
    for rank, cols, zu, summed in got:
        for party in (0, 1):
            assert np.array_equal(zu[party], ref_up[party][:, cols])      # up: the rank's columns, no exchange
            assert np.array_equal(summed[party], ref_dn[party])           # down: the sum over ranks, on every rank
        seen[cols] = True
    assert seen.all()                                                      # the shards cover every active neuron once


def test_partition_helpers():
    mask = np.array([1, 0, 1, 1, 0, 0, 1, 1, 1], np.uint8)
    world, block = 3, 4
    all_cols = []
    for r in range(world):
        assert np.array_equal(shard.owned_blocks(9, r, world), np.arange(r, 9, world))
        assert np.array_equal(shard.local_mask(mask, r, world), mask[r::world])
        cols = shard.local_columns(mask, block, r, world)
        # the rank's active neurons, through its own mask, are the same neurons as its columns of the global list
        glob = np.flatnonzero(np.repeat(mask, block))
        loc = shard.owned_neurons(9, block, r, world)[np.flatnonzero(np.repeat(mask[r::world], block))]
        assert np.array_equal(glob[cols], loc)
        all_cols.append(cols)
    assert np.array_equal(np.sort(np.concatenate(all_cols)), np.arange(int(mask.sum()) * block))
    # one process, no process group: the reduction is the identity
    t = torch.arange(6, dtype=torch.int64)
    assert torch.equal(shard.add_over_ranks(t.clone()), t)
    # wrap-around: the integer sum is the ring sum
    a = np.array([0xFFFFFFFFFFFFFFFF, 0x8000000000000000], U64)
    s = (torch.from_numpy(a.view(np.int64).copy()) + torch.from_numpy(a.view(np.int64).copy())).numpy().view(U64)
    assert s[0] == U64(0xFFFFFFFFFFFFFFFE) and s[1] == U64(0)
    Wup = np.arange(9 * block * 2, dtype=U64).reshape(9 * block, 2)
    W2 = np.ascontiguousarray(Wup.T)
    a_up, a_dn = shard.slice_stored_weights(Wup, W2, block, 1, world)
    assert np.array_equal(a_up, Wup[shard.owned_neurons(9, block, 1, world)]) and np.array_equal(a_dn, a_up.T)
