"""Sharding one FFN layer over the neuron dimension: one process per GPU, rank r owns the mask blocks b with
b mod world == r (a static partition, so every rank stores only its slice of W1 / WG / W2).

Up-projection (Protocol 2): the active columns of the result are independent, so every rank runs its own
product over its own active neurons with its column slice of the dealer's triple; nothing is exchanged between
the ranks.  Down-projection (Protocol 3): the contraction index is the neuron, so every rank's product is a
partial sum of Eq. 1; the partial sums of each party's share are added over the ranks (addition of shares is
local in Section 2.1; here it is one integer all-reduce per party, which wraps mod 2^64 like the ring), and
only then truncated.  The triple's C' share is a summand of Eq. 1 that must enter the sum once: rank 0 loads it,
the other ranks load zeros.

This module holds the index arithmetic of that partition and the reduction call; the products themselves are
the library's.  It works on any torch.distributed backend (nccl on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import numpy as np


def owned_blocks(n_blocks: int, rank: int, world: int) -> np.ndarray:
    """Ids of the mask blocks rank `rank` owns: rank, rank + world, rank + 2 world, ..."""
    return np.arange(rank, n_blocks, world, dtype=np.int64)


def local_mask(block_mask: np.ndarray, rank: int, world: int) -> np.ndarray:
    """The rank's block mask: the global mask at the blocks it owns (its local block j is global block
    rank + j * world)."""
    return np.ascontiguousarray(np.asarray(block_mask, dtype=np.uint8)[rank::world])


def owned_neurons(n_blocks: int, block: int, rank: int, world: int) -> np.ndarray:
    """Global neuron ids of the rank's slice of d_ff, in local order."""
    b = owned_blocks(n_blocks, rank, world)
    return (b[:, None] * block + np.arange(block, dtype=np.int64)[None, :]).reshape(-1)


def local_columns(block_mask: np.ndarray, block: int, rank: int, world: int) -> np.ndarray:
    """Positions, in the GLOBAL compact order of the active neurons (ascending neuron id), of the rank's active
    neurons, in the rank's own compact order.  Slices the triples and the hidden state of the whole layer into
    the rank's: A'[:, cols], B'[cols, :], H[:, cols], B[:, cols], C[:, cols]."""
    m = np.asarray(block_mask, dtype=np.uint8) != 0
    active = np.flatnonzero(m)                       # global ids of the active blocks, ascending
    mine = np.flatnonzero(active % world == rank)    # their positions in the compact block order
    return (mine[:, None] * block + np.arange(block, dtype=np.int64)[None, :]).reshape(-1)


def slice_stored_weights(W_up_stored: np.ndarray, W2_stored: np.ndarray, block: int, rank: int, world: int):
    """The rank's slice of weights in the library's stored layout: rows of W1 / WG [d_ff, d_model], columns of
    W2 [d_model, d_ff]."""
    neurons = owned_neurons(W_up_stored.shape[0] // block, block, rank, world)
    return np.ascontiguousarray(W_up_stored[neurons, :]), np.ascontiguousarray(W2_stored[:, neurons])


def add_over_ranks(share):
    """In-place sum over all ranks of one party's partial result (a torch int64 tensor holding ring words): the
    two's-complement sum of 64-bit integers is the sum mod 2^64.  Identity for one process."""
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(share, op=dist.ReduceOp.SUM)
    return share
