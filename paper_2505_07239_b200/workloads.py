"""Seeded synthetic workloads for the sparse secret-shared FFN path.

This module only *draws inputs*: plaintext activations and weights, their
fixed-point encodings, uniformly random additive shares, block masks with the
structure of each benchmark configuration, and the dealer's Beaver triples.
It holds none of the protocol's arithmetic (no masking, no Eq. 1, no
truncation); both the CPU oracle used by the tests and the CUDA library are
fed from here and otherwise share nothing.

All matrices are produced in the paper's mathematical shapes (X [T, d],
W1 [d, D], W2 [D, d], B [K, N]); `lib_layout` transposes the right-hand
operands into the output-feature-major layout the CUDA library stores.

Random numbers come from a counter-based generator defined here: word number
`c` of stream `s` under master seed `m` is finalise(m, s, c), so any tensor can
be regenerated independently of every other.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import numpy as np

U64 = np.uint64
_MASK64 = (1 << 64) - 1


# ---------------------------------------------------------------------------
# counter-based generator
# ---------------------------------------------------------------------------
def _stream_id(name: str) -> int:
    """Deterministic 64-bit id of a stream name (multiply-xor over the bytes)."""
    h = 0x243F6A8885A308D3
    for ch in name.encode():
        h = ((h ^ ch) * 0x100000001B3 + 0x9E3779B97F4A7C15) & _MASK64
        h ^= h >> 29
    return h


def _finalise(z: np.ndarray) -> np.ndarray:
    """Bijective 64-bit finaliser: two xor-shift-multiply rounds and a last xor-shift."""
    with np.errstate(over="ignore"):
        z = (z ^ (z >> U64(30))) * U64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> U64(27))) * U64(0x94D049BB133111EB)
        z = z ^ (z >> U64(31))
    return z


def random_u64(seed: int, stream: str, count: int, offset: int = 0) -> np.ndarray:
    """`count` uniform 64-bit words of stream `stream` under master seed `seed`."""
    sid = _stream_id(stream)
    base = (sid * 0xD1342543DE82EF95 + (seed & _MASK64) * 0x2545F4914F6CDD1D + 0x632BE59BD9B4E019) & _MASK64
    with np.errstate(over="ignore"):
        ctr = np.arange(offset, offset + count, dtype=U64) * U64(0x9E3779B97F4A7C15) + U64(base)
    return _finalise(_finalise(ctr) ^ U64(sid))


def random_unit(seed: int, stream: str, count: int) -> np.ndarray:
    """Uniform doubles in [0, 1) from the top 53 bits of each word."""
    return (random_u64(seed, stream, count) >> U64(11)).astype(np.float64) * (1.0 / (1 << 53))


def random_normal(seed: int, stream: str, count: int, sigma: float) -> np.ndarray:
    """N(0, sigma) by the polar-free Box-Muller transform on two uniform streams."""
    u1 = random_unit(seed, stream + "/bm1", count)
    u2 = random_unit(seed, stream + "/bm2", count)
    r = np.sqrt(-2.0 * np.log(1.0 - u1))
    return sigma * r * np.cos(2.0 * math.pi * u2)


# ---------------------------------------------------------------------------
# fixed point and sharing (data preparation by the data owner / model owner)
# ---------------------------------------------------------------------------
def encode(v: np.ndarray, frac_bits: int) -> np.ndarray:
    """Real -> ring: round(v * 2^f) as a two's-complement 64-bit word."""
    return np.floor(v * float(1 << frac_bits) + 0.5).astype(np.int64).view(U64)


def decode(u: np.ndarray, frac_bits: int) -> np.ndarray:
    """Ring -> real: signed interpretation divided by 2^f."""
    return np.ascontiguousarray(u).view(np.int64).astype(np.float64) / float(1 << frac_bits)


def split_shares(value: np.ndarray, seed: int, stream: str):
    """Additive sharing: share 0 uniform, share 1 = value - share 0 (mod 2^64)."""
    s0 = random_u64(seed, stream + "/share0", value.size).reshape(value.shape)
    with np.errstate(over="ignore"):
        s1 = value - s0
    return s0, s1


# ---------------------------------------------------------------------------
# configurations
# ---------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class FFNConfig:
    name: str
    tokens: int
    d_model: int
    d_ff: int
    block: int
    frac_bits: int
    gated: bool
    active_fraction: float
    mask_kind: str            # "uniform" | "runs" | "pool_union"
    x_dist: str               # "uniform" | "normal"
    w_dist: str               # "uniform" | "normal0.02"
    steps: int = 1            # decode: number of single-token steps, fresh mask each
    stacked: int = 0          # weight matrices stacked in the up-projection; 0 = 2 if gated else 1

    @property
    def n_blocks(self) -> int:
        return self.d_ff // self.block

    @property
    def groups(self) -> int:
        return self.stacked if self.stacked else (2 if self.gated else 1)

    def n_active_blocks(self, sparsity: Optional[float] = None) -> int:
        p = self.active_fraction if sparsity is None else 1.0 - sparsity
        return max(1, int(math.floor(p * self.n_blocks + 0.5)))


CONFIGS: Dict[str, FFNConfig] = {
    "tiny": FFNConfig("tiny", 16, 256, 1024, 32, 12, False, 0.10, "uniform", "uniform", "uniform"),
    "opt125m": FFNConfig("opt125m", 128, 768, 3072, 32, 13, False, 0.10, "runs", "normal", "normal0.02"),
    "opt1.3b": FFNConfig("opt1.3b", 512, 2048, 8192, 32, 16, False, 0.10, "uniform", "normal", "normal0.02"),
    "llama7b": FFNConfig("llama7b", 256, 4096, 11008, 64, 16, True, 0.15, "pool_union", "normal", "normal0.02"),
    "opt6.7b-decode": FFNConfig("opt6.7b-decode", 32, 4096, 16384, 32, 16, False, 0.08, "uniform", "normal",
                                "normal0.02", steps=64),
}
SWEEP_SPARSITIES = (0.0, 0.5, 0.8, 0.9, 0.95)


# ---------------------------------------------------------------------------
# block masks
# ---------------------------------------------------------------------------
def _choose_k(seed: int, stream: str, population: int, k: int) -> np.ndarray:
    keys = random_u64(seed, stream, population)
    return np.sort(np.argsort(keys, kind="stable")[:k])


def block_mask(cfg: FFNConfig, seed: int, sparsity: Optional[float] = None, step: int = 0) -> np.ndarray:
    """0/1 byte per block, with the structure the configuration names."""
    nb = cfg.n_blocks
    k = cfg.n_active_blocks(sparsity)
    tag = f"{cfg.name}/mask/s{sparsity}/step{step}"
    m = np.zeros(nb, dtype=np.uint8)
    if cfg.mask_kind == "uniform":
        m[_choose_k(seed, tag, nb, k)] = 1
    elif cfg.mask_kind == "runs":
        # runs of active blocks: uniform start among free blocks, length
        # Geometric(1/4) on {1,2,...} (mean 4), clipped by occupied blocks,
        # the end of the layer and the remaining budget
        u = random_unit(seed, tag + "/runs", 4 * nb + 16)
        pos = 0
        placed = 0
        while placed < k:
            free = np.flatnonzero(m == 0)
            start = int(free[int(u[pos] * len(free))])
            length = 1 + int(math.floor(math.log(1.0 - u[pos + 1]) / math.log(0.75)))
            pos += 2
            b = start
            while b < nb and m[b] == 0 and length > 0 and placed < k:
                m[b] = 1
                b += 1
                length -= 1
                placed += 1
    elif cfg.mask_kind == "pool_union":
        # candidate pool of exactly k blocks; each token activates a pool block
        # with probability 0.05; the layer mask is the union over tokens
        pool = _choose_k(seed, tag + "/pool", nb, k)
        u = random_unit(seed, tag + "/tok", cfg.tokens * k).reshape(cfg.tokens, k)
        hit = (u < 0.05).any(axis=0)
        m[pool[hit]] = 1
        if not m.any():
            m[pool[0]] = 1
    else:
        raise ValueError(cfg.mask_kind)
    return m


def active_neurons(mask: np.ndarray, block: int) -> np.ndarray:
    """Ascending neuron indices of the active blocks (for building inputs only)."""
    blocks = np.flatnonzero(mask)
    return (blocks[:, None] * block + np.arange(block)[None, :]).reshape(-1).astype(np.int32)


# ---------------------------------------------------------------------------
# plaintext tensors and their shares
# ---------------------------------------------------------------------------
def _draw(dist: str, seed: int, stream: str, shape) -> np.ndarray:
    count = int(np.prod(shape))
    if dist == "uniform":
        return (2.0 * random_unit(seed, stream, count) - 1.0).reshape(shape)
    if dist == "normal":
        return random_normal(seed, stream, count, 1.0).reshape(shape)
    if dist == "normal0.02":
        return random_normal(seed, stream, count, 0.02).reshape(shape)
    raise ValueError(dist)


def model_shares(cfg: FFNConfig, seed: int, plain: bool = True) -> dict:
    """Weights of one FFN: encoded ring values and the two shares of each.

    Returns {"W1": (ring, s0, s1), "WG": ... (gated only), "W2": ...} in
    mathematical shapes W1/WG [d, D], W2 [D, d].  With plain=False the weights
    are not drawn from their distribution at all: the shares themselves are
    uniform words (their sum is then an arbitrary ring element), which is all
    a timing run or a share-parity test needs, and is much cheaper.
    """
    out = {}
    names = [("W1", (cfg.d_model, cfg.d_ff)), ("W2", (cfg.d_ff, cfg.d_model))]
    if cfg.groups >= 2:
        names.insert(1, ("WG", (cfg.d_model, cfg.d_ff)))
    if cfg.groups == 3:
        names.append(("W3", (cfg.d_model, cfg.d_ff)))
    for name, shape in names:
        if plain:
            ring = encode(_draw(cfg.w_dist, seed, f"{cfg.name}/{name}", shape), cfg.frac_bits)
            s0, s1 = split_shares(ring, seed, f"{cfg.name}/{name}")
        else:
            count = int(np.prod(shape))
            s0 = random_u64(seed, f"{cfg.name}/{name}/share0", count).reshape(shape)
            s1 = random_u64(seed, f"{cfg.name}/{name}/share1", count).reshape(shape)
            with np.errstate(over="ignore"):
                ring = s0 + s1
        out[name] = (ring, s0, s1)
    return out


def activation_shares(cfg: FFNConfig, seed: int, step: int = 0, tokens: Optional[int] = None):
    """Input activations X [T, d]: (ring, share0, share1)."""
    T = cfg.tokens if tokens is None else tokens
    ring = encode(_draw(cfg.x_dist, seed, f"{cfg.name}/X/step{step}", (T, cfg.d_model)), cfg.frac_bits)
    s0, s1 = split_shares(ring, seed, f"{cfg.name}/X/step{step}")
    return ring, s0, s1


def hidden_shares(cfg: FFNConfig, seed: int, n_active: int, step: int = 0, tokens: Optional[int] = None):
    """A synthetic post-activation hidden state [T, n] for exercising the
    down-projection alone: |N(0,1)| with about half the entries zero, encoded
    and shared.  (The end-to-end tests derive the hidden state from the
    up-projection instead.)"""
    T = cfg.tokens if tokens is None else tokens
    v = _draw("normal", seed, f"{cfg.name}/H/step{step}", (T, n_active))
    ring = encode(np.maximum(v, 0.0), cfg.frac_bits)
    s0, s1 = split_shares(ring, seed, f"{cfg.name}/H/step{step}")
    return ring, s0, s1


def ring_matmul(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """Exact product mod 2^64 of two uint64 matrices (library integer matmul)."""
    try:
        import torch

        ta = torch.from_numpy(np.ascontiguousarray(a).view(np.int64))
        tb = torch.from_numpy(np.ascontiguousarray(b).view(np.int64))
        return (ta @ tb).numpy().view(U64)
    except ImportError:  # pragma: no cover
        with np.errstate(over="ignore"):
            return a @ b


def dealer_triple(seed: int, stream: str, rows: int, inner: int, cols: int, valid: bool = True) -> dict:
    """Matrix Beaver triple for one [rows, inner] x [inner, cols] product.

    A, B uniform; C = A B mod 2^64; each split into two uniform shares.  With
    valid=False the C shares are just uniform words (no product is formed):
    share-by-share parity and timing do not need c = ab, only the
    reconstruction checks do.
    """
    A = random_u64(seed, stream + "/A", rows * inner).reshape(rows, inner)
    B = random_u64(seed, stream + "/B", inner * cols).reshape(inner, cols)
    A0, A1 = split_shares(A, seed, stream + "/A")
    B0, B1 = split_shares(B, seed, stream + "/B")
    if valid:
        C = ring_matmul(A, B)
        C0, C1 = split_shares(C, seed, stream + "/C")
    else:
        C = None
        C0 = random_u64(seed, stream + "/C/share0", rows * cols).reshape(rows, cols)
        C1 = random_u64(seed, stream + "/C/share1", rows * cols).reshape(rows, cols)
    return {"A": (A, A0, A1), "B": (B, B0, B1), "C": (C, C0, C1)}


def token_block_masks(seed: int, stream: str, tokens: int, n_blocks: int, p_token: float) -> np.ndarray:
    """Per-token 0/1 masks over `n_blocks` active blocks, each entry Bernoulli(p_token), repaired so that every
    block keeps at least one token (the block mask is the union of the token masks) and every token at least one
    block.  uint8 [tokens, n_blocks]."""
    u = random_unit(seed, stream, tokens * n_blocks).reshape(tokens, n_blocks)
    m = (np.abs(u) < p_token).astype(np.uint8)
    pick_t = random_u64(seed, stream + "/fix_t", n_blocks) % np.uint64(tokens)
    pick_b = random_u64(seed, stream + "/fix_b", tokens) % np.uint64(max(1, n_blocks))
    for b in np.nonzero(m.sum(axis=0) == 0)[0]:
        m[int(pick_t[b]), b] = 1
    for t in np.nonzero(m.sum(axis=1) == 0)[0]:
        m[t, int(pick_b[t])] = 1
    return m


def token_block_masks_clustered(seed: int, stream: str, tokens: int, n_blocks: int, clusters: int, p_token: float,
                                dead_tokens: int = 0, dead_blocks: int = 0) -> np.ndarray:
    """Per-token masks whose bipartite graph falls into (at least) `clusters` connected components: a batch that
    mixes requests with disjoint sets of active blocks.  Every token and every block is dealt to one cluster at
    random (so the members of a cluster are scattered over the index range); inside a cluster entries are
    Bernoulli(p_token), repaired so that every token has a block and every block a token of its cluster.  The first
    `dead_tokens` tokens and `dead_blocks` blocks of a seeded shuffle get no entry at all.  uint8 [tokens, n_blocks]."""
    tc = (random_u64(seed, stream + "/tc", tokens) % np.uint64(clusters)).astype(np.int64)
    bc = (random_u64(seed, stream + "/bc", n_blocks) % np.uint64(clusters)).astype(np.int64)
    bc[np.argsort(random_u64(seed, stream + "/bseed", n_blocks), kind="stable")[:min(clusters, n_blocks)]] = \
        np.arange(min(clusters, n_blocks))                       # every cluster owns a block when there are enough
    tc[np.argsort(random_u64(seed, stream + "/tseed", tokens), kind="stable")[:min(clusters, tokens)]] = \
        np.arange(min(clusters, tokens))
    u = random_unit(seed, stream, tokens * n_blocks).reshape(tokens, n_blocks)
    same = tc[:, None] == bc[None, :]
    m = ((np.abs(u) < p_token) & same).astype(np.uint8)
    rank = random_u64(seed, stream + "/fix", tokens * n_blocks).reshape(tokens, n_blocks) >> np.uint64(1)
    rank = np.where(same, rank, np.uint64(0xFFFFFFFFFFFFFFFF))
    for t in np.nonzero(m.sum(axis=1) == 0)[0]:
        m[t, int(np.argmin(rank[t]))] = 1
    for b in np.nonzero(m.sum(axis=0) == 0)[0]:
        m[int(np.argmin(rank[:, b])), b] = 1
    m[np.argsort(random_u64(seed, stream + "/dt", tokens), kind="stable")[:dead_tokens], :] = 0
    m[:, np.argsort(random_u64(seed, stream + "/db", n_blocks), kind="stable")[:dead_blocks]] = 0
    return m


def bipartite_components(S: np.ndarray):
    """Connected components of the bipartite graph rows x columns with the non-zeros of S as edges, by a library
    routine (scipy).  Returns (row_label, col_label) with -1 for nodes without an edge; labels are arbitrary."""
    from scipy.sparse import coo_matrix
    from scipy.sparse.csgraph import connected_components

    T, n = S.shape
    r, c = np.nonzero(S)
    adj = coo_matrix((np.ones(r.size, np.int8), (r, T + c)), shape=(T + n, T + n))
    _, lab = connected_components(adj, directed=False)
    row, col = lab[:T].astype(np.int64), lab[T:].astype(np.int64)
    row[~(S != 0).any(axis=1)] = -1
    col[~(S != 0).any(axis=0)] = -1
    return row, col


def dealer_triple_components(seed: int, stream: str, S: np.ndarray, inner: int) -> dict:
    """Stacked per-component triples of a SOMM product with result distribution S [rows, cols]: A [rows, inner] and
    B [inner, cols] uniform (row r / column c carry the mask of their component's triple), C = A B on the component
    blocks.  The C shares are uniformly random OFF the blocks: whoever uses them has to ignore those words."""
    rows, cols = S.shape
    A = random_u64(seed, stream + "/A", rows * inner).reshape(rows, inner)
    B = random_u64(seed, stream + "/B", inner * cols).reshape(inner, cols)
    A0, A1 = split_shares(A, seed, stream + "/A")
    B0, B1 = split_shares(B, seed, stream + "/B")
    rl, cl = bipartite_components(S)
    same = (rl[:, None] == cl[None, :]) & (rl[:, None] >= 0)
    C = np.where(same, ring_matmul(A, B), U64(0))
    C0, C1 = split_shares(C, seed, stream + "/C")
    junk = random_u64(seed, stream + "/C/junk", rows * cols).reshape(rows, cols)
    C0 = np.where(same, C0, junk)
    return {"A": (A, A0, A1), "B": (B, B0, B1), "C": (C, C0, C1), "same_component": same}


def dealer_triple_rowsets(seed: int, stream: str, S: np.ndarray, cols: int) -> dict:
    """Triple of a SIMM product whose left operand has the sparsity distribution S [rows, inner]: A' and B' uniform,
    C' = (S * A') B' (only the entries of A' on the support take part), each split into two uniform shares.  The A'
    shares are left uniformly random OFF the support too: whoever uses them has to ignore those words."""
    rows, inner = S.shape
    A = random_u64(seed, stream + "/A", rows * inner).reshape(rows, inner)
    B = random_u64(seed, stream + "/B", inner * cols).reshape(inner, cols)
    A0, A1 = split_shares(A, seed, stream + "/A")
    B0, B1 = split_shares(B, seed, stream + "/B")
    C = ring_matmul(np.where(S != 0, A, U64(0)), B)
    C0, C1 = split_shares(C, seed, stream + "/C")
    return {"A": (A, A0, A1), "B": (B, B0, B1), "C": (C, C0, C1)}


def dealer_triple_elementwise(seed: int, stream: str, shape) -> dict:
    """Element-wise Beaver triple: a, b uniform, c = a * b mod 2^64 element by element, each split into two
    uniform shares.  Returns {"a": (a, a0, a1), "b": ..., "c": ...}."""
    count = int(np.prod(shape))
    a = random_u64(seed, stream + "/a", count).reshape(shape)
    b = random_u64(seed, stream + "/b", count).reshape(shape)
    with np.errstate(over="ignore"):
        c = a * b
    return {"a": (a, *split_shares(a, seed, stream + "/a")), "b": (b, *split_shares(b, seed, stream + "/b")),
            "c": (c, *split_shares(c, seed, stream + "/c"))}


def dealer_truncation_pair(seed: int, stream: str, shape, frac_bits: int) -> dict:
    """The dealer's pair for one truncation by `frac_bits`: r uniform in the ring and r' = floor(r / 2^f) with r
    read as a signed 64-bit integer, each split into two uniform shares.  Returns {"r": (r, r0, r1), "rp": ...}."""
    count = int(np.prod(shape))
    r = random_u64(seed, stream + "/r", count).reshape(shape)
    rp = (r.view(np.int64) >> np.int64(frac_bits)).view(np.uint64)
    return {"r": (r, *split_shares(r, seed, stream + "/r")), "rp": (rp, *split_shares(rp, seed, stream + "/rp"))}


def random_permutation(seed: int, stream: str, count: int) -> np.ndarray:
    """Seeded uniform permutation of range(count) (rank of random keys), int32."""
    keys = random_u64(seed, stream, count)
    return np.argsort(keys, kind="stable").astype(np.int32)


def dealer_shuffle(seed: int, stream: str, rows: int, cols: int, inverse_of: Optional[dict] = None) -> dict:
    """What the trusted dealer hands out for one oblivious shuffle of the rows of a
    [rows, cols] matrix (Protocol 1, offline stage): pi, (tau_0, tau_1), (rho_0, rho_1)
    with pi = rho_0 o tau_1 = rho_1 o tau_0, masks (a_0, a_1), (b_0, b_1).
    A permutation p acts as (p(x))[j] = x[p[j]].

    With `inverse_of` (the material of an earlier shuffle) the sub-permutations are the
    ones each party derives locally to undo that shuffle, tau'_i = rho_i^{-1} and
    rho'_i = tau_i^{-1}; the masks are fresh.
    """
    def inv(p):
        out = np.empty_like(p)
        out[p] = np.arange(p.size, dtype=np.int32)
        return out

    if inverse_of is None:
        pi = random_permutation(seed, stream + "/pi", rows)
        tau = (random_permutation(seed, stream + "/tau0", rows), random_permutation(seed, stream + "/tau1", rows))
        # rho_0 = pi o tau_1^{-1}: (p o q)[j] = q[p[j]]
        rho = (inv(tau[1])[pi], inv(tau[0])[pi])
    else:
        tau = (inv(inverse_of["rho"][0]), inv(inverse_of["rho"][1]))
        rho = (inv(inverse_of["tau"][0]), inv(inverse_of["tau"][1]))
        pi = inv(inverse_of["pi"])
    a = tuple(random_u64(seed, stream + f"/a{i}", rows * cols).reshape(rows, cols) for i in (0, 1))
    c = random_u64(seed, stream + "/c", rows * cols).reshape(rows, cols)
    b = (a[1][rho[0]] + c, a[0][rho[1]] - c)
    return {"pi": pi, "tau": tau, "rho": rho, "a": a, "b": b, "c": c}


def reshare(value: np.ndarray, seed: int, stream: str):
    """Fresh uniform sharing of a ring tensor (used after the activation functionality)."""
    return split_shares(value, seed, stream)


def lib_layout(right_operand: np.ndarray) -> np.ndarray:
    """[inner, cols] (paper shape) -> [cols, inner] contiguous (library storage)."""
    return np.ascontiguousarray(right_operand.T)
