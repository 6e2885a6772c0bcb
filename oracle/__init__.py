"""TEST INFRASTRUCTURE -- ctypes front end of the CPU oracle (`comet_oracle.cpp`).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares nothing with the CUDA library.  Arrays are numpy
uint64, C-contiguous, in the paper's mathematical shapes.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "comet_oracle.cpp")
_LIB = os.path.join(_HERE, "libcomet_oracle.so")
_lib = None

U64 = np.uint64


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (plain -O2, no threading, no arch flags)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-o", _LIB, _SRC])
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _p(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be C-contiguous"
    return a.ctypes.data_as(ctypes.c_void_p)


def _u64(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == U64
    return a


def reconstruct(s0, s1):
    s0, s1 = _u64(s0), _u64(s1)
    out = np.empty_like(s0)
    lib().orc_reconstruct(_p(s0), _p(s1), _p(out), ctypes.c_size_t(s0.size))
    return out


def index_set(block_mask, block: int, groups: int = 1) -> np.ndarray:
    m = np.ascontiguousarray(block_mask, dtype=np.uint8)
    I = np.empty(max(1, m.size * block * groups), dtype=np.int32)
    n = lib().orc_index_set(_p(m), ctypes.c_int(m.size), ctypes.c_int(block), ctypes.c_int(groups), _p(I))
    return I[:n].copy()


def index_cols(Y, I):
    Y = _u64(Y)
    I = np.ascontiguousarray(I, dtype=np.int32)
    K, D = Y.shape
    out = np.empty((K, I.size), dtype=U64)
    lib().orc_index_cols(_p(Y), ctypes.c_int(K), ctypes.c_int(D), _p(I), ctypes.c_int(I.size), _p(out))
    return out


def index_rows(Y, I):
    Y = _u64(Y)
    I = np.ascontiguousarray(I, dtype=np.int32)
    D, N = Y.shape
    out = np.empty((I.size, N), dtype=U64)
    lib().orc_index_rows(_p(Y), ctypes.c_int(N), _p(I), ctypes.c_int(I.size), _p(out))
    return out


def merge_cols(R, I, D: int):
    R = _u64(R)
    I = np.ascontiguousarray(I, dtype=np.int32)
    T, n = R.shape
    Z = np.empty((T, D), dtype=U64)
    lib().orc_merge_cols(_p(R), ctypes.c_int(T), ctypes.c_int(n), _p(I), ctypes.c_int(D), _p(Z))
    return Z


def mask_operand(share, mask_share):
    share, mask_share = _u64(share), _u64(mask_share)
    assert share.shape == mask_share.shape
    out = np.empty_like(share)
    lib().orc_mask_operand(_p(share), _p(mask_share), _p(out), ctypes.c_size_t(share.size))
    return out


def beaver_combine(party: int, E, F, Ai, Bi, Ci):
    E, F, Ai, Bi, Ci = map(_u64, (E, F, Ai, Bi, Ci))
    T, K = E.shape
    K2, N = F.shape
    assert K2 == K and Ai.shape == (T, K) and Bi.shape == (K, N) and Ci.shape == (T, N)
    Z = np.empty((T, N), dtype=U64)
    lib().orc_beaver_combine(ctypes.c_int(party), ctypes.c_int(T), ctypes.c_int(K), ctypes.c_int(N),
                             _p(E), _p(F), _p(Ai), _p(Bi), _p(Ci), _p(Z))
    return Z


def beaver_combine_at(party: int, E, F, Ai, Bi, Ci, rows, cols):
    E, F, Ai, Bi, Ci = map(_u64, (E, F, Ai, Bi, Ci))
    T, K = E.shape
    _, N = F.shape
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    cols = np.ascontiguousarray(cols, dtype=np.int32)
    out = np.empty(rows.size, dtype=U64)
    lib().orc_beaver_combine_at(ctypes.c_int(party), ctypes.c_int(K), ctypes.c_int(N),
                                _p(E), _p(F), _p(Ai), _p(Bi), _p(Ci),
                                ctypes.c_int(rows.size), _p(rows), _p(cols), _p(out))
    return out


def _pairs(*pairs):
    flat = []
    for s0, s1 in pairs:
        flat += [_u64(s0), _u64(s1)]
    return flat


def pi_matmul(X, Y, A, B, C):
    """Both parties of Pi_MatMul.  Each argument is a pair (share0, share1).
    Returns dict with E, F, Z pairs."""
    X0, X1, Y0, Y1, A0, A1, B0, B1, C0, C1 = _pairs(X, Y, A, B, C)
    T, K = X0.shape
    _, N = Y0.shape
    E0, E1 = np.empty((T, K), U64), np.empty((T, K), U64)
    F0, F1 = np.empty((K, N), U64), np.empty((K, N), U64)
    Z0, Z1 = np.empty((T, N), U64), np.empty((T, N), U64)
    lib().orc_pi_matmul(ctypes.c_int(T), ctypes.c_int(K), ctypes.c_int(N),
                        *[_p(a) for a in (X0, X1, Y0, Y1, A0, A1, B0, B1, C0, C1, E0, E1, F0, F1, Z0, Z1)])
    return {"E": (E0, E1), "F": (F0, F1), "Z": (Z0, Z1)}


def somm(X, Y, I, A, B, C):
    """Protocol 2 with a token-shared mask.  Y pair is [K, Dy]; I indexes its
    columns.  Returns compact messages and result: E [T,K], F [K,n], R [T,n]."""
    X0, X1, Y0, Y1, A0, A1, B0, B1, C0, C1 = _pairs(X, Y, A, B, C)
    I = np.ascontiguousarray(I, dtype=np.int32)
    T, K = X0.shape
    _, Dy = Y0.shape
    n = I.size
    assert A0.shape == (T, K) and B0.shape == (K, n) and C0.shape == (T, n)
    E0, E1 = np.empty((T, K), U64), np.empty((T, K), U64)
    F0, F1 = np.empty((K, n), U64), np.empty((K, n), U64)
    R0, R1 = np.empty((T, n), U64), np.empty((T, n), U64)
    lib().orc_somm(ctypes.c_int(T), ctypes.c_int(K), ctypes.c_int(Dy), _p(I), ctypes.c_int(n),
                   *[_p(a) for a in (X0, X1, Y0, Y1, A0, A1, B0, B1, C0, C1, E0, E1, F0, F1, R0, R1)])
    return {"E": (E0, E1), "F": (F0, F1), "Z": (R0, R1)}


def simm(X, Y, I, A, B, C):
    """Protocol 3 with a token-shared mask.  X pair is compact [T,n]; Y pair is
    [D, N]; I lists the neuron of each compact column.  Returns E [T,n],
    F [n,N], Z [T,N]."""
    X0, X1, Y0, Y1, A0, A1, B0, B1, C0, C1 = _pairs(X, Y, A, B, C)
    I = np.ascontiguousarray(I, dtype=np.int32)
    T, n = X0.shape
    _, N = Y0.shape
    assert I.size == n and A0.shape == (T, n) and B0.shape == (n, N) and C0.shape == (T, N)
    E0, E1 = np.empty((T, n), U64), np.empty((T, n), U64)
    F0, F1 = np.empty((n, N), U64), np.empty((n, N), U64)
    Z0, Z1 = np.empty((T, N), U64), np.empty((T, N), U64)
    lib().orc_simm(ctypes.c_int(T), ctypes.c_int(n), ctypes.c_int(N), _p(I),
                   *[_p(a) for a in (X0, X1, Y0, Y1, A0, A1, B0, B1, C0, C1, E0, E1, F0, F1, Z0, Z1)])
    return {"E": (E0, E1), "F": (F0, F1), "Z": (Z0, Z1)}


def components_dfs(S):
    """Connected components of the bipartite graph of S [T, n] (the first step of Protocol 2).
    Returns (row_comp [T], col_comp [n], L); -1 marks a node without an edge."""
    S = np.ascontiguousarray(S, dtype=np.uint8)
    T, n = S.shape
    rc, cc = np.empty(T, np.int32), np.empty(n, np.int32)
    L = lib().orc_components_dfs(ctypes.c_int(T), ctypes.c_int(n), _p(S), _p(rc), _p(cc))
    return rc, cc, int(L)


def somm_components(X, Y, I, S, A, B, C):
    """Protocol 2 over the connected components of S [T, n].  Y pair is [K, Dy]; I maps compact columns to
    columns of Y; A [T,K], B [K,n], C [T,n] hold the per-component triples stacked.  Returns compact E [T,K],
    F [K,n], Z [T,n] (zero outside the component blocks), the partition and the cost counters."""
    X0, X1, Y0, Y1, A0, A1, B0, B1, C0, C1 = _pairs(X, Y, A, B, C)
    I = np.ascontiguousarray(I, dtype=np.int32)
    S = np.ascontiguousarray(S, dtype=np.uint8)
    T, K = X0.shape
    _, Dy = Y0.shape
    n = I.size
    assert S.shape == (T, n) and A0.shape == (T, K) and B0.shape == (K, n) and C0.shape == (T, n)
    E0, E1 = np.empty((T, K), U64), np.empty((T, K), U64)
    F0, F1 = np.empty((K, n), U64), np.empty((K, n), U64)
    R0, R1 = np.empty((T, n), U64), np.empty((T, n), U64)
    rc, cc = np.empty(T, np.int32), np.empty(n, np.int32)
    cost = np.zeros(2, np.int64)
    L = lib().orc_somm_components(ctypes.c_int(T), ctypes.c_int(K), ctypes.c_int(Dy), _p(I), ctypes.c_int(n), _p(S),
                                  *[_p(a) for a in (X0, X1, Y0, Y1, A0, A1, B0, B1, C0, C1, E0, E1, F0, F1, R0, R1)],
                                  _p(rc), _p(cc), _p(cost))
    return {"E": (E0, E1), "F": (F0, F1), "Z": (R0, R1), "row_comp": rc, "col_comp": cc, "L": int(L),
            "masked_nodes": int(cost[0]), "dot_products": int(cost[1])}


def simm_rowsets(X, Y, I, S, A, B, C):
    """Protocol 3 with per-column row sets: S is the [T, n] sparsity distribution of the compact X
    (non-zero = present).  Returns E [T,n] (zero off the support), F [n,N], Z [T,N] and the number of
    masked entries of X."""
    X0, X1, Y0, Y1, A0, A1, B0, B1, C0, C1 = _pairs(X, Y, A, B, C)
    I = np.ascontiguousarray(I, dtype=np.int32)
    S = np.ascontiguousarray(S, dtype=np.uint8)
    T, n = X0.shape
    _, N = Y0.shape
    assert I.size == n and S.shape == (T, n) and A0.shape == (T, n) and B0.shape == (n, N) and C0.shape == (T, N)
    E0, E1 = np.empty((T, n), U64), np.empty((T, n), U64)
    F0, F1 = np.empty((n, N), U64), np.empty((n, N), U64)
    Z0, Z1 = np.empty((T, N), U64), np.empty((T, N), U64)
    lib().orc_simm_rowsets.restype = ctypes.c_longlong
    masked = lib().orc_simm_rowsets(ctypes.c_int(T), ctypes.c_int(n), ctypes.c_int(N), _p(I), _p(S),
                                    *[_p(a) for a in (X0, X1, Y0, Y1, A0, A1, B0, B1, C0, C1, E0, E1, F0, F1, Z0, Z1)])
    return {"E": (E0, E1), "F": (F0, F1), "Z": (Z0, Z1), "masked": int(masked)}


def truncate(party: int, Z, frac_bits: int):
    Z = _u64(Z)
    out = np.empty_like(Z)
    lib().orc_truncate(ctypes.c_int(party), _p(Z), _p(out), ctypes.c_size_t(Z.size), ctypes.c_int(frac_bits))
    return out


# ---------------------------------------------------------------------------
# Oblivious shuffle (Protocol 1).  Permutations are int32 index arrays acting on
# the rows of [rows, cols] uint64 matrices: (pi(x))[j] = x[pi[j]].
# ---------------------------------------------------------------------------
def _perm(p) -> np.ndarray:
    p = np.ascontiguousarray(p, dtype=np.int32)
    assert p.ndim == 1
    return p


def _rows2d(x) -> np.ndarray:
    x = _u64(x)
    return x.reshape(x.shape[0], -1)


def apply_permutation(perm, x):
    perm, x2 = _perm(perm), _rows2d(x)
    out = np.empty_like(x2)
    lib().orc_apply_permutation(_p(perm), _p(x2), _p(out), ctypes.c_int(x2.shape[0]), ctypes.c_int(x2.shape[1]))
    return out.reshape(np.shape(x))


def compose_permutations(p, q):
    """p o q as operators: (p o q)(x) = p(q(x))."""
    p, q = _perm(p), _perm(q)
    out = np.empty_like(p)
    lib().orc_compose_permutations(_p(p), _p(q), _p(out), ctypes.c_int(p.size))
    return out


def invert_permutation(p):
    p = _perm(p)
    out = np.empty_like(p)
    lib().orc_invert_permutation(_p(p), _p(out), ctypes.c_int(p.size))
    return out


def shuffle_offline(pi, tau, a, c):
    """Offline stage: tau = (tau_0, tau_1), a = (a_0, a_1), c the dealer's random
    matrix.  Returns rho = (rho_0, rho_1), b = (b_0, b_1)."""
    pi, t0, t1 = _perm(pi), _perm(tau[0]), _perm(tau[1])
    a0, a1, c2 = _rows2d(a[0]), _rows2d(a[1]), _rows2d(c)
    rows, cols = a0.shape
    r0, r1 = np.empty_like(pi), np.empty_like(pi)
    b0, b1 = np.empty_like(a0), np.empty_like(a0)
    lib().orc_shuffle_offline(ctypes.c_int(rows), ctypes.c_int(cols), _p(pi), _p(t0), _p(t1), _p(a0), _p(a1), _p(c2),
                              _p(r0), _p(r1), _p(b0), _p(b1))
    shape = np.shape(a[0])
    return (r0, r1), (b0.reshape(shape), b1.reshape(shape))


def shuffle_online(x, tau, rho, a, b):
    """Online stage for both parties.  Returns messages y = (y_0, y_1) and results z = (z_0, z_1)."""
    x0, x1 = _rows2d(x[0]), _rows2d(x[1])
    rows, cols = x0.shape
    arrs = [_perm(tau[0]), _perm(tau[1]), _perm(rho[0]), _perm(rho[1]),
            _rows2d(a[0]), _rows2d(a[1]), _rows2d(b[0]), _rows2d(b[1])]
    outs = [np.empty_like(x0) for _ in range(4)]
    lib().orc_shuffle_online(ctypes.c_int(rows), ctypes.c_int(cols), _p(x0), _p(x1), *[_p(v) for v in arrs],
                             *[_p(o) for o in outs])
    shape = np.shape(x[0])
    y0, y1, z0, z1 = (o.reshape(shape) for o in outs)
    return (y0, y1), (z0, z1)


def beaver_mul(x, y, a, b, c):
    """Element-wise Beaver product of Eq. 1 for both parties.  Every argument is a pair of
    equally shaped uint64 arrays.  Returns dict with the messages D, E and the result Z (pairs)."""
    arrs = _pairs(x, y, a, b, c)
    shape = arrs[0].shape
    for v in arrs:
        assert v.shape == shape
    outs = [np.empty(shape, U64) for _ in range(6)]
    lib().orc_beaver_mul(ctypes.c_size_t(arrs[0].size), *[_p(v) for v in arrs], *[_p(o) for o in outs])
    return {"D": (outs[0], outs[1]), "E": (outs[2], outs[3]), "Z": (outs[4], outs[5])}


def truncate_pair(z, r, rp, frac_bits: int):
    """Truncation with a dealer's pair (r, r' = floor(r / 2^f)) for both parties: z, r, rp are pairs of
    equally shaped uint64 arrays.  Returns dict with the messages M = z - r (pair) and the result OUT (pair)."""
    arrs = _pairs(z, r, rp)
    shape = arrs[0].shape
    for v in arrs:
        assert v.shape == shape
    outs = [np.empty(shape, U64) for _ in range(4)]
    lib().orc_truncate_pair(ctypes.c_size_t(arrs[0].size), ctypes.c_int(frac_bits), *[_p(v) for v in arrs],
                            *[_p(o) for o in outs])
    return {"M": (outs[0], outs[1]), "OUT": (outs[2], outs[3])}


def add_bias(Zi, bias_i):
    """One party's local addition of its bias share [N] to every row of its share [T, N]."""
    Zi, bias_i = _u64(Zi), _u64(bias_i)
    T, N = Zi.shape
    assert bias_i.shape == (N,)
    out = np.empty_like(Zi)
    lib().orc_add_bias(ctypes.c_int(T), ctypes.c_int(N), _p(Zi), _p(bias_i), _p(out))
    return out
