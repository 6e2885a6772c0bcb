"""TEST INFRASTRUCTURE -- plaintext references that sit around the secret-shared path.

* `activation`: the ideal functionality standing in for the secure non-linear
  layer between the two projections (Section 3.3: the non-linear protocol is
  unchanged and only sees the active entries).  It reconstructs, applies ReLU
  (or ReLU(gate) * up for the ReLU-fied gated FFN of Section 7.1) in the ring's
  signed interpretation, and returns the plaintext ring value to be re-shared.
* `plain_ffn_float64`: the float64 masked FFN the decoded result is compared to.
* `plain_ffn_integer`: the same FFN on unshared ring integers with exact floor
  truncations, i.e. what the shares would reconstruct to without the +1 ulp
  of local truncation.
"""
from __future__ import annotations

import numpy as np

U64 = np.uint64


def _signed(u: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(u).view(np.int64)


def activation(H0: np.ndarray, H1: np.ndarray, gated: bool, frac_bits: int) -> np.ndarray:
    """H0, H1: shares of the truncated up-projection, compact [T, g*n].
    Returns the plaintext ring tensor [T, n] after the activation."""
    with np.errstate(over="ignore"):
        h = _signed(H0 + H1)
    if not gated:
        return np.maximum(h, 0).view(U64)
    n = h.shape[1] // 2
    gate, up = h[:, :n], h[:, n:]
    prod = np.maximum(gate, 0) * up          # magnitudes far below 2^63
    return (prod >> np.int64(frac_bits)).view(U64)   # arithmetic shift = floor


def plain_ffn_float64(x, W1, W2, I, WG=None):
    """Masked FFN in float64 on real-valued inputs: only neurons in I exist."""
    if WG is None:
        h = np.maximum(x @ W1[:, I], 0.0)
    else:
        h = np.maximum(x @ WG[:, I], 0.0) * (x @ W1[:, I])
    return h @ W2[I, :]


def plain_ffn_integer(xr, W1r, W2r, I, frac_bits, WGr=None):
    """Masked FFN on ring integers (uint64 arrays holding two's-complement
    fixed-point values) with floor truncation after every product."""
    f = np.int64(frac_bits)
    x = _signed(xr)
    with np.errstate(over="ignore"):
        up = (x @ _signed(W1r)[:, I]) >> f
        if WGr is None:
            h = np.maximum(up, 0)
        else:
            gate = (x @ _signed(WGr)[:, I]) >> f
            h = (np.maximum(gate, 0) * up) >> f
        y = (h @ _signed(W2r)[I, :]) >> f
    return y.view(U64)
