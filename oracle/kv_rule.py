"""TEST INFRASTRUCTURE -- the KV-cache manager's request planning (Section 6 of the paper), plain Python.

Merging (Section 6.1): when a token is generated with some heads activated, every (token, head) entry of an
activated head that is absent from the cache is requested, all in one batch.  Prefetching (Section 6.2): a head
that is NOT activated and has L2 absent entries is added to the batch only if the communication saved later,
2*L2*x, exceeds the extra communication now, 2*(w + x*max(0, L2 - L1)), i.e. if L2 > w/x + max(0, L2 - L1), with
x the token vector size, w the size of one head's weight matrix and L1 the misses of the activated heads (read
here as the number of tokens the merged refill batch sends anyway).
"""
from __future__ import annotations

import numpy as np


def plan(present: np.ndarray, active: np.ndarray, x: int, w: int):
    """present [tokens, heads] (non-zero = cached), active [heads].  Returns (request [tokens, heads] uint8,
    prefetch [heads] uint8, L1)."""
    tokens, heads = present.shape
    request = np.zeros((tokens, heads), np.uint8)
    for h in range(heads):
        if active[h]:
            for t in range(tokens):
                if not present[t, h]:
                    request[t, h] = 1
    L1 = int(request.any(axis=1).sum())
    prefetch = np.zeros(heads, np.uint8)
    for h in range(heads):
        if active[h]:
            continue
        L2 = int((present[:, h] == 0).sum())
        extra = 2 * (w + x * max(0, L2 - L1))
        saved = 2 * L2 * x
        if saved > extra:
            prefetch[h] = 1
            for t in range(tokens):
                if not present[t, h]:
                    request[t, h] = 1
    return request, prefetch, L1
