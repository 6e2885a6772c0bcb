"""Pins of the oracle's truncation with a dealer's pair (built from Section 2.1's Reconstruction and Addition;
the paper itself has no truncation protocol, so the pins are closed forms, invariants and hand-made words)."""
import os

import numpy as np

import oracle
from paper_2505_07239_b200 import workloads as wl

U64 = np.uint64
MASK = (1 << 64) - 1


def _signed(v: int) -> int:
    v &= MASK
    return v - (1 << 64) if v >> 63 else v


def _arr(vals):
    return np.array([int(v) & MASK for v in vals], dtype=object).astype(U64)


def test_hand_computed_words(golden_dir):
    rows = [ln.split() for ln in open(os.path.join(golden_dir, "truncate_pair_hand_words.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 4
    for row in rows:
        f = int(row[0])
        z0, z1, r0, r1, p0, p1, m0, m1, o0, o1 = (_arr([eval(t)]) for t in row[1:])
        got = oracle.truncate_pair((z0, z1), (r0, r1), (p0, p1), f)
        assert [int(got["M"][0][0]), int(got["M"][1][0])] == [int(m0[0]), int(m1[0])], row
        assert [int(got["OUT"][0][0]), int(got["OUT"][1][0])] == [int(o0[0]), int(o1[0])], row


def _random_case(seed, count, f, magnitude_bits):
    raw = wl.random_u64(seed, "z", count)
    z = (raw.view(np.int64) >> np.int64(64 - magnitude_bits)).view(U64)       # signed, |z| < 2^(bits-1)
    pair = wl.dealer_truncation_pair(seed, "pair", (count,), f)
    return z, wl.split_shares(z, seed, "z"), pair


def test_sum_is_the_floor_or_one_less_against_python_integers():
    for f, bits in ((12, 30), (16, 40), (1, 20), (31, 45)):
        z, zs, pair = _random_case(11 + f, 4096, f, bits)
        got = oracle.truncate_pair(zs, pair["r"][1:], pair["rp"][1:], f)
        total = got["OUT"][0] + got["OUT"][1]
        diffs = set()
        for t in range(z.size):
            want = _signed(int(z[t])) >> f                         # Python's >> on integers is the floor
            diffs.add(_signed(int(total[t])) - want)
        assert diffs <= {-1, 0} and diffs == {-1, 0}, (f, diffs)    # both occur on 4096 random elements
        # the opened value is z - r
        assert np.array_equal(got["M"][0] + got["M"][1], z - pair["r"][0])


def test_zero_mask_gives_the_exact_floor():
    f, count = 13, 257
    z, zs, _ = _random_case(3, count, f, 50)
    zero = np.zeros(count, U64)
    r = wl.split_shares(zero, 3, "r")
    rp = wl.split_shares(zero, 3, "rp")
    got = oracle.truncate_pair(zs, r, rp, f)
    total = got["OUT"][0] + got["OUT"][1]
    assert [_signed(int(v)) for v in total] == [_signed(int(v)) >> f for v in z]


def test_multiples_of_the_scale_are_divided_exactly():
    f, count = 16, 300
    z, _, pair = _random_case(4, count, f, 40)
    z = (z >> U64(f)) << U64(f)                                     # low f bits zero (still the same signed range)
    r = (pair["r"][0] >> U64(f)) << U64(f)
    rp = (r.view(np.int64) >> np.int64(f)).view(U64)
    got = oracle.truncate_pair(wl.split_shares(z, 4, "z"), wl.split_shares(r, 4, "r"), wl.split_shares(rp, 4, "rp"), f)
    total = got["OUT"][0] + got["OUT"][1]
    assert [_signed(int(v)) for v in total] == [_signed(int(v)) // (1 << f) for v in z]


def test_public_term_goes_to_the_party_with_factor_i():
    # Section 2.1 "Addition": [z]_i = ... + (i-1) c for parties 1, 2, so the first party's result is its share of r'
    f = 12
    _, zs, pair = _random_case(5, 64, f, 30)
    got = oracle.truncate_pair(zs, pair["r"][1:], pair["rp"][1:], f)
    assert np.array_equal(got["OUT"][0], pair["rp"][1])
    assert not np.array_equal(got["OUT"][1], pair["rp"][2])


def test_agrees_with_the_local_truncation_within_one_unit():
    # two different protocols for the same functionality: their reconstructions differ by at most 1 + 1 units
    f = 16
    z, zs, pair = _random_case(6, 2048, f, 40)
    a = oracle.truncate_pair(zs, pair["r"][1:], pair["rp"][1:], f)["OUT"]
    b = (oracle.truncate(0, zs[0], f), oracle.truncate(1, zs[1], f))
    d = {_signed(int(x)) for x in (b[0] + b[1]) - (a[0] + a[1])}
    assert d <= {0, 1, 2}


def test_dealer_pair_is_consistent():
    pair = wl.dealer_truncation_pair(9, "p", (5, 7), 16)
    r, r0, r1 = pair["r"]
    rp, p0, p1 = pair["rp"]
    assert np.array_equal(r0 + r1, r) and np.array_equal(p0 + p1, rp)
    assert [[_signed(int(v)) for v in row] for row in rp] == [[_signed(int(v)) >> 16 for v in row] for row in r]
