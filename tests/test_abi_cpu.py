"""CPU-only checks of the C ABI: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching a GPU."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def cb():
    from paper_2505_07239_b200.build import build_library

    build_library()
    from paper_2505_07239_b200 import binding

    return binding


def test_every_declared_symbol_is_exported(cb):
    header = open(os.path.join(ROOT, "include", "comet.h")).read()
    declared = set(re.findall(r"\b(comet_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(cb.library(), name), name
    assert declared == set(cb.EXPORTS) | declared          # binding lists nothing the header lacks
    assert set(cb.EXPORTS) <= declared


def test_strerror_and_codes(cb):
    lib = cb.library()
    assert lib.comet_strerror(0) == b"ok"
    seen = {lib.comet_strerror(-k) for k in range(1, 7)}
    assert len(seen) == 6 and b"unknown error code" not in seen
    assert lib.comet_strerror(-99) == b"unknown error code"


def test_init_validates_before_any_cuda_call(cb):
    lib = cb.library()
    h = ctypes.c_void_p()
    assert lib.comet_init(None, None, ctypes.byref(h)) == -1
    good = dict(max_tokens=16, d_model=256, d_ff=1024, block=32, frac_bits=12, gated=0, device=0, max_active=0,
                matmul_path=0)
    bad = [
        (dict(good, gated=3), -1), (dict(good, gated=-1), -1), (dict(good, matmul_path=7), -1), (dict(good, device=-1), -1),
        (dict(good, max_tokens=0), -2), (dict(good, d_model=250), -2), (dict(good, d_ff=1000), -2),
        (dict(good, block=8), -2), (dict(good, block=24), -2), (dict(good, frac_bits=0), -2),
        (dict(good, frac_bits=32), -2), (dict(good, max_active=48), -2), (dict(good, max_active=2048), -2),
    ]
    for kw, code in bad:
        cfg = cb.CometConfig(**kw)
        assert lib.comet_init(ctypes.byref(cfg), None, ctypes.byref(h)) == code, kw
        assert not h.value


def test_null_context_is_rejected(cb):
    lib = cb.library()
    n = ctypes.c_int32()
    assert lib.comet_ffn_up(None, 4) == -1
    assert lib.comet_ffn_down(None, 4) == -1
    assert lib.comet_truncate(None, cb.Z_UP) == -1
    assert lib.comet_set_mask(None, None, 0, 4, ctypes.byref(n)) == -1
    assert lib.comet_load_shares(None, 0, cb.X, None, 0, 1, 1) == -1
    assert lib.comet_stats(None, None) == -1
    lib.comet_destroy(None)
