"""Thin ctypes binding of libcomet_b200.so (the C ABI of include/comet.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  Tensors are torch uint64/int64 CUDA tensors or numpy/torch host
arrays; torch is used for device memory and streams and for nothing else.
There is no CPU fallback: if the shared library is missing or fails to load,
importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np
import torch

from .build import LIB_PATH, build_library, is_current

OK = 0
DEVICE, HOST = 0, 1
PATH_AUTO, PATH_SIMT, PATH_LIMB = 0, 1, 2

(X, W1, WG, W2, A_UP, B_UP, C_UP, H, A_DN, B_DN, C_DN,
 E_UP, F_UP, Z_UP, E_DN, F_DN, Y, W3) = range(18)
NUM_TENSORS = 18

EXPORTS = (
    "comet_init", "comet_destroy", "comet_load_shares", "comet_set_mask", "comet_ffn_up", "comet_ffn_down",
    "comet_truncate", "comet_get", "comet_get_index", "comet_stats", "comet_strerror", "comet_last_cuda_error",
    "comet_set_profiling", "comet_beaver_matmul_static", "comet_shuffle", "comet_invert_permutation",
    "comet_beaver_mul", "comet_set_token_mask", "comet_get_components", "comet_kv_plan",
    "comet_add_bias", "comet_bind_shares", "comet_truncate_pair", "comet_synchronize", "comet_inject_timeout",
    "comet_pipe_probe", "comet_device_pointer",
)
STATIC_SCRATCH_WORDS = 1 << 20
ERR_SCRATCH_LIMIT = -7
ERR_TIMEOUT = -6
NUM_PHASES = 5
PHASE_NAMES = ("compact", "open", "prep", "combine", "truncate")


class CometConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "max_tokens", "d_model", "d_ff", "block", "frac_bits", "gated", "device", "max_active", "matmul_path")]


class CometStats(ctypes.Structure):
    _fields_ = [("message_bytes", ctypes.c_int64), ("ring_macs", ctypes.c_int64), ("n_active", ctypes.c_int32),
                ("n_active_blocks", ctypes.c_int32), ("tokens", ctypes.c_int32), ("matmul_path", ctypes.c_int32),
                ("kernel_launches", ctypes.c_int64), ("phase_ms", ctypes.c_double * 5),
                ("phase_launches", ctypes.c_int64 * 5), ("n_components", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("tensor_tile_macs", ctypes.c_int64)]


class CometError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {_lib.comet_strerror(code).decode()} ({code})")
        self.code = code


def _load():
    if not is_current():
        # missing, or built from other sources than the ones in the tree: rebuild rather than run stale kernels
        try:
            build_library()
        except (OSError, subprocess.CalledProcessError) as exc:
            raise ImportError(
                f"{LIB_PATH} is missing or stale and could not be rebuilt ({exc}); build it with "
                "`python -m paper_2505_07239_b200.build` (there is no CPU fallback)") from exc
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    lib.comet_init.argtypes = [ctypes.POINTER(CometConfig), vp, ctypes.POINTER(vp)]
    lib.comet_destroy.argtypes = [vp]
    lib.comet_destroy.restype = None
    lib.comet_load_shares.argtypes = [vp, ctypes.c_int, ctypes.c_int, vp, ctypes.c_int, i64, i64]
    lib.comet_bind_shares.argtypes = [vp, ctypes.c_int, ctypes.c_int, vp, i64, i64]
    lib.comet_set_mask.argtypes = [vp, vp, ctypes.c_int, i32, ctypes.POINTER(i32)]
    lib.comet_set_token_mask.argtypes = [vp, vp, ctypes.c_int, i32, i32, ctypes.POINTER(i64)]
    lib.comet_get_components.argtypes = [vp, vp, vp, ctypes.c_int, ctypes.POINTER(i32)]
    lib.comet_ffn_up.argtypes = [vp, i32]
    lib.comet_ffn_down.argtypes = [vp, i32]
    lib.comet_truncate.argtypes = [vp, ctypes.c_int]
    lib.comet_get.argtypes = [vp, ctypes.c_int, ctypes.c_int, vp, ctypes.c_int, i64, ctypes.POINTER(i64)]
    lib.comet_get_index.argtypes = [vp, vp, ctypes.c_int, i32, ctypes.POINTER(i32)]
    lib.comet_stats.argtypes = [vp, ctypes.POINTER(CometStats)]
    lib.comet_strerror.argtypes = [ctypes.c_int]
    lib.comet_strerror.restype = ctypes.c_char_p
    lib.comet_last_cuda_error.argtypes = [vp]
    lib.comet_set_profiling.argtypes = [vp, ctypes.c_int]
    lib.comet_synchronize.argtypes = [vp]
    lib.comet_inject_timeout.argtypes = [vp]
    lib.comet_device_pointer.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.POINTER(vp)]
    lib.comet_pipe_probe.argtypes = [vp, ctypes.c_int, i32, i32, ctypes.POINTER(ctypes.c_float),
                                     ctypes.POINTER(ctypes.c_double)]
    pair = ctypes.c_void_p * 2
    lib.comet_beaver_matmul_static.argtypes = [vp, pair, pair, pair, pair, pair, pair, i32, i32, i32]
    lib.comet_shuffle.argtypes = [vp, pair, pair, pair, pair, pair, pair, pair, i64, i64, vp]
    lib.comet_invert_permutation.argtypes = [vp, vp, vp, i64, vp]
    lib.comet_add_bias.argtypes = [vp, pair, pair, i64, i64]
    lib.comet_truncate_pair.argtypes = [vp, pair, pair, pair, pair, i64, i32]
    lib.comet_kv_plan.argtypes = [vp, vp, i32, i32, i64, i64, vp, vp, ctypes.POINTER(i32)]
    lib.comet_beaver_mul.argtypes = [vp, pair, pair, pair, pair, pair, pair, pair, pair, i64]
    return lib


_lib = _load()


def library():
    """The loaded ctypes library (for tests that poke the raw ABI)."""
    return _lib


def _ptr_loc(t):
    """(address, location, element count) of a torch tensor or numpy array of 8-byte words."""
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"] and t.dtype.itemsize == 8
        return t.ctypes.data, HOST, t.size
    assert t.is_contiguous() and t.element_size() == 8
    return t.data_ptr(), (DEVICE if t.is_cuda else HOST), t.numel()


class Comet:
    """One secret-shared FFN layer on one GPU (both parties), over the C ABI."""

    def __init__(self, max_tokens: int, d_model: int, d_ff: int, block: int, frac_bits: int, gated: bool = False,
                 device: int = 0, max_active: int = 0, matmul_path: int = PATH_AUTO,
                 stream: Optional[torch.cuda.Stream] = None):
        self.cfg = CometConfig(max_tokens, d_model, d_ff, block, frac_bits, int(gated), device, max_active,
                               matmul_path)
        self.device = torch.device("cuda", device)
        self.stream = stream
        self._h = ctypes.c_void_p()
        sp = ctypes.c_void_p(stream.cuda_stream if stream is not None else 0)
        self._check(_lib.comet_init(ctypes.byref(self.cfg), sp, ctypes.byref(self._h)), "comet_init")
        self.groups = int(gated) + 1
        self.n_active = 0

    # ------------------------------------------------------------------ plumbing
    def _check(self, code: int, what: str):
        if code != OK:
            raise CometError(code, what)

    def close(self):
        if self._h:
            _lib.comet_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def synchronize(self):
        """Wait for the context's work; raises if one of its kernels gave up on a bounded wait."""
        self._check(_lib.comet_synchronize(self._h), "comet_synchronize")

    # ------------------------------------------------------------------ the six calls
    def load_shares(self, party: int, tensor_id: int, t):
        ptr, loc, _ = _ptr_loc(t)
        rows, cols = t.shape
        self._check(_lib.comet_load_shares(self._h, party, tensor_id, ptr, loc, rows, cols), "comet_load_shares")

    def bind_shares(self, party: int, tensor_id: int, t):
        """Use a CUDA tensor of 8-byte words in place (no copy); the caller keeps it alive and unchanged."""
        ptr, loc, _ = _ptr_loc(t)
        assert loc == DEVICE
        rows, cols = t.shape
        self._check(_lib.comet_bind_shares(self._h, party, tensor_id, ptr, rows, cols), "comet_bind_shares")

    def set_mask(self, mask) -> int:
        if isinstance(mask, np.ndarray):
            assert mask.dtype == np.uint8 and mask.flags["C_CONTIGUOUS"]
            ptr, loc, nb = mask.ctypes.data, HOST, mask.size
        else:
            assert mask.dtype == torch.uint8 and mask.is_contiguous()
            ptr, loc, nb = mask.data_ptr(), (DEVICE if mask.is_cuda else HOST), mask.numel()
        n = ctypes.c_int32(0)
        self._check(_lib.comet_set_mask(self._h, ptr, loc, nb, ctypes.byref(n)), "comet_set_mask")
        self.n_active = n.value
        return n.value

    def set_token_mask(self, mask) -> int:
        """Per-token mask over the active blocks, [tokens, n_active_blocks] uint8 (numpy or torch), or None to
        clear it.  Returns the number of non-zero entries of the hidden state under it."""
        masked = ctypes.c_int64(0)
        if mask is None:
            self._check(_lib.comet_set_token_mask(self._h, None, DEVICE, 0, 0, ctypes.byref(masked)),
                        "comet_set_token_mask")
            return 0
        if isinstance(mask, np.ndarray):
            assert mask.dtype == np.uint8 and mask.flags["C_CONTIGUOUS"] and mask.ndim == 2
            ptr, loc = mask.ctypes.data, HOST
        else:
            assert mask.dtype == torch.uint8 and mask.is_contiguous() and mask.dim() == 2
            ptr, loc = mask.data_ptr(), (DEVICE if mask.is_cuda else HOST)
        self._check(_lib.comet_set_token_mask(self._h, ptr, loc, mask.shape[0], mask.shape[1], ctypes.byref(masked)),
                    "comet_set_token_mask")
        return masked.value

    def get_components(self, tokens: int, n_active_blocks: int):
        """(row_label [tokens], blk_label [n_active_blocks], number of components) under the current token mask."""
        rl = torch.empty(tokens, dtype=torch.int32, device=self.device)
        bl = torch.empty(n_active_blocks, dtype=torch.int32, device=self.device)
        cnt = ctypes.c_int32(0)
        self._check(_lib.comet_get_components(self._h, rl.data_ptr(), bl.data_ptr(), DEVICE, ctypes.byref(cnt)),
                    "comet_get_components")
        self.synchronize()
        return rl.cpu().numpy(), bl.cpu().numpy(), cnt.value

    def ffn_up(self, tokens: int):
        self._check(_lib.comet_ffn_up(self._h, tokens), "comet_ffn_up")

    def ffn_down(self, tokens: int):
        self._check(_lib.comet_ffn_down(self._h, tokens), "comet_ffn_down")

    def truncate(self, tensor_id: int):
        self._check(_lib.comet_truncate(self._h, tensor_id), "comet_truncate")

    # ------------------------------------------------------------------ read-back
    def get_into(self, party: int, tensor_id: int, out) -> int:
        """Copy a tensor into caller memory (device tensor, or pinned/pageable host array)."""
        ptr, loc, cap = _ptr_loc(out)
        written = ctypes.c_int64(0)
        self._check(_lib.comet_get(self._h, party, tensor_id, ptr, loc, cap, ctypes.byref(written)), "comet_get")
        return written.value

    def get(self, party: int, tensor_id: int, shape) -> np.ndarray:
        """Read a tensor back to a numpy uint64 array of the given stored shape."""
        out = torch.empty(int(np.prod(shape)), dtype=torch.int64, device=self.device)
        n = self.get_into(party, tensor_id, out)
        self.synchronize()
        assert n == out.numel(), (n, shape)
        return out.cpu().numpy().view(np.uint64).reshape(shape)

    def result_view(self, party: int, tensor_id: int, shape) -> torch.Tensor:
        """The library's own buffer of a result tensor (Z_UP or Y) as a torch int64 tensor of the given stored
        shape, sharing memory with the library (no copy): for in-place collectives between two calls of the path."""
        addr = ctypes.c_void_p()
        self._check(_lib.comet_device_pointer(self._h, party, tensor_id, ctypes.byref(addr)), "comet_device_pointer")

        class _View:                             # the CUDA array interface: address, shape and element type
            __cuda_array_interface__ = {"shape": tuple(int(v) for v in shape), "typestr": "<i8",
                                        "data": (addr.value, False), "version": 2, "strides": None}

        return torch.as_tensor(_View(), device=self.device)

    def get_index(self) -> np.ndarray:
        nb = self.cfg.d_ff // self.cfg.block
        out = torch.empty(nb, dtype=torch.int32, device=self.device)
        cnt = ctypes.c_int32(0)
        self._check(_lib.comet_get_index(self._h, out.data_ptr(), DEVICE, nb, ctypes.byref(cnt)), "comet_get_index")
        self.synchronize()
        return out[:cnt.value].cpu().numpy()

    def set_profiling(self, on: bool):
        self._check(_lib.comet_set_profiling(self._h, int(on)), "comet_set_profiling")

    def stats(self) -> CometStats:
        s = CometStats()
        self._check(_lib.comet_stats(self._h, ctypes.byref(s)), "comet_stats")
        return s


def to_device(a: np.ndarray, device="cuda:0") -> torch.Tensor:
    """numpy uint64 -> torch int64 CUDA tensor holding the same words."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int64)).to(device)


def beaver_matmul_static(X, A, Y, B, C, Z, stream: Optional[torch.cuda.Stream] = None) -> int:
    """Allocation-free dense Beaver product for both parties (comet_beaver_matmul_static).

    For callers that cannot allocate device memory when they need the product
    (all memory already owned by a framework's pool, or a serving loop that must
    not stall on cudaMalloc): the message buffers live in an 8 MiB array inside
    the library.  Each argument is a pair (party 0, party 1) of CUDA tensors of
    8-byte words on the current device: X, A [T, K]; Y, B [N, K]; C, Z [T, N].
    Returns the library's status code (0 = ok) instead of raising, so that the
    size-limit refusal can be observed.  Calls that overlap on the GPU race on
    the shared array: keep them on one stream.
    """
    T, K = X[0].shape
    N = Y[0].shape[0]
    pair = ctypes.c_void_p * 2

    def ptrs(ts, shape):
        for t in ts:
            assert t.is_cuda and t.is_contiguous() and t.element_size() == 8 and tuple(t.shape) == shape
        return pair(ts[0].data_ptr(), ts[1].data_ptr())

    sp = ctypes.c_void_p(stream.cuda_stream if stream is not None else 0)
    return _lib.comet_beaver_matmul_static(sp, ptrs(X, (T, K)), ptrs(A, (T, K)), ptrs(Y, (N, K)), ptrs(B, (N, K)),
                                           ptrs(C, (T, N)), ptrs(Z, (T, N)), T, K, N)


PIPE_TENSOR_I8, PIPE_ALU_U64 = 0, 1


def pipe_probe(pipe: int, launches: int, work: int, stream: Optional[torch.cuda.Stream] = None):
    """Measured rate of a multiply pipe (comet_pipe_probe): returns (ms per launch [launches], multiply-adds per
    launch): 8-bit ones for PIPE_TENSOR_I8, 64-bit ones for PIPE_ALU_U64."""
    ms = (ctypes.c_float * launches)()
    macs = ctypes.c_double(0.0)
    sp = ctypes.c_void_p(stream.cuda_stream if stream is not None else 0)
    code = _lib.comet_pipe_probe(sp, pipe, launches, work, ms, ctypes.byref(macs))
    if code != OK:
        raise CometError(code, "comet_pipe_probe")
    return [float(v) for v in ms], macs.value


def _pair(ts, shape=None, dtype=None):
    for t in ts:
        assert t.is_cuda and t.is_contiguous()
        assert shape is None or tuple(t.shape) == tuple(shape)
        assert dtype is None or t.dtype == dtype
    return (ctypes.c_void_p * 2)(ts[0].data_ptr(), ts[1].data_ptr())


def shuffle(X, tau, rho, a, b, stream: Optional[torch.cuda.Stream] = None, bad_index_flag=None):
    """Oblivious shuffle of the rows of a shared matrix (comet_shuffle), both parties.

    Each argument is a pair (party 0, party 1) of CUDA tensors: X, a, b of 8-byte
    words with the same shape [rows, ...]; tau, rho int32 of length rows.
    Returns (Y, Z): the two messages and the two shares of pi(x).  Only the
    output tensors are allocated here (torch); the arithmetic is the library's.
    """
    rows = X[0].shape[0]
    cols = X[0].numel() // rows
    Y = [torch.empty_like(X[0]) for _ in (0, 1)]
    Z = [torch.empty_like(X[0]) for _ in (0, 1)]
    sp = ctypes.c_void_p(stream.cuda_stream if stream is not None else 0)
    flag = ctypes.c_void_p(bad_index_flag.data_ptr() if bad_index_flag is not None else 0)
    for t in (*X, *a, *b):
        assert t.element_size() == 8
    code = _lib.comet_shuffle(sp, _pair(X), _pair(tau, (rows,), torch.int32), _pair(rho, (rows,), torch.int32),
                              _pair(a, X[0].shape), _pair(b, X[0].shape), _pair(Y), _pair(Z), rows, cols, flag)
    if code != OK:
        raise CometError(code, "comet_shuffle")
    return Y, Z


def invert_permutation(perm, stream: Optional[torch.cuda.Stream] = None, bad_index_flag=None):
    """inverse[perm[j]] = j on the device (comet_invert_permutation)."""
    assert perm.is_cuda and perm.dtype == torch.int32 and perm.is_contiguous()
    out = torch.empty_like(perm)
    sp = ctypes.c_void_p(stream.cuda_stream if stream is not None else 0)
    flag = ctypes.c_void_p(bad_index_flag.data_ptr() if bad_index_flag is not None else 0)
    code = _lib.comet_invert_permutation(sp, perm.data_ptr(), out.data_ptr(), perm.numel(), flag)
    if code != OK:
        raise CometError(code, "comet_invert_permutation")
    return out


def beaver_mul(X, Y, A, B, C, stream: Optional[torch.cuda.Stream] = None):
    """Element-wise Beaver product of two shared tensors (comet_beaver_mul), both parties.
    Every argument is a pair of equally shaped CUDA tensors of 8-byte words.
    Returns (D, E, Z): the messages x - a and y - b, and the shares of x * y."""
    shape = X[0].shape
    for t in (*X, *Y, *A, *B, *C):
        assert t.element_size() == 8 and t.shape == shape
    D = [torch.empty_like(X[0]) for _ in (0, 1)]
    E = [torch.empty_like(X[0]) for _ in (0, 1)]
    Z = [torch.empty_like(X[0]) for _ in (0, 1)]
    sp = ctypes.c_void_p(stream.cuda_stream if stream is not None else 0)
    code = _lib.comet_beaver_mul(sp, _pair(X), _pair(Y), _pair(A), _pair(B), _pair(C), _pair(D), _pair(E), _pair(Z),
                                 X[0].numel())
    if code != OK:
        raise CometError(code, "comet_beaver_mul")
    return D, E, Z


def truncate_pair(Z, R, RP, frac_bits: int, stream: Optional[torch.cuda.Stream] = None):
    """Truncation with a dealer's pair (comet_truncate_pair), both parties: Z is replaced by shares of
    floor(z / 2^frac_bits) (or one less).  Z, R, RP are pairs of equally shaped CUDA tensors of 8-byte words.
    Returns the messages M = Z - R (a pair)."""
    shape = Z[0].shape
    for t in (*Z, *R, *RP):
        assert t.element_size() == 8 and t.shape == shape
    M = [torch.empty_like(Z[0]) for _ in (0, 1)]
    sp = ctypes.c_void_p(stream.cuda_stream if stream is not None else 0)
    code = _lib.comet_truncate_pair(sp, _pair(Z), _pair(R), _pair(RP), _pair(M), Z[0].numel(), frac_bits)
    if code != OK:
        raise CometError(code, "comet_truncate_pair")
    return M


def kv_plan(present: np.ndarray, active: np.ndarray, x: int, w: int):
    """KV-cache manager's request planning (comet_kv_plan, host logic): returns (request [tokens, heads] uint8,
    prefetch [heads] uint8, L1).  `request` is the per-token head mask of the merged refill + prefetch batch."""
    present = np.ascontiguousarray(present, dtype=np.uint8)
    active = np.ascontiguousarray(active, dtype=np.uint8)
    tokens, heads = present.shape
    request = np.empty((tokens, heads), np.uint8)
    prefetch = np.empty(heads, np.uint8)
    l1 = ctypes.c_int32(0)
    code = _lib.comet_kv_plan(present.ctypes.data, active.ctypes.data, tokens, heads, x, w, request.ctypes.data,
                              prefetch.ctypes.data, ctypes.byref(l1))
    if code != OK:
        raise CometError(code, "comet_kv_plan")
    return request, prefetch, l1.value


def add_bias(Z, bias, stream: Optional[torch.cuda.Stream] = None):
    """Z[i][r, :] += bias[i] in place for both parties (comet_add_bias)."""
    rows, cols = Z[0].shape
    for t in bias:
        assert t.element_size() == 8 and tuple(t.shape) == (cols,)
    sp = ctypes.c_void_p(stream.cuda_stream if stream is not None else 0)
    code = _lib.comet_add_bias(sp, _pair(Z, (rows, cols)), _pair(bias), rows, cols)
    if code != OK:
        raise CometError(code, "comet_add_bias")
