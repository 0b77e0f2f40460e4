"""CPU oracle for the variance-based gradient compression hot path -- TEST INFRASTRUCTURE.

Thin ctypes access to ``vgc_oracle.c`` (plain C, built with gcc, no CUDA).  Only the test
suite, the smoke check and the benchmark's CPU-baseline leg may import this package; the
CUDA library and its Python binding never do.  Arrays are numpy, C-contiguous.

Each function cites the passage of the paper it follows in ``vgc_oracle.c``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vgc_oracle.c")
_LIB = os.path.join(_HERE, "libvgc_oracle.so")

EXP_NONE = -(2 ** 31)

_CFLAGS = ["-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c11", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(["gcc", *_CFLAGS, "-o", tmp, _SRC], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        f32p = ctypes.POINTER(ctypes.c_float)
        u32p = ctypes.POINTER(ctypes.c_uint32)
        i32p = ctypes.POINTER(ctypes.c_int32)
        i = ctypes.c_int
        lib.oracle_sqgrad_linear.argtypes = [f32p, f32p, i, i, i, ctypes.c_float, i, f32p]
        lib.oracle_sqgrad_linear.restype = None
        conv_shape = [i] * 11
        lib.oracle_sqgrad_conv.argtypes = [f32p, f32p, *conv_shape, ctypes.c_float, i, f32p]
        lib.oracle_sqgrad_conv.restype = None
        lib.oracle_sqgrad_conv_entries.argtypes = [f32p, f32p, *conv_shape, ctypes.c_float,
                                                   ctypes.POINTER(ctypes.c_int64), ctypes.c_int64, f32p]
        lib.oracle_sqgrad_conv_entries.restype = None
        lib.oracle_sqgrad_conv_exact.argtypes = [f32p, f32p, *conv_shape, ctypes.c_float, f32p]
        lib.oracle_sqgrad_conv_exact.restype = None
        lib.oracle_compress.argtypes = [f32p, f32p, f32p, f32p, ctypes.c_uint64, u32p, i,
                                        ctypes.c_float, ctypes.c_float, u32p, ctypes.c_uint64, i32p,
                                        u32p, u32p, u32p, ctypes.POINTER(ctypes.c_uint8)]
        lib.oracle_compress.restype = ctypes.c_int
        lib.oracle_decode_accumulate.argtypes = [ctypes.POINTER(u32p), u32p, ctypes.POINTER(i32p), i,
                                                 u32p, i, ctypes.c_float, f32p, ctypes.c_uint64]
        lib.oracle_decode_accumulate.restype = ctypes.c_uint64
        lib.oracle_compress_hybrid.argtypes = [f32p, f32p, f32p, f32p, ctypes.c_uint64, ctypes.c_float,
                                               ctypes.c_float, ctypes.c_float, i, u32p, ctypes.c_uint64, u32p,
                                               ctypes.POINTER(ctypes.c_uint8)]
        lib.oracle_compress_hybrid.restype = ctypes.c_int
        lib.oracle_decode_hybrid.argtypes = [ctypes.POINTER(u32p), u32p, i, ctypes.c_float, ctypes.c_float, f32p,
                                             ctypes.c_uint64]
        lib.oracle_decode_hybrid.restype = ctypes.c_uint64
        u8p = ctypes.POINTER(ctypes.c_uint8)
        lib.oracle_pack_indices.argtypes = [u32p, ctypes.c_uint32, u8p, ctypes.c_uint64]
        lib.oracle_pack_indices.restype = ctypes.c_uint64
        lib.oracle_unpack_indices.argtypes = [u8p, ctypes.c_uint32, u32p]
        lib.oracle_unpack_indices.restype = ctypes.c_int
        _lib = lib
    return _lib


def _f32(a, name):
    a = np.ascontiguousarray(a)
    if a.dtype != np.float32:
        raise TypeError(f"{name} must be float32, got {a.dtype}")
    return a


def _ptr(a, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def sqgrad_linear(x, delta, scale=1.0, out=None):
    """S[j,i] = scale * sum_z (delta[z,j] * x[z,i])^2 ; x [B,in], delta [B,out] -> S [out,in].

    ``out`` given: the statistic is added to it (fp64 add, one rounding)."""
    x = _f32(x, "x"); delta = _f32(delta, "delta")
    B, n_in = x.shape
    B2, n_out = delta.shape
    assert B == B2
    acc = out is not None
    S = np.zeros((n_out, n_in), np.float32) if out is None else out
    assert S.dtype == np.float32 and S.flags.c_contiguous and S.shape == (n_out, n_in)
    _load().oracle_sqgrad_linear(_ptr(x, ctypes.c_float), _ptr(delta, ctypes.c_float), B, n_in, n_out,
                                 float(scale), int(acc), _ptr(S, ctypes.c_float))
    return S


def _conv_args(x, delta, kernel, stride, padding):
    x = _f32(x, "x"); delta = _f32(delta, "delta")
    B, C, H, W = x.shape
    B2, Cout, Ho, Wo = delta.shape
    Kh, Kw = kernel
    sh, sw = stride
    ph, pw = padding
    assert B == B2
    assert Ho == (H + 2 * ph - Kh) // sh + 1 and Wo == (W + 2 * pw - Kw) // sw + 1, "delta shape"
    return x, delta, (B, C, H, W, Cout, Kh, Kw, sh, sw, ph, pw)


def sqgrad_conv(x, delta, kernel, stride=(1, 1), padding=(0, 0), scale=1.0, out=None):
    """Position-as-sample conv statistic, S [Cout,C,Kh,Kw]; x NCHW, delta [B,Cout,Ho,Wo]."""
    x, delta, shp = _conv_args(x, delta, kernel, stride, padding)
    B, C, H, W, Cout, Kh, Kw = shp[:7]
    acc = out is not None
    S = np.zeros((Cout, C, Kh, Kw), np.float32) if out is None else out
    assert S.dtype == np.float32 and S.flags.c_contiguous and S.shape == (Cout, C, Kh, Kw)
    _load().oracle_sqgrad_conv(_ptr(x, ctypes.c_float), _ptr(delta, ctypes.c_float), *shp,
                               float(scale), int(acc), _ptr(S, ctypes.c_float))
    return S


def sqgrad_conv_entries(x, delta, kernel, stride, padding, scale, flat_idx):
    """The conv statistic at the listed flat OIHW positions only."""
    x, delta, shp = _conv_args(x, delta, kernel, stride, padding)
    idx = np.ascontiguousarray(flat_idx, dtype=np.int64)
    out = np.zeros(idx.shape, np.float32)
    _load().oracle_sqgrad_conv_entries(_ptr(x, ctypes.c_float), _ptr(delta, ctypes.c_float), *shp,
                                       float(scale), _ptr(idx, ctypes.c_int64), idx.size,
                                       _ptr(out, ctypes.c_float))
    return out


def sqgrad_conv_exact(x, delta, kernel, stride=(1, 1), padding=(0, 0), scale=1.0):
    """Per-example conv gradients, squared and summed (keeps the cross terms between positions)."""
    x, delta, shp = _conv_args(x, delta, kernel, stride, padding)
    B, C, H, W, Cout, Kh, Kw = shp[:7]
    S = np.zeros((Cout, C, Kh, Kw), np.float32)
    _load().oracle_sqgrad_conv_exact(_ptr(x, ctypes.c_float), _ptr(delta, ctypes.c_float), *shp,
                                     float(scale), _ptr(S, ctypes.c_float))
    return S


class Message:
    """One worker's packed message: words (u32, ascending index), per-group exponents, counters."""

    def __init__(self, words, group_exp, nnz, n_criterion, n_dropped, mask, overflow):
        self.words = words
        self.group_exp = group_exp
        self.nnz = nnz
        self.n_criterion = n_criterion
        self.n_dropped = n_dropped
        self.mask = mask
        self.overflow = overflow


def compress(g, s, r, v, group_offsets, alpha, zeta, capacity=None, want_mask=True):
    """One step of Algorithm 1 over the flat buffer; r and v are updated IN PLACE."""
    g = _f32(g, "g"); s = _f32(s, "s")
    for name, a in (("r", r), ("v", v)):
        if not (isinstance(a, np.ndarray) and a.dtype == np.float32 and a.flags.c_contiguous):
            raise TypeError(f"{name} must be a contiguous float32 array (updated in place)")
    n = g.size
    assert s.size == n and r.size == n and v.size == n
    offs = np.ascontiguousarray(group_offsets, dtype=np.uint32)
    K = offs.size - 1
    assert K >= 0 and (K == 0 or (offs[0] == 0 and offs[-1] == n))
    cap = n if capacity is None else int(capacity)
    words = np.zeros(max(cap, 1), np.uint32)
    gexp = np.zeros(max(K, 1), np.int32)
    cnt = np.zeros(3, np.uint32)
    mask = np.zeros(max(n, 1), np.uint8) if want_mask else None
    over = _load().oracle_compress(
        _ptr(g, ctypes.c_float), _ptr(s, ctypes.c_float), _ptr(r, ctypes.c_float), _ptr(v, ctypes.c_float),
        n, _ptr(offs, ctypes.c_uint32), K, float(alpha), float(zeta),
        _ptr(words, ctypes.c_uint32), cap, _ptr(gexp, ctypes.c_int32),
        _ptr(cnt[0:1], ctypes.c_uint32), _ptr(cnt[1:2], ctypes.c_uint32), _ptr(cnt[2:3], ctypes.c_uint32),
        _ptr(mask, ctypes.c_uint8) if want_mask else None)
    nnz = int(cnt[0])
    return Message(words[:min(nnz, cap)].copy(), gexp[:K].copy(), nnz, int(cnt[1]), int(cnt[2]),
                   mask[:n] if want_mask else None, bool(over))


def decode_accumulate(messages, group_offsets, scale, u):
    """u[idx] += scale * decoded value for every word of every message, in message order.

    ``messages``: sequence of (words u32 array, group_exp i32 array).  u is updated IN PLACE.
    Returns the number of words skipped because their index was out of range."""
    if not (isinstance(u, np.ndarray) and u.dtype == np.float32 and u.flags.c_contiguous):
        raise TypeError("u must be a contiguous float32 array (updated in place)")
    offs = np.ascontiguousarray(group_offsets, dtype=np.uint32)
    K = offs.size - 1
    W = len(messages)
    u32p = ctypes.POINTER(ctypes.c_uint32)
    i32p = ctypes.POINTER(ctypes.c_int32)
    keep = []
    wptrs = (u32p * max(W, 1))()
    eptrs = (i32p * max(W, 1))()
    nnz = np.zeros(max(W, 1), np.uint32)
    for w, (words, gexp) in enumerate(messages):
        words = np.ascontiguousarray(words, dtype=np.uint32)
        gexp = np.ascontiguousarray(gexp, dtype=np.int32)
        assert gexp.size == K
        keep.append((words, gexp))
        wptrs[w] = _ptr(words, ctypes.c_uint32)
        eptrs[w] = _ptr(gexp, ctypes.c_int32)
        nnz[w] = words.size
    return int(_load().oracle_decode_accumulate(wptrs, _ptr(nnz, ctypes.c_uint32), eptrs, W,
                                                _ptr(offs, ctypes.c_uint32), K, float(scale),
                                                _ptr(u, ctypes.c_float), u.size))


def compress_hybrid(g, s, r, v, alpha, zeta, tau, pre_update_r=True, capacity=None, want_mask=True):
    """One step of the hybrid algorithm (Algorithm 2); r and v are updated IN PLACE.  Returns a Message whose
    words are index << 4 | sign << 3 (group_exp is empty, n_criterion == nnz)."""
    g = _f32(g, "g"); s = _f32(s, "s")
    n = g.size
    cap = n if capacity is None else int(capacity)
    words = np.zeros(max(cap, 1), np.uint32)
    cnt = np.zeros(1, np.uint32)
    mask = np.zeros(max(n, 1), np.uint8) if want_mask else None
    over = _load().oracle_compress_hybrid(
        _ptr(g, ctypes.c_float), _ptr(s, ctypes.c_float), _ptr(r, ctypes.c_float), _ptr(v, ctypes.c_float), n,
        float(alpha), float(zeta), float(tau), int(bool(pre_update_r)), _ptr(words, ctypes.c_uint32), cap,
        _ptr(cnt, ctypes.c_uint32), _ptr(mask, ctypes.c_uint8) if want_mask else None)
    nnz = int(cnt[0])
    return Message(words[:min(nnz, cap)].copy(), np.zeros(0, np.int32), nnz, nnz, 0, mask[:n] if want_mask else None,
                   bool(over))


def decode_hybrid(word_arrays, tau, scale, u):
    """u[idx] += scale * (+-tau) for every word of every message (message order); u IN PLACE."""
    W = len(word_arrays)
    u32p = ctypes.POINTER(ctypes.c_uint32)
    keep = [np.ascontiguousarray(w, dtype=np.uint32) for w in word_arrays]
    ptrs = (u32p * max(W, 1))()
    nnz = np.zeros(max(W, 1), np.uint32)
    for k, w in enumerate(keep):
        ptrs[k] = _ptr(w, ctypes.c_uint32)
        nnz[k] = w.size
    return int(_load().oracle_decode_hybrid(ptrs, _ptr(nnz, ctypes.c_uint32), W, float(tau), float(scale),
                                            _ptr(u, ctypes.c_float), u.size))


PACK_RUN = 256


def pack_indices(words) -> np.ndarray:
    """The message's words (uint32, ascending index) with the index field stored as differences in the base-128
    variable-length code: uint8 array [run table][payload] (Sec. 4.2, last paragraph; format in vgc_oracle.c)."""
    words = np.ascontiguousarray(words, dtype=np.uint32)
    lib = _load()
    u32p, u8p = ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(ctypes.c_uint8)
    runs = (words.size + PACK_RUN - 1) // PACK_RUN
    out = np.zeros(4 * (runs + 1) + 5 * words.size, np.uint8)
    size = lib.oracle_pack_indices(words.ctypes.data_as(u32p), words.size, out.ctypes.data_as(u8p), out.size)
    assert size <= out.size
    return out[:size].copy()


def unpack_indices(packed, nnz: int) -> np.ndarray:
    """Inverse of pack_indices: the nnz 32-bit words.  Raises ValueError on a malformed stream."""
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    words = np.zeros(nnz, np.uint32)
    u32p, u8p = ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(ctypes.c_uint8)
    if _load().oracle_unpack_indices(packed.ctypes.data_as(u8p), nnz, words.ctypes.data_as(u32p)) != 0:
        raise ValueError("malformed index stream")
    return words
