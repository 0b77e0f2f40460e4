"""Variance-based gradient compression hot path on NVIDIA B200 -- Python binding.

Thin ctypes marshalling over the C ABI declared in ``include/vgc.h`` (same entry-point names).
Every step of the path runs in the CUDA library ``libvgc.so`` built from ``csrc/``; this module
only checks tensors, passes pointers and sizes, and raises on a non-zero status.  PyTorch is
used for device memory and streams.  There is no CPU fallback: if the library is missing or
was not built, every call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

from ._build import LIB_PATH, build  # noqa: F401  (build is re-exported)

VGC_OK = 0
VGC_DEV_CAPACITY = 1
VGC_DEV_TIMEOUT = 2
VGC_DEV_RANGE = 4
VGC_EXP_NONE = -(2 ** 31)
VGC_MAX_PARAMS = 1 << 28

EXPORTS = [
    "vgc_status_string", "vgc_version", "vgc_kernel_launch_count",
    "vgc_sqgrad_linear_workspace_bytes", "vgc_sqgrad_linear",
    "vgc_sqgrad_conv_workspace_bytes", "vgc_sqgrad_conv",
    "vgc_sqgrad_conv_batch_workspace_bytes", "vgc_sqgrad_conv_batch", "vgc_sqgrad_plan_hint",
    "vgc_sqgrad_conv_exact_workspace_bytes", "vgc_sqgrad_conv_exact",
    "vgc_sqgrad_conv_exact_batch_workspace_bytes", "vgc_sqgrad_conv_exact_batch",
    "vgc_compress_workspace_bytes", "vgc_compress", "vgc_compress_static",
    "vgc_decode_accumulate", "vgc_step_host",
    "vgc_compress_hybrid_workspace_bytes", "vgc_compress_hybrid", "vgc_decode_accumulate_hybrid",
    "vgc_decode_sum", "vgc_decode_sum_hybrid",
    "vgc_pack_bound_bytes", "vgc_pack_workspace_bytes", "vgc_pack_indices", "vgc_unpack_indices",
]


class VgcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({_status_string(status)})")


class _MessageStruct(ctypes.Structure):      # mirrors vgc_message
    _fields_ = [("words", ctypes.c_void_p), ("capacity", ctypes.c_uint32), ("group_exp", ctypes.c_void_p),
                ("nnz", ctypes.c_void_p), ("n_criterion", ctypes.c_void_p), ("n_dropped", ctypes.c_void_p),
                ("mask", ctypes.c_void_p), ("dev_status", ctypes.c_void_p)]


class _LayerHostStruct(ctypes.Structure):    # mirrors vgc_layer_host
    _fields_ = [(name, ctypes.c_int) for name in ("is_conv", "B", "C", "H", "W", "Cout", "Kh", "Kw", "stride_h",
                                                  "stride_w", "pad_h", "pad_w")] + \
               [("x_host", ctypes.c_void_p), ("delta_host", ctypes.c_void_p), ("x_dev", ctypes.c_void_p),
                ("delta_dev", ctypes.c_void_p)]


class _HybridMessageStruct(ctypes.Structure):    # mirrors vgc_hybrid_message
    _fields_ = [("words", ctypes.c_void_p), ("capacity", ctypes.c_uint32), ("nnz", ctypes.c_void_p),
                ("mask", ctypes.c_void_p), ("dev_status", ctypes.c_void_p)]


class _ViewStruct(ctypes.Structure):         # mirrors vgc_message_view
    _fields_ = [("words", ctypes.c_void_p), ("nnz", ctypes.c_void_p), ("group_exp", ctypes.c_void_p),
                ("max_words", ctypes.c_uint32)]


_lib = None


def load_library():
    """Load libvgc.so (raises if it has not been built) and declare the entry points."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run paper_1802_06058_b200.build() "
                           "(needs nvcc); there is no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.vgc_status_string.argtypes = [i]; lib.vgc_status_string.restype = ctypes.c_char_p
    lib.vgc_version.argtypes = []; lib.vgc_version.restype = i
    lib.vgc_kernel_launch_count.argtypes = []; lib.vgc_kernel_launch_count.restype = ctypes.c_uint64
    lib.vgc_sqgrad_linear_workspace_bytes.argtypes = [i, i, i]
    lib.vgc_sqgrad_linear_workspace_bytes.restype = sz
    lib.vgc_sqgrad_linear.argtypes = [vp, vp, i, i, i, f, i, vp, vp, sz, vp]
    lib.vgc_sqgrad_linear.restype = i
    lib.vgc_sqgrad_conv_workspace_bytes.argtypes = [i] * 11
    lib.vgc_sqgrad_conv_workspace_bytes.restype = sz
    lib.vgc_sqgrad_conv.argtypes = [vp, vp] + [i] * 11 + [f, i, vp, vp, sz, vp]
    lib.vgc_sqgrad_conv.restype = i
    lib.vgc_sqgrad_conv_batch_workspace_bytes.argtypes = [i] * 12
    lib.vgc_sqgrad_conv_batch_workspace_bytes.restype = sz
    lib.vgc_sqgrad_conv_batch.argtypes = [i, vp, vp, vp] + [i] * 11 + [f, i, vp, sz, vp]
    lib.vgc_sqgrad_conv_batch.restype = i
    lib.vgc_sqgrad_plan_hint.argtypes = [i]; lib.vgc_sqgrad_plan_hint.restype = None
    lib.vgc_sqgrad_conv_exact_workspace_bytes.argtypes = [i] * 11
    lib.vgc_sqgrad_conv_exact_workspace_bytes.restype = sz
    lib.vgc_sqgrad_conv_exact.argtypes = lib.vgc_sqgrad_conv.argtypes
    lib.vgc_sqgrad_conv_exact.restype = i
    lib.vgc_sqgrad_conv_exact_batch_workspace_bytes.argtypes = [i] * 12
    lib.vgc_sqgrad_conv_exact_batch_workspace_bytes.restype = sz
    lib.vgc_sqgrad_conv_exact_batch.argtypes = lib.vgc_sqgrad_conv_batch.argtypes
    lib.vgc_sqgrad_conv_exact_batch.restype = i
    lib.vgc_compress_workspace_bytes.argtypes = [sz, i]
    lib.vgc_compress_workspace_bytes.restype = sz
    lib.vgc_compress.argtypes = [vp, vp, vp, vp, sz, vp, i, f, f, ctypes.POINTER(_MessageStruct), vp, sz, vp]
    lib.vgc_compress.restype = i
    lib.vgc_compress_static.argtypes = [vp, vp, vp, vp, sz, vp, i, f, f, ctypes.POINTER(_MessageStruct), vp]
    lib.vgc_compress_static.restype = i
    lib.vgc_step_host.argtypes = [ctypes.POINTER(_LayerHostStruct), i, vp, vp, vp, vp, vp, sz, vp, i, f, f, f,
                                  ctypes.POINTER(_MessageStruct), vp, vp, vp, sz, vp, sz, vp]
    lib.vgc_step_host.restype = i
    lib.vgc_decode_accumulate.argtypes = [ctypes.POINTER(_ViewStruct), i, vp, i, f, vp, sz, vp, vp]
    lib.vgc_decode_accumulate.restype = i
    lib.vgc_decode_sum.argtypes = lib.vgc_decode_accumulate.argtypes
    lib.vgc_decode_sum.restype = i
    lib.vgc_compress_hybrid_workspace_bytes.argtypes = [sz]
    lib.vgc_compress_hybrid_workspace_bytes.restype = sz
    lib.vgc_compress_hybrid.argtypes = [vp, vp, vp, vp, sz, f, f, f, i, ctypes.POINTER(_HybridMessageStruct), vp, sz, vp]
    lib.vgc_compress_hybrid.restype = i
    lib.vgc_decode_accumulate_hybrid.argtypes = [ctypes.POINTER(_ViewStruct), i, f, f, vp, sz, vp, vp]
    lib.vgc_decode_accumulate_hybrid.restype = i
    lib.vgc_decode_sum_hybrid.argtypes = lib.vgc_decode_accumulate_hybrid.argtypes
    lib.vgc_decode_sum_hybrid.restype = i
    lib.vgc_pack_bound_bytes.argtypes = [ctypes.c_uint32]; lib.vgc_pack_bound_bytes.restype = sz
    lib.vgc_pack_workspace_bytes.argtypes = [ctypes.c_uint32]; lib.vgc_pack_workspace_bytes.restype = sz
    lib.vgc_pack_indices.argtypes = [vp, vp, ctypes.c_uint32, vp, sz, vp, vp, vp, sz, vp]
    lib.vgc_pack_indices.restype = i
    lib.vgc_unpack_indices.argtypes = [vp, vp, ctypes.c_uint32, vp, vp, vp]
    lib.vgc_unpack_indices.restype = i
    _lib = lib
    return lib


def _status_string(status: int) -> str:
    try:
        return load_library().vgc_status_string(int(status)).decode()
    except Exception:  # pragma: no cover
        return "?"


def _check(status: int, where: str):
    if status != VGC_OK:
        raise VgcError(status, where)


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ws(ws: Optional[torch.Tensor]):
    if ws is None:
        return None, 0
    if not ws.is_cuda or not ws.is_contiguous():
        raise ValueError("workspace must be a contiguous CUDA tensor")
    return ws.data_ptr(), ws.numel() * ws.element_size()


def vgc_version() -> int:
    return load_library().vgc_version()


def vgc_kernel_launch_count() -> int:
    return load_library().vgc_kernel_launch_count()


# ------------------------------------------------------------------------------------------ (1)
def vgc_sqgrad_linear_workspace_bytes(B: int, n_in: int, n_out: int) -> int:
    return load_library().vgc_sqgrad_linear_workspace_bytes(B, n_in, n_out)


def vgc_sqgrad_linear(x, delta, scale: float, S, accumulate: bool = False, ws=None, stream=None):
    """S[out,in] (+)= scale * sum_z delta[z,:]^2 (outer) x[z,:]^2 ; x [B,in], delta [B,out]."""
    B, n_in = x.shape
    B2, n_out = delta.shape
    if B != B2 or S.numel() != n_in * n_out:
        raise ValueError("shape mismatch")
    wp, wb = _ws(ws)
    st = load_library().vgc_sqgrad_linear(_dev(x, torch.float32, "x"), _dev(delta, torch.float32, "delta"),
                                          B, n_in, n_out, float(scale), int(bool(accumulate)),
                                          _dev(S, torch.float32, "S"), wp, wb, _stream(stream))
    _check(st, "vgc_sqgrad_linear")
    return S


def vgc_sqgrad_conv_workspace_bytes(B, C, H, W, Cout, Kh, Kw, sh, sw, ph, pw) -> int:
    return load_library().vgc_sqgrad_conv_workspace_bytes(B, C, H, W, Cout, Kh, Kw, sh, sw, ph, pw)


def vgc_sqgrad_conv(x, delta, kernel, stride, padding, scale: float, S, accumulate: bool = False,
                    ws=None, stream=None):
    """S[Cout,C,Kh,Kw] (+)= scale * sum over (example, output position) of squared contributions."""
    B, C, H, W = x.shape
    B2, Cout, Ho, Wo = delta.shape
    Kh, Kw = kernel
    sh, sw = stride
    ph, pw = padding
    if B != B2 or S.numel() != Cout * C * Kh * Kw:
        raise ValueError("shape mismatch")
    if Ho != (H + 2 * ph - Kh) // sh + 1 or Wo != (W + 2 * pw - Kw) // sw + 1:
        raise ValueError("delta spatial shape does not match the convolution geometry")
    wp, wb = _ws(ws)
    st = load_library().vgc_sqgrad_conv(_dev(x, torch.float32, "x"), _dev(delta, torch.float32, "delta"),
                                        B, C, H, W, Cout, Kh, Kw, sh, sw, ph, pw, float(scale),
                                        int(bool(accumulate)), _dev(S, torch.float32, "S"), wp, wb,
                                        _stream(stream))
    _check(st, "vgc_sqgrad_conv")
    return S


def vgc_sqgrad_conv_exact_workspace_bytes(B, C, H, W, Cout, Kh, Kw, sh, sw, ph, pw) -> int:
    return load_library().vgc_sqgrad_conv_exact_workspace_bytes(B, C, H, W, Cout, Kh, Kw, sh, sw, ph, pw)


def vgc_sqgrad_conv_exact(x, delta, kernel, stride, padding, scale: float, S, accumulate: bool = False,
                          ws=None, stream=None):
    """S[Cout,C,Kh,Kw] (+)= scale * sum over examples of the squared per-example weight gradient."""
    B, C, H, W = x.shape
    B2, Cout, Ho, Wo = delta.shape
    Kh, Kw = kernel
    sh, sw = stride
    ph, pw = padding
    if B != B2 or S.numel() != Cout * C * Kh * Kw:
        raise ValueError("shape mismatch")
    if Ho != (H + 2 * ph - Kh) // sh + 1 or Wo != (W + 2 * pw - Kw) // sw + 1:
        raise ValueError("delta spatial shape does not match the convolution geometry")
    wp, wb = _ws(ws)
    st = load_library().vgc_sqgrad_conv_exact(_dev(x, torch.float32, "x"), _dev(delta, torch.float32, "delta"),
                                              B, C, H, W, Cout, Kh, Kw, sh, sw, ph, pw, float(scale),
                                              int(bool(accumulate)), _dev(S, torch.float32, "S"), wp, wb,
                                              _stream(stream))
    _check(st, "vgc_sqgrad_conv_exact")
    return S


def vgc_sqgrad_plan_hint(concurrent_launches: int) -> None:
    """Tell the planner how many sqgrad calls run side by side (streams with separate workspaces): each then
    takes that share of the SMs.  Set it before asking for workspace sizes."""
    load_library().vgc_sqgrad_plan_hint(int(concurrent_launches))


def vgc_sqgrad_conv_batch_workspace_bytes(n_layers, B, C, H, W, Cout, Kh, Kw, sh, sw, ph, pw, exact: bool = False) -> int:
    lib = load_library()
    fn = lib.vgc_sqgrad_conv_exact_batch_workspace_bytes if exact else lib.vgc_sqgrad_conv_batch_workspace_bytes
    return fn(n_layers, B, C, H, W, Cout, Kh, Kw, sh, sw, ph, pw)


def vgc_sqgrad_conv_exact_batch(xs, deltas, kernel, stride, padding, scale: float, Ss, accumulate: bool = False,
                                ws=None, stream=None):
    """vgc_sqgrad_conv_exact for several layers of one geometry in one call."""
    return vgc_sqgrad_conv_batch(xs, deltas, kernel, stride, padding, scale, Ss, accumulate, ws, stream, exact=True)


def vgc_sqgrad_conv_batch(xs, deltas, kernel, stride, padding, scale: float, Ss, accumulate: bool = False,
                          ws=None, stream=None, exact: bool = False):
    """vgc_sqgrad_conv for several layers of one geometry (lists of tensors of equal shapes) in one call
    (``exact``: the per-example statistic, vgc_sqgrad_conv_exact_batch)."""
    n = len(xs)
    if len(deltas) != n or len(Ss) != n:
        raise ValueError("xs, deltas, Ss must have the same length")
    if n == 0:
        return Ss
    B, C, H, W = xs[0].shape
    B2, Cout, Ho, Wo = deltas[0].shape
    Kh, Kw = kernel
    sh, sw = stride
    ph, pw = padding
    if B != B2 or Ho != (H + 2 * ph - Kh) // sh + 1 or Wo != (W + 2 * pw - Kw) // sw + 1:
        raise ValueError("delta shape does not match the convolution geometry")
    for x, d, S in zip(xs, deltas, Ss):
        if tuple(x.shape) != (B, C, H, W) or tuple(d.shape) != (B, Cout, Ho, Wo) or S.numel() != Cout * C * Kh * Kw:
            raise ValueError("all layers of a batch must have the same shapes")
    ptrs = ctypes.c_void_p * n
    xp = ptrs(*[_dev(x, torch.float32, "x") for x in xs])
    dp = ptrs(*[_dev(d, torch.float32, "delta") for d in deltas])
    sp = ptrs(*[_dev(S, torch.float32, "S") for S in Ss])
    wp, wb = _ws(ws)
    lib = load_library()
    fn = lib.vgc_sqgrad_conv_exact_batch if exact else lib.vgc_sqgrad_conv_batch
    st = fn(n, xp, dp, sp, B, C, H, W, Cout, Kh, Kw, sh, sw, ph, pw, float(scale), int(bool(accumulate)), wp, wb,
            _stream(stream))
    _check(st, "vgc_sqgrad_conv_exact_batch" if exact else "vgc_sqgrad_conv_batch")
    return Ss


# ------------------------------------------------------------------------------------------ (2)
class MessageBuffers:
    """Device buffers behind a vgc_message: words, per-group exponents, counters, optional mask.

    ``counters`` is int32[4] on the device: nnz, n_criterion, n_dropped, dev_status."""

    def __init__(self, capacity: int, K: int, n: int = 0, with_mask: bool = False, device="cuda"):
        self.capacity = int(capacity)
        self.K = int(K)
        self.words = torch.empty(max(self.capacity, 1), dtype=torch.int32, device=device)
        self.group_exp = torch.empty(max(self.K, 1), dtype=torch.int32, device=device)
        self.counters = torch.zeros(4, dtype=torch.int32, device=device)
        self.mask = torch.zeros(n, dtype=torch.uint8, device=device) if with_mask else None

    def struct(self) -> _MessageStruct:
        c = self.counters.data_ptr()
        return _MessageStruct(self.words.data_ptr(), self.capacity, self.group_exp.data_ptr(), c, c + 4, c + 8,
                              self.mask.data_ptr() if self.mask is not None else None, c + 12)

    def view(self) -> _ViewStruct:
        return _ViewStruct(self.words.data_ptr(), self.counters.data_ptr(), self.group_exp.data_ptr(),
                           min(self.capacity, self.words.numel()))

    def read(self):
        """Device -> host copy (synchronises): dict with words (numpy uint32), group_exp, counters."""
        nnz, n_criterion, n_dropped, dev_status = (int(c) & 0xFFFFFFFF for c in self.counters.tolist())
        kept = min(nnz, self.capacity)
        return {"words": self.words[:kept].cpu().numpy().view("uint32"),
                "group_exp": self.group_exp[:self.K].cpu().numpy(),
                "nnz": nnz, "n_criterion": n_criterion, "n_dropped": n_dropped, "dev_status": dev_status,
                "mask": None if self.mask is None else self.mask.cpu().numpy()}


def vgc_compress_workspace_bytes(n: int, K: int) -> int:
    return load_library().vgc_compress_workspace_bytes(n, K)


def vgc_compress(g, s, r, v, group_offsets, alpha: float, zeta: float, out: MessageBuffers, ws, stream=None):
    """One step of Algorithm 1 over the flat buffer + Encode(); r, v updated in place.
    ``s=None``: v already contains this step's squared-gradient sums (sqgrad with accumulate into v)."""
    n = g.numel()
    if (s is not None and s.numel() != n) or r.numel() != n or v.numel() != n:
        raise ValueError("g, s, r, v must have the same length")
    K = group_offsets.numel() - 1
    if out.K != K:
        raise ValueError("message buffers were made for a different number of groups")
    if out.mask is not None and out.mask.numel() != n:
        raise ValueError("mask length")
    wp, wb = _ws(ws)
    msg = out.struct()
    st = load_library().vgc_compress(_dev(g, torch.float32, "g"), None if s is None else _dev(s, torch.float32, "s"),
                                     _dev(r, torch.float32, "r"), _dev(v, torch.float32, "v"), n,
                                     _dev(group_offsets, torch.int32, "group_offsets"), K, float(alpha),
                                     float(zeta), ctypes.byref(msg), wp, wb, _stream(stream))
    _check(st, "vgc_compress")
    return out


VGC_COMPRESS_STATIC_MAX_PARAMS = 1 << 21
VGC_COMPRESS_STATIC_MAX_GROUPS = 1024


def vgc_compress_static(g, s, r, v, group_offsets, alpha: float, zeta: float, out: MessageBuffers, stream=None):
    """vgc_compress for callers that cannot allocate a workspace (memory planned up front, plug-ins
    running inside someone else's step, hosts that lend only the call's tensors): the scratch is a fixed
    array inside the library, so n is limited to VGC_COMPRESS_STATIC_MAX_PARAMS.  Nothing is allocated by
    this call -- the binding passes pointers only.  Calls on one device share the scratch: do not let
    two of them overlap on the GPU.  Make the first call on a device outside any stream capture."""
    n = g.numel()
    if s.numel() != n or r.numel() != n or v.numel() != n:
        raise ValueError("g, s, r, v must have the same length")
    K = group_offsets.numel() - 1
    if out.K != K:
        raise ValueError("message buffers were made for a different number of groups")
    msg = out.struct()
    st = load_library().vgc_compress_static(_dev(g, torch.float32, "g"), _dev(s, torch.float32, "s"),
                                            _dev(r, torch.float32, "r"), _dev(v, torch.float32, "v"), n,
                                            _dev(group_offsets, torch.int32, "group_offsets"), K, float(alpha),
                                            float(zeta), ctypes.byref(msg), _stream(stream))
    _check(st, "vgc_compress_static")
    return out


# ------------------------------------------------------------------------------------------ (3)
def vgc_decode_accumulate(messages: Sequence, group_offsets, scale: float, u, dev_status, stream=None,
                          overwrite: bool = False):
    """u[idx] += scale * decoded value over all words of all messages.

    ``messages``: MessageBuffers objects, or (words int32, nnz int32[1], group_exp int32) tensor triples; the
    decoder reads at most as many words as the words tensor holds.
    ``dev_status``: int32[1] device tensor (zeroed by the caller) receiving VGC_DEV_* bits.
    ``overwrite``: write u = scale * sum instead (vgc_decode_sum): u is neither read nor needs clearing."""
    W = len(messages)
    views = (_ViewStruct * max(W, 1))()
    for w, m in enumerate(messages):
        if isinstance(m, MessageBuffers):
            views[w] = m.view()
        else:
            words, nnz, gexp = m
            views[w] = _ViewStruct(_dev(words, torch.int32, "words"), _dev(nnz, torch.int32, "nnz"),
                                   _dev(gexp, torch.int32, "group_exp"), words.numel())
    K = group_offsets.numel() - 1
    lib = load_library()
    fn = lib.vgc_decode_sum if overwrite else lib.vgc_decode_accumulate
    st = fn(views, W, _dev(group_offsets, torch.int32, "group_offsets"), K, float(scale), _dev(u, torch.float32, "u"),
            u.numel(), _dev(dev_status, torch.int32, "dev_status"), _stream(stream))
    _check(st, "vgc_decode_sum" if overwrite else "vgc_decode_accumulate")
    return u


def vgc_decode_sum(messages: Sequence, group_offsets, scale: float, u, dev_status, stream=None):
    """u = scale * (sum of all words of all messages); every element of u is written."""
    return vgc_decode_accumulate(messages, group_offsets, scale, u, dev_status, stream, overwrite=True)


# ------------------------------------------------------------------------------------------ (4)
class HybridMessageBuffers:
    """Device buffers behind a vgc_hybrid_message.  ``counters`` is int32[2]: nnz, dev_status."""

    def __init__(self, capacity: int, n: int = 0, with_mask: bool = False, device="cuda"):
        self.capacity = int(capacity)
        self.words = torch.empty(max(self.capacity, 1), dtype=torch.int32, device=device)
        self.counters = torch.zeros(2, dtype=torch.int32, device=device)
        self.mask = torch.zeros(n, dtype=torch.uint8, device=device) if with_mask else None

    def struct(self) -> _HybridMessageStruct:
        c = self.counters.data_ptr()
        return _HybridMessageStruct(self.words.data_ptr(), self.capacity, c,
                                    self.mask.data_ptr() if self.mask is not None else None, c + 4)

    def view(self) -> _ViewStruct:
        return _ViewStruct(self.words.data_ptr(), self.counters.data_ptr(), None, min(self.capacity, self.words.numel()))

    def read(self):
        nnz, dev_status = (int(c) & 0xFFFFFFFF for c in self.counters.tolist())
        return {"words": self.words[:min(nnz, self.capacity)].cpu().numpy().view("uint32"), "nnz": nnz,
                "dev_status": dev_status, "mask": None if self.mask is None else self.mask.cpu().numpy()}


def vgc_compress_hybrid_workspace_bytes(n: int) -> int:
    return load_library().vgc_compress_hybrid_workspace_bytes(n)


def vgc_compress_hybrid(g, s, r, v, alpha: float, zeta: float, tau: float, out: HybridMessageBuffers, ws,
                        correction_from_updated_r: bool = False, stream=None):
    """One step of Algorithm 2 over the flat buffer; r, v updated in place.  ``s=None`` as for vgc_compress."""
    n = g.numel()
    if (s is not None and s.numel() != n) or r.numel() != n or v.numel() != n:
        raise ValueError("g, s, r, v must have the same length")
    if out.mask is not None and out.mask.numel() != n:
        raise ValueError("mask length")
    wp, wb = _ws(ws)
    msg = out.struct()
    st = load_library().vgc_compress_hybrid(
        _dev(g, torch.float32, "g"), None if s is None else _dev(s, torch.float32, "s"), _dev(r, torch.float32, "r"),
        _dev(v, torch.float32, "v"), n, float(alpha), float(zeta), float(tau), int(bool(correction_from_updated_r)),
        ctypes.byref(msg), wp, wb, _stream(stream))
    _check(st, "vgc_compress_hybrid")
    return out


def vgc_decode_sum_hybrid(messages: Sequence, tau: float, scale: float, u, dev_status, stream=None):
    """u = scale * (sum of +-tau over all words); every element of u is written."""
    return vgc_decode_accumulate_hybrid(messages, tau, scale, u, dev_status, stream, overwrite=True)


def vgc_decode_accumulate_hybrid(messages: Sequence, tau: float, scale: float, u, dev_status, stream=None,
                                 overwrite: bool = False):
    """u[idx] += scale * (+-tau) over all words of all messages (HybridMessageBuffers or (words, nnz) pairs)."""
    W = len(messages)
    views = (_ViewStruct * max(W, 1))()
    for w, m in enumerate(messages):
        if isinstance(m, HybridMessageBuffers):
            views[w] = m.view()
        else:
            words, nnz = m
            views[w] = _ViewStruct(_dev(words, torch.int32, "words"), _dev(nnz, torch.int32, "nnz"), None, words.numel())
    lib = load_library()
    fn = lib.vgc_decode_sum_hybrid if overwrite else lib.vgc_decode_accumulate_hybrid
    st = fn(views, W, float(tau), float(scale), _dev(u, torch.float32, "u"), u.numel(),
            _dev(dev_status, torch.int32, "dev_status"), _stream(stream))
    _check(st, "vgc_decode_accumulate_hybrid")
    return u


# ------------------------------------------------------------------------------------------ (5)
def vgc_pack_bound_bytes(max_words: int) -> int:
    return load_library().vgc_pack_bound_bytes(int(max_words))


def vgc_pack_workspace_bytes(max_words: int) -> int:
    return load_library().vgc_pack_workspace_bytes(int(max_words))


def vgc_pack_indices(words, nnz, packed, packed_bytes, dev_status, ws, stream=None):
    """words int32 [max_words] + nnz int32 [1] (device) -> packed uint8 (device): the index field as differences in
    the base-128 code; packed_bytes int32 [1] (device) receives the stream's length."""
    wp, wb = _ws(ws)
    st = load_library().vgc_pack_indices(_dev(words, torch.int32, "words"), _dev(nnz, torch.int32, "nnz"), words.numel(),
                                         _dev(packed, torch.uint8, "packed"), packed.numel(),
                                         _dev(packed_bytes, torch.int32, "packed_bytes"),
                                         _dev(dev_status, torch.int32, "dev_status"), wp, wb, _stream(stream))
    _check(st, "vgc_pack_indices")
    return packed


def vgc_unpack_indices(packed, nnz, words, dev_status, stream=None):
    """The inverse of vgc_pack_indices: rebuilds min(nnz, words.numel()) words (device int32)."""
    st = load_library().vgc_unpack_indices(_dev(packed, torch.uint8, "packed"), _dev(nnz, torch.int32, "nnz"), words.numel(),
                                           _dev(words, torch.int32, "words"), _dev(dev_status, torch.int32, "dev_status"),
                                           _stream(stream))
    _check(st, "vgc_unpack_indices")
    return words


def _host(t: torch.Tensor, dtype, name: str) -> int:
    if not isinstance(t, torch.Tensor) or t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous CPU tensor of {dtype}")
    return t.data_ptr()


def vgc_step_host(layers, g_host, g_dev, s_dev, r, v, group_offsets, alpha, zeta, scale, out: MessageBuffers,
                  words_host, counters_host, ws_sqgrad, ws_compress, stream=None):
    """One worker step from host buffers.  ``layers``: list of dicts with keys is_conv, B, C, H, W, Cout,
    Kh, Kw, stride, pad, x_host, delta_host (CPU, ideally pinned) and x_dev, delta_dev (CUDA staging).
    Returns (nnz, n_criterion, n_dropped, dev_status) as read back into ``counters_host``."""
    arr = (_LayerHostStruct * max(len(layers), 1))()
    for k, L in enumerate(layers):
        arr[k] = _LayerHostStruct(int(L["is_conv"]), L["B"], L["C"], L.get("H", 1), L.get("W", 1), L["Cout"],
                                  L.get("Kh", 1), L.get("Kw", 1), L.get("stride", 1), L.get("stride", 1),
                                  L.get("pad", 0), L.get("pad", 0),
                                  _host(L["x_host"], torch.float32, "x_host"), _host(L["delta_host"], torch.float32, "delta_host"),
                                  _dev(L["x_dev"], torch.float32, "x_dev"), _dev(L["delta_dev"], torch.float32, "delta_dev"))
    n = g_dev.numel()
    K = group_offsets.numel() - 1
    wsp, wsb = _ws(ws_sqgrad)
    wcp, wcb = _ws(ws_compress)
    msg = out.struct()
    st = load_library().vgc_step_host(arr, len(layers), _host(g_host, torch.float32, "g_host"),
                                      _dev(g_dev, torch.float32, "g_dev"), _dev(s_dev, torch.float32, "s_dev"),
                                      _dev(r, torch.float32, "r"), _dev(v, torch.float32, "v"), n,
                                      _dev(group_offsets, torch.int32, "group_offsets"), K, float(alpha), float(zeta),
                                      float(scale), ctypes.byref(msg), _host(words_host, torch.int32, "words_host"),
                                      _host(counters_host, torch.int32, "counters_host"), wsp, wsb, wcp, wcb,
                                      _stream(stream))
    _check(st, "vgc_step_host")
    return tuple(int(c) & 0xFFFFFFFF for c in counters_host.tolist())


def offsets_tensor(offsets, device="cuda") -> torch.Tensor:
    """Group offsets (uint32 values < 2^31) as the int32 device tensor the binding passes."""
    import numpy as np
    return torch.from_numpy(np.asarray(offsets, dtype=np.int64).astype(np.int32)).to(device)
