"""ctypes binding of libdab.so: same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors used as device memory; every step of the method runs inside the
library's kernels.  If the library has not been built or cannot be loaded, importing the functions
raises: there is no other implementation to fall back to.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdab.so")

DAB_OK = 0
DAB_MAX_N = 16384
ROW_DEGENERATE = 1
ROW_NONFINITE = 2

EXPORTS = ("dab_status_string", "dab_words_per_row", "dab_default_ld", "dab_binarize", "dab_pack", "dab_binary_gemm",
           "dab_conv_output_size", "dab_binary_conv_workspace", "dab_binary_conv", "dab_binarize_patches",
           "dab_binary_conv_contract", "dab_sign_binarize", "dab_sign_patches", "dab_binary_conv_sign", "dab_binary_conv_host_workspace",
           "dab_binary_conv_host", "dab_binary_conv_static_capacity", "dab_binary_conv_static", "dab_popc_probe",
           "dab_set_contraction", "dab_get_contraction", "dab_contraction_wait_failures", "dab_wbin_conv", "dab_wbin_conv_workspace", "dab_binarize_train", "dab_binarize_backward", "dab_set_patch_coder", "dab_get_patch_coder", "dab_binary_conv_host_async", "dab_binary_conv_host_wait",
           "dab_network_output_shape", "dab_network_workspace", "dab_network_forward", "dab_debug_bounds_enabled",
           "dab_debug_bounds_report")


class DabError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


class ConvDesc(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("N", "C", "H", "W", "Cout", "kh", "kw", "stride_h", "stride_w", "pad_h", "pad_w")]


_lib = None


def use_library(path: str) -> None:
    """Load the library from `path` instead of the in-tree libdab.so (e.g. the bounds-checking libdab_debug.so).
    Only before the first call into the library."""
    global LIB_PATH
    if _lib is not None and os.path.abspath(path) != os.path.abspath(LIB_PATH):
        raise RuntimeError("a library is already loaded from %s" % LIB_PATH)
    LIB_PATH = path


class BoundsReport(C.Structure):
    _fields_ = [("violations", C.c_uint64), ("index", C.c_int64), ("extent", C.c_int64), ("file_hash", C.c_uint32),
                ("line", C.c_int32)]


def lib() -> C.CDLL:
    """Loads libdab.so (raises if it is missing: build it with `python -m paper_1804_02941_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libdab.so not built at %s; run `python -m paper_1804_02941_b200.build`" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        L.dab_status_string.restype = C.c_char_p
        L.dab_status_string.argtypes = [C.c_int]
        L.dab_words_per_row.restype = C.c_int32
        L.dab_default_ld.restype = C.c_int32
        L.dab_binary_conv_workspace.restype = C.c_size_t
        L.dab_binary_conv_host_workspace.restype = C.c_size_t
        vp, i64, i32 = C.c_void_p, C.c_int64, C.c_int32
        L.dab_binarize.argtypes = [vp, i64, i32, i64, vp, vp, vp, vp, i32, vp, vp]
        L.dab_pack.argtypes = [vp, i64, i32, i64, vp, i32, vp, vp]
        L.dab_binary_gemm.argtypes = [i64, i64, i32, vp, i32, vp, vp, vp, vp, i32, vp, vp, vp, vp, i64, vp, i64, vp]
        L.dab_conv_output_size.argtypes = [vp, vp, vp]
        L.dab_binary_conv_workspace.argtypes = [vp]
        L.dab_binary_conv_host_workspace.argtypes = [vp]
        L.dab_binary_conv.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp, C.c_size_t, vp, vp, vp, vp, i32, vp, vp, vp]
        L.dab_binarize_patches.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp, vp]
        L.dab_sign_patches.argtypes = L.dab_binarize_patches.argtypes
        L.dab_sign_binarize.argtypes = L.dab_binarize.argtypes
        L.dab_binary_conv_sign.argtypes = L.dab_binary_conv.argtypes
        L.dab_binary_conv_contract.argtypes = [vp, vp, i32, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp]
        L.dab_binary_conv_host.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp, C.c_size_t, vp]
        L.dab_binary_conv_host_async.argtypes = L.dab_binary_conv_host.argtypes
        L.dab_binary_conv_host_wait.argtypes = [vp]
        L.dab_binary_conv_static_capacity.restype = C.c_size_t
        L.dab_binary_conv_static_capacity.argtypes = []
        L.dab_binary_conv_static.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp]
        L.dab_popc_probe.argtypes = [vp, i32, i32, vp]
        L.dab_debug_bounds_enabled.restype = i32
        L.dab_debug_bounds_report.argtypes = [C.POINTER(BoundsReport), i32]
        L.dab_wbin_conv.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, C.c_size_t, vp]
        L.dab_wbin_conv_workspace.restype = C.c_size_t
        L.dab_wbin_conv_workspace.argtypes = [vp]
        L.dab_binarize_train.argtypes = [vp, i64, i32, i64, vp, i64, vp, i64, vp, vp, vp, vp, i32, vp, vp]
        L.dab_binarize_backward.argtypes = [vp, i64, i32, i64, vp, i32, vp, vp, i64, vp, i64, vp]
        L.dab_set_contraction.argtypes = [i32]
        L.dab_set_patch_coder.argtypes = [i32]
        L.dab_get_patch_coder.argtypes = []
        L.dab_get_contraction.argtypes = []
        L.dab_contraction_wait_failures.argtypes = [vp]
        L.dab_network_output_shape.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp]
        L.dab_network_workspace.restype = C.c_size_t
        L.dab_network_workspace.argtypes = [vp, i32, i32, i32, i32, i32]
        L.dab_network_forward.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp, C.c_size_t, vp, vp]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().dab_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != DAB_OK:
        raise DabError(status, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _dev(t, dtype, name):
    if not isinstance(t, torch.Tensor) or not t.is_cuda or t.dtype != dtype:
        raise TypeError("%s must be a CUDA tensor of dtype %s" % (name, dtype))
    return t


# ------------------------------------------------------------------------------------------------------------
# Output allocation.  With guards switched on (the GPU tests do this), every output tensor this module creates sits
# between two 256-byte guard zones filled with a pattern; guards_check() verifies that no kernel wrote into them.
# It stands in for a memory checker: it catches writes just before or behind an output, not every stray access.
# ------------------------------------------------------------------------------------------------------------
_GUARD = 256
_GUARD_BYTE = 0xA5
_guards_on = False
_guarded = []


def guards_enable(on: bool) -> None:
    global _guards_on
    _guards_on = bool(on)
    if not on:
        _guarded.clear()


def _new(shape, dtype, device):
    if not _guards_on:
        return torch.empty(shape, dtype=dtype, device=device)
    if isinstance(shape, int):
        shape = (shape,)
    numel = 1
    for d in shape:
        numel *= int(d)
    nbytes = numel * torch.empty((), dtype=dtype).element_size()
    pad = (-nbytes) % 16
    raw = torch.full((_GUARD + nbytes + pad + _GUARD,), _GUARD_BYTE, dtype=torch.uint8, device=device)
    _guarded.append((raw, nbytes))
    return raw[_GUARD:_GUARD + nbytes].view(dtype).view(tuple(int(d) for d in shape))


def guards_check() -> int:
    """Verifies the guard zones of every tensor handed out since the last check; returns how many were checked."""
    torch.cuda.synchronize()
    n = len(_guarded)
    for raw, nbytes in _guarded:
        front, back = raw[:_GUARD], raw[_GUARD + nbytes:]
        if not (bool((front == _GUARD_BYTE).all()) and bool((back == _GUARD_BYTE).all())):
            _guarded.clear()
            raise AssertionError("a kernel wrote outside an output tensor of %d bytes" % nbytes)
    _guarded.clear()
    return n


def dab_words_per_row(n: int) -> int:
    return int(lib().dab_words_per_row(C.c_int32(n)))


def dab_default_ld(n: int) -> int:
    return int(lib().dab_default_ld(C.c_int32(n)))


@dataclass
class Coded:
    """Two-level codes of a batch of rows, as device tensors."""
    mask: torch.Tensor    # rows x ld int32 (bit pattern of the uint32 words)
    K: torch.Tensor       # rows int32
    alpha: torch.Tensor   # rows fp32
    beta: torch.Tensor    # rows fp32
    flags: torch.Tensor   # rows int32 (ROW_* bits)
    n: int

    @property
    def ld(self) -> int:
        return self.mask.shape[1]


def dab_sign_binarize(values: torch.Tensor, ld_mask: int | None = None, stream=None) -> "Coded":
    """Sign coding of rows (mask = [x >= 0], alpha = mean|x|, beta = -alpha); outputs as dab_binarize."""
    return dab_binarize(values, ld_mask, stream, _entry="dab_sign_binarize")


def dab_binarize(values: torch.Tensor, ld_mask: int | None = None, stream=None, _entry: str = "dab_binarize") -> Coded:
    """rows x n fp32 (row stride = values.stride(0)) -> K, alpha, beta, packed mask, flags."""
    _dev(values, torch.float32, "values")
    if values.dim() != 2 or values.stride(1) != 1:
        raise ValueError("values must be 2-D with unit inner stride")
    rows, n = values.shape
    ld = dab_default_ld(n) if ld_mask is None else ld_mask
    dev = values.device
    out = Coded(_new((rows, ld), torch.int32, dev), _new(rows, torch.int32, dev),
                _new(rows, torch.float32, dev), _new(rows, torch.float32, dev),
                _new(rows, torch.int32, dev), n)
    ldv = values.stride(0) if rows > 1 else max(n, values.stride(0))
    st = getattr(lib(), _entry)(_ptr(values), rows, n, ldv, _ptr(out.K), _ptr(out.alpha), _ptr(out.beta),
                                _ptr(out.mask), ld, _ptr(out.flags), _stream(stream))
    _check(st, _entry)
    return out


def dab_binarize_into(values, K, alpha, beta, mask, flags=None, stream=None) -> None:
    """Same call with caller-provided outputs (no allocation)."""
    rows, n = values.shape
    ldv = values.stride(0) if rows > 1 else max(n, values.stride(0))
    st = lib().dab_binarize(_ptr(values), rows, n, ldv, _ptr(K), _ptr(alpha), _ptr(beta), _ptr(mask), mask.stride(0),
                            _ptr(flags), _stream(stream))
    _check(st, "dab_binarize")


def dab_pack(bits: torch.Tensor, ld_mask: int | None = None, stream=None):
    """rows x n uint8 (0/1) -> (rows x ld int32 words, K int32)."""
    _dev(bits, torch.uint8, "bits")
    if bits.dim() != 2 or bits.stride(1) != 1:
        raise ValueError("bits must be 2-D with unit inner stride")
    rows, n = bits.shape
    ld = dab_default_ld(n) if ld_mask is None else ld_mask
    mask = _new((rows, ld), torch.int32, bits.device)
    K = _new(rows, torch.int32, bits.device)
    ldb = bits.stride(0) if rows > 1 else max(n, bits.stride(0))
    _check(lib().dab_pack(_ptr(bits), rows, n, ldb, _ptr(mask), ld, _ptr(K), _stream(stream)), "dab_pack")
    return mask, K


def dab_binary_gemm(a: Coded, b: Coded, want_p11: bool = False, out: torch.Tensor | None = None, stream=None):
    """C[i,j] = coded row i of `a` (activation side) . coded row j of `b` (weight side); M x N fp32."""
    if a.n != b.n:
        raise ValueError("row lengths differ")
    M, N = a.mask.shape[0], b.mask.shape[0]
    dev = a.mask.device
    Cm = _new((M, N), torch.float32, dev) if out is None else out
    p11 = _new((M, N), torch.int32, dev) if want_p11 else None
    st = lib().dab_binary_gemm(M, N, a.n, _ptr(a.mask), a.ld, _ptr(a.K), _ptr(a.alpha), _ptr(a.beta), _ptr(b.mask),
                               b.ld, _ptr(b.K), _ptr(b.alpha), _ptr(b.beta), _ptr(Cm), Cm.stride(0) if M > 1 else max(N, 1),
                               _ptr(p11), N, _stream(stream))
    _check(st, "dab_binary_gemm")
    return (Cm, p11) if want_p11 else Cm


def make_desc(x_shape, Cout, kh, kw, stride=(1, 1), pad=(0, 0)) -> ConvDesc:
    N, Cc, H, W = x_shape
    return ConvDesc(N, Cc, H, W, Cout, kh, kw, stride[0], stride[1], pad[0], pad[1])


def dab_conv_output_size(desc: ConvDesc):
    ho, wo = C.c_int32(), C.c_int32()
    _check(lib().dab_conv_output_size(C.byref(desc), C.byref(ho), C.byref(wo)), "dab_conv_output_size")
    return ho.value, wo.value


def dab_binary_conv_workspace(desc: ConvDesc) -> int:
    return int(lib().dab_binary_conv_workspace(C.byref(desc)))


def dab_binary_conv_host_workspace(desc: ConvDesc) -> int:
    return int(lib().dab_binary_conv_host_workspace(C.byref(desc)))


@dataclass
class ConvDetails:
    pK: torch.Tensor
    pgamma: torch.Tensor
    pdelta: torch.Tensor
    pmask: torch.Tensor
    pflags: torch.Tensor
    p11: torch.Tensor


def dab_binary_conv(x: torch.Tensor, w: Coded, kh: int, kw: int, stride=(1, 1), pad=(0, 0), details: bool = False,
                    y: torch.Tensor | None = None, workspace: torch.Tensor | None = None, stream=None,
                    sign_inputs: bool = False):
    """x: N x C x H x W fp32 (contiguous); w: filters coded by dab_binarize on [Cout x C*kh*kw] -> y NCHW fp32.
    sign_inputs: code the patches by sign and mean magnitude (dab_binary_conv_sign) instead of the optimal split."""
    _dev(x, torch.float32, "x")
    if not x.is_contiguous():
        raise ValueError("x must be contiguous NCHW")
    Cout = w.mask.shape[0]
    desc = make_desc(tuple(x.shape), Cout, kh, kw, stride, pad)
    if w.n != x.shape[1] * kh * kw:
        raise ValueError("filter length does not match C*kh*kw")
    Ho, Wo = dab_conv_output_size(desc)
    dev = x.device
    if y is None:
        y = _new((x.shape[0], Cout, Ho, Wo), torch.float32, dev)
    need = dab_binary_conv_workspace(desc)
    if workspace is None:
        workspace = _new(need, torch.uint8, dev)
    det = None
    if details:
        P = x.shape[0] * Ho * Wo
        det = ConvDetails(_new(P, torch.int32, dev), _new(P, torch.float32, dev),
                          _new(P, torch.float32, dev),
                          _new((P, dab_default_ld(w.n)), torch.int32, dev),
                          _new(P, torch.int32, dev),
                          _new((P, Cout), torch.int32, dev))
    entry = lib().dab_binary_conv_sign if sign_inputs else lib().dab_binary_conv
    st = entry(C.byref(desc), _ptr(x), _ptr(w.mask), w.ld, _ptr(w.K), _ptr(w.alpha), _ptr(w.beta),
                               _ptr(y), _ptr(workspace), workspace.numel(),
                               _ptr(det.pK) if det else None, _ptr(det.pgamma) if det else None,
                               _ptr(det.pdelta) if det else None, _ptr(det.pmask) if det else None,
                               det.pmask.shape[1] if det else 0, _ptr(det.pflags) if det else None,
                               _ptr(det.p11) if det else None, _stream(stream))
    _check(st, "dab_binary_conv")
    return (y, det) if details else y


def dab_sign_patches(desc: ConvDesc, x: torch.Tensor, pK, pgamma, pdelta, pmask, pflags=None, stream=None) -> None:
    """Sign coding of every patch (stage 1 of dab_binary_conv_sign) with caller-provided outputs."""
    st = lib().dab_sign_patches(C.byref(desc), _ptr(x), _ptr(pK), _ptr(pgamma), _ptr(pdelta), _ptr(pmask),
                                pmask.stride(0), _ptr(pflags), _stream(stream))
    _check(st, "dab_sign_patches")


def dab_binarize_patches(desc: ConvDesc, x: torch.Tensor, pK, pgamma, pdelta, pmask, pflags=None, stream=None) -> None:
    """Stage 1 of dab_binary_conv with caller-provided outputs (pmask: patches x ld int32)."""
    st = lib().dab_binarize_patches(C.byref(desc), _ptr(x), _ptr(pK), _ptr(pgamma), _ptr(pdelta), _ptr(pmask),
                                    pmask.stride(0), _ptr(pflags), _stream(stream))
    _check(st, "dab_binarize_patches")


def dab_binary_conv_contract(desc: ConvDesc, pmask, pK, pgamma, pdelta, w: Coded, y: torch.Tensor, p11=None,
                             stream=None) -> None:
    """Stage 2 of dab_binary_conv: coded patches x coded filters -> y (NCHW)."""
    st = lib().dab_binary_conv_contract(C.byref(desc), _ptr(pmask), pmask.stride(0), _ptr(pK), _ptr(pgamma),
                                        _ptr(pdelta), _ptr(w.mask), w.ld, _ptr(w.K), _ptr(w.alpha), _ptr(w.beta),
                                        _ptr(y), _ptr(p11), _stream(stream))
    _check(st, "dab_binary_conv_contract")


def dab_binary_conv_host(x_host: torch.Tensor, w: Coded, kh: int, kw: int, stride=(1, 1), pad=(0, 0),
                         y_host: torch.Tensor | None = None, workspace: torch.Tensor | None = None, stream=None,
                         wait: bool = True):
    """Host tensors in and out (pinned memory recommended); the library does the copies.  wait=False queues the
    layer and returns (dab_binary_conv_host_async): call dab_binary_conv_host_wait before reading y_host."""
    if x_host.is_cuda or x_host.dtype != torch.float32 or not x_host.is_contiguous():
        raise TypeError("x_host must be a contiguous fp32 host tensor")
    Cout = w.mask.shape[0]
    desc = make_desc(tuple(x_host.shape), Cout, kh, kw, stride, pad)
    Ho, Wo = dab_conv_output_size(desc)
    if y_host is None:
        y_host = torch.empty((x_host.shape[0], Cout, Ho, Wo), dtype=torch.float32).pin_memory()
    need = dab_binary_conv_host_workspace(desc)
    if workspace is None:
        if not wait:
            raise ValueError("wait=False needs a caller-owned workspace that outlives the queued work")
        workspace = _new(need, torch.uint8, w.mask.device)
    fn = lib().dab_binary_conv_host if wait else lib().dab_binary_conv_host_async
    st = fn(C.byref(desc), C.c_void_p(x_host.data_ptr()), _ptr(w.mask), w.ld, _ptr(w.K),
                                    _ptr(w.alpha), _ptr(w.beta), C.c_void_p(y_host.data_ptr()), _ptr(workspace),
                                    workspace.numel(), _stream(stream))
    _check(st, "dab_binary_conv_host")
    return y_host


def dab_binary_conv_host_wait(stream=None) -> None:
    """Blocks until every layer queued with wait=False on the current device has finished."""
    _check(lib().dab_binary_conv_host_wait(_stream(stream)), "dab_binary_conv_host_wait")


def dab_binary_conv_static_capacity() -> int:
    return int(lib().dab_binary_conv_static_capacity())


def dab_binary_conv_static(x: torch.Tensor, w: Coded, kh: int, kw: int, stride=(1, 1), pad=(0, 0),
                           y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """dab_binary_conv on the library's built-in scratch array (no workspace; see include/dab.h for its limits).

    Only the output tensor is created here when the caller passes none; the library call itself allocates nothing."""
    _dev(x, torch.float32, "x")
    if not x.is_contiguous():
        raise ValueError("x must be contiguous NCHW")
    Cout = w.mask.shape[0]
    desc = make_desc(tuple(x.shape), Cout, kh, kw, stride, pad)
    Ho, Wo = dab_conv_output_size(desc)
    if y is None:
        y = _new((x.shape[0], Cout, Ho, Wo), torch.float32, x.device)
    st = lib().dab_binary_conv_static(C.byref(desc), _ptr(x), _ptr(w.mask), w.ld, _ptr(w.K), _ptr(w.alpha),
                                      _ptr(w.beta), _ptr(y), _stream(stream))
    _check(st, "dab_binary_conv_static")
    return y


def dab_wbin_conv_workspace(desc: ConvDesc) -> int:
    return int(lib().dab_wbin_conv_workspace(C.byref(desc)))


def dab_wbin_conv(x: torch.Tensor, w: Coded, kh: int, kw: int, stride=(1, 1), pad=(0, 0),
                  y: torch.Tensor | None = None, workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Weights-only binarized convolution: fp32 NCHW input against the two-level filters `w`."""
    _dev(x, torch.float32, "x")
    if not x.is_contiguous():
        raise ValueError("x must be contiguous NCHW")
    Cout = w.mask.shape[0]
    desc = make_desc(tuple(x.shape), Cout, kh, kw, stride, pad)
    Ho, Wo = dab_conv_output_size(desc)
    if y is None:
        y = _new((x.shape[0], Cout, Ho, Wo), torch.float32, x.device)
    need = dab_wbin_conv_workspace(desc)
    if workspace is None:
        workspace = _new(need, torch.uint8, x.device)
    st = lib().dab_wbin_conv(C.byref(desc), _ptr(x), _ptr(w.mask), w.ld, _ptr(w.alpha), _ptr(w.beta), _ptr(y),
                             _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream))
    _check(st, "dab_wbin_conv")
    return y


def dab_binarize_train(W: torch.Tensor, want_dense: bool = True, stream=None):
    """Algorithm 2 steps 4-13 on the rows of W: returns (Wc, Coded of Wc, Wt or None)."""
    _dev(W, torch.float32, "W")
    if W.dim() != 2 or W.stride(1) != 1:
        raise ValueError("W must be a 2-D tensor with contiguous rows")
    rows, n = W.shape
    ld = dab_default_ld(n)
    dev = W.device
    Wc = _new((rows, n), torch.float32, dev)
    Wt = _new((rows, n), torch.float32, dev) if want_dense else None
    out = Coded(_new((rows, ld), torch.int32, dev), _new(rows, torch.int32, dev),
                _new(rows, torch.float32, dev), _new(rows, torch.float32, dev),
                _new(rows, torch.int32, dev), n)
    st = lib().dab_binarize_train(_ptr(W), rows, n, W.stride(0) if rows > 1 else n, _ptr(Wc), n, _ptr(Wt), n, _ptr(out.K),
                                  _ptr(out.alpha), _ptr(out.beta), _ptr(out.mask), ld, _ptr(out.flags), _stream(stream))
    _check(st, "dab_binarize_train")
    return Wc, out, Wt


def dab_binarize_backward(Wc: torch.Tensor, coded: Coded, grad_Wt: torch.Tensor, stream=None) -> torch.Tensor:
    """Theorem 4: the gradient with respect to the real-valued weights from the gradient with respect to W~."""
    _dev(Wc, torch.float32, "Wc")
    _dev(grad_Wt, torch.float32, "grad_Wt")
    rows, n = Wc.shape
    if not (Wc.is_contiguous() and grad_Wt.is_contiguous() and grad_Wt.shape == Wc.shape):
        raise ValueError("Wc and grad_Wt must be contiguous and of one shape")
    gW = _new(tuple(Wc.shape), Wc.dtype, Wc.device)
    st = lib().dab_binarize_backward(_ptr(Wc), rows, n, n, _ptr(coded.mask), coded.ld, _ptr(coded.K), _ptr(grad_Wt), n,
                                     _ptr(gW), n, _stream(stream))
    _check(st, "dab_binarize_backward")
    return gW


def dab_popc_probe(blocks: int, iters: int, sink: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    if sink is None:
        sink = torch.empty(blocks * 256, dtype=torch.int32, device="cuda")
    _check(lib().dab_popc_probe(_ptr(sink), blocks, iters, _stream(stream)), "dab_popc_probe")
    return sink


def dab_debug_bounds_enabled() -> bool:
    return bool(lib().dab_debug_bounds_enabled())


def dab_debug_bounds_report(reset: bool = True) -> dict:
    """Violations recorded by a library built with the index checks (DabError with status 2 from an ordinary one).
    `file` is the name of the source file of the first violation, found by hashing the names under csrc/."""
    r = BoundsReport()
    _check(lib().dab_debug_bounds_report(C.byref(r), int(reset)), "dab_debug_bounds_report")
    name = None
    if r.violations:
        for f in os.listdir(os.path.join(_HERE, "csrc")):
            h = 2166136261
            for ch in f.encode():
                h = ((h ^ ch) * 16777619) & 0xFFFFFFFF
            if h == r.file_hash:
                name = f
    return {"violations": int(r.violations), "index": int(r.index), "extent": int(r.extent), "file": name, "line": int(r.line)}


CONTRACT_AUTO, CONTRACT_TENSOR, CONTRACT_POPC = 0, 1, 2


def dab_set_contraction(path: int) -> None:
    """Process-wide choice of the contraction kernel: CONTRACT_AUTO (default), CONTRACT_TENSOR or CONTRACT_POPC."""
    _check(lib().dab_set_contraction(int(path)), "dab_set_contraction")


PATCHES_AUTO, PATCHES_SORT, PATCHES_HIST, PATCHES_PIXEL = 0, 1, 2, 3


def dab_set_patch_coder(coder: int) -> None:
    """PATCHES_AUTO (default), PATCHES_SORT (full sort per row), PATCHES_HIST (histogram-pruned search per row) or
    PATCHES_PIXEL (per-pixel histograms shared by overlapping patches); see include/dab.h."""
    _check(lib().dab_set_patch_coder(int(coder)), "dab_set_patch_coder")


def dab_get_patch_coder() -> int:
    return int(lib().dab_get_patch_coder())


def dab_get_contraction() -> int:
    return int(lib().dab_get_contraction())


def dab_contraction_wait_failures() -> int:
    """Barrier waits of the tensor-core kernel that ran out on the current device (0 on a correct run)."""
    c = C.c_uint32(0)
    _check(lib().dab_contraction_wait_failures(C.byref(c)), "dab_contraction_wait_failures")
    return int(c.value)


# ------------------------------------------------------------------------------------------------------------
# Whole networks (dab_network_forward): the layer records are filled from torch tensors; nothing is computed here
# ------------------------------------------------------------------------------------------------------------
LAYER_KINDS = {"conv_dense": 0, "conv_binary": 1, "affine": 2, "relu": 3, "maxpool": 4, "save": 5, "add": 6}


class Layer(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("kind", "on_saved", "Cout", "kh", "kw", "stride_h", "stride_w", "pad_h", "pad_w", "ldw")] + \
               [(k, C.c_void_p) for k in ("d_weights", "d_bias", "d_wmask", "d_wK", "d_walpha", "d_wbeta", "d_scale", "d_shift")]


class Network:
    """A chain of layers resident on a device: the C records plus the tensors they point to (kept alive here).
    layers: dicts as produced by dab_synth.networks ("kind", geometry, numpy or torch weights); the filters of the
    binarized layers are coded once, by dab_binarize, when the network is built."""

    def __init__(self, layers, device="cuda"):
        self.device = torch.device(device)
        self.keep = []
        self.records = (Layer * len(layers))()
        self.kinds = [l["kind"] for l in layers]
        for rec, l in zip(self.records, layers):
            rec.kind = LAYER_KINDS[l["kind"]]
            rec.on_saved = 1 if l.get("on_saved") else 0
            if "kh" in l:
                rec.kh, rec.kw = l["kh"], l["kw"]
                rec.stride_h, rec.stride_w = l["stride"]
                rec.pad_h, rec.pad_w = l["pad"]
            if l["kind"] == "conv_dense":
                w = self._t(l["w"])
                rec.Cout, rec.d_weights = w.shape[0], w.data_ptr()
                if l.get("bias") is not None:
                    rec.d_bias = self._t(l["bias"]).data_ptr()
            elif l["kind"] == "conv_binary":
                coded = dab_binarize(self._t(l["w"]))
                self.keep.append(coded)
                rec.Cout, rec.ldw = coded.mask.shape[0], coded.ld
                rec.d_wmask, rec.d_wK = coded.mask.data_ptr(), coded.K.data_ptr()
                rec.d_walpha, rec.d_wbeta = coded.alpha.data_ptr(), coded.beta.data_ptr()
            elif l["kind"] == "affine":
                rec.d_scale, rec.d_shift = self._t(l["scale"]).data_ptr(), self._t(l["shift"]).data_ptr()

    def _t(self, a):
        t = a if isinstance(a, torch.Tensor) else torch.from_numpy(a)
        t = t.to(self.device, torch.float32).contiguous()
        self.keep.append(t)
        return t

    def __len__(self):
        return len(self.records)


def dab_network_output_shape(net: Network, x_shape):
    N, Cc, H, W = x_shape
    co, ho, wo = C.c_int32(0), C.c_int32(0), C.c_int32(0)
    _check(lib().dab_network_output_shape(net.records, len(net), N, Cc, H, W, C.byref(co), C.byref(ho), C.byref(wo)),
           "dab_network_output_shape")
    return co.value, ho.value, wo.value


def dab_network_forward(net: Network, x: torch.Tensor, keep_layers: bool = False, layer_shapes=None, stream=None):
    """Runs the chain on x (N x C x H x W fp32, contiguous).  keep_layers: also return every layer's output tensor
    (layer_shapes: their shapes, one (C, H, W) per layer, as the caller knows them from the network definition)."""
    _dev(x, torch.float32, "x")
    N, Cc, H, W = x.shape
    co, ho, wo = dab_network_output_shape(net, tuple(x.shape))
    y = _new((N, co, ho, wo), torch.float32, x.device)
    need = int(lib().dab_network_workspace(net.records, len(net), N, Cc, H, W))
    ws = _new(need, torch.uint8, x.device)
    outs, ptrs = None, None
    if keep_layers:
        outs = [_new((N,) + tuple(s), torch.float32, x.device) for s in layer_shapes]
        ptrs = (C.c_void_p * len(net))(*[o.data_ptr() for o in outs])
    _check(lib().dab_network_forward(net.records, len(net), N, Cc, H, W, _ptr(x), _ptr(y), _ptr(ws), need, ptrs, _stream(stream)),
           "dab_network_forward")
    return (y, outs) if keep_layers else y
