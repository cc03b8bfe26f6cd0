"""numpy front end of the CPU checker (``dab_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Nothing under this directory may be imported by the
CUDA library's package; only the tests, the smoke check and the CPU-baseline
leg of the benchmark use it.  The C file is compiled with gcc on first use.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dab_oracle.c")
_HDR = os.path.join(_HERE, "dab_oracle.h")
_LIB = os.path.join(_HERE, "libdab_oracle.so")

FLAG_DEGENERATE = 1
FLAG_NONFINITE = 2


def build(force: bool = False) -> str:
    """Compile the checker (gcc, -O2, no FMA contraction, OpenMP over independent rows)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC",
                               "-shared", "-Wall", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


class ConvDesc(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("N", "C", "H", "W", "Cout", "kh", "kw", "stride_h", "stride_w", "pad_h", "pad_w")]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_get_threads.restype = C.c_int
    return _lib


def set_threads(t: int) -> None:
    lib().oracle_set_threads(C.c_int(int(t)))


def get_threads() -> int:
    return int(lib().oracle_get_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


@dataclass
class Binarized:
    e: np.ndarray        # rows x n uint8
    K: np.ndarray        # rows int32
    alpha: np.ndarray    # rows fp32
    beta: np.ndarray     # rows fp32
    flags: np.ndarray    # rows uint32
    s_star: np.ndarray   # rows int32
    best_D: np.ndarray   # rows fp64
    gap: np.ndarray      # rows fp64


def binarize(values: np.ndarray) -> Binarized:
    """Rows of a 2-D fp32 array -> two-level codes (Section 4.1, Algorithm 1)."""
    v = np.ascontiguousarray(values, dtype=np.float32)
    assert v.ndim == 2
    rows, n = v.shape
    out = Binarized(np.zeros((rows, n), np.uint8), np.zeros(rows, np.int32), np.zeros(rows, np.float32),
                    np.zeros(rows, np.float32), np.zeros(rows, np.uint32), np.zeros(rows, np.int32),
                    np.zeros(rows, np.float64), np.zeros(rows, np.float64))
    if rows and n:
        lib().oracle_binarize(_p(v), C.c_int64(rows), C.c_int32(n), C.c_int64(n), _p(out.e), _p(out.K), _p(out.alpha),
                              _p(out.beta), _p(out.flags), _p(out.s_star), _p(out.best_D), _p(out.gap))
    return out


def sign_code(values: np.ndarray) -> Binarized:
    """Rows -> sign masks with one scale (alpha = mean|w|, beta = -alpha): the XNOR-style code of FBin inputs."""
    v = np.ascontiguousarray(values, dtype=np.float32)
    rows, n = v.shape
    out = Binarized(np.zeros((rows, n), np.uint8), np.zeros(rows, np.int32), np.zeros(rows, np.float32),
                    np.zeros(rows, np.float32), np.zeros(rows, np.uint32), np.zeros(rows, np.int32),
                    np.zeros(rows, np.float64), np.full(rows, np.inf))
    if rows and n:
        lib().oracle_sign(_p(v), C.c_int64(rows), C.c_int32(n), C.c_int64(n), _p(out.e), _p(out.K), _p(out.alpha),
                          _p(out.beta), _p(out.flags))
    return out


def pack(bits: np.ndarray, ld_mask: int | None = None):
    """0/1 bytes (rows x n) -> (uint32 words rows x ld_mask, K per row)."""
    b = np.ascontiguousarray(bits, dtype=np.uint8)
    rows, n = b.shape
    wd = (n + 31) // 32
    if ld_mask is None:
        ld_mask = (wd + 3) // 4 * 4
    mask = np.zeros((rows, ld_mask), np.uint32)
    K = np.zeros(rows, np.int32)
    if rows:
        lib().oracle_pack(_p(b), C.c_int64(rows), C.c_int32(n), C.c_int64(n), _p(mask), C.c_int32(ld_mask), _p(K))
    return mask, K


def gemm(fA, gamma, delta, eB, alpha, beta):
    """Coded rows A (M x n masks, gamma/delta) times coded rows B (N x n masks, alpha/beta) -> (C fp32 MxN, p11 int32)."""
    fA = np.ascontiguousarray(fA, np.uint8)
    eB = np.ascontiguousarray(eB, np.uint8)
    M, n = fA.shape
    N = eB.shape[0]
    assert eB.shape[1] == n
    gamma, delta, alpha, beta = (np.ascontiguousarray(a, np.float32) for a in (gamma, delta, alpha, beta))
    Cm = np.zeros((M, N), np.float32)
    p11 = np.zeros((M, N), np.int32)
    if M and N:
        lib().oracle_gemm(C.c_int64(M), C.c_int64(N), C.c_int32(n), _p(fA), _p(gamma), _p(delta), _p(eB), _p(alpha),
                          _p(beta), _p(Cm), _p(p11))
    return Cm, p11


def conv_out_hw(H, W, kh, kw, stride, pad):
    return (H + 2 * pad[0] - kh) // stride[0] + 1, (W + 2 * pad[1] - kw) // stride[1] + 1


@dataclass
class ConvResult:
    y: np.ndarray
    p_e: np.ndarray | None
    p_K: np.ndarray | None
    p_gamma: np.ndarray | None
    p_delta: np.ndarray | None
    p_flags: np.ndarray | None
    p_p11: np.ndarray | None


def _desc(x_shape, Cout, kh, kw, stride, pad):
    N, Cc, H, W = x_shape
    return ConvDesc(N, Cc, H, W, Cout, kh, kw, stride[0], stride[1], pad[0], pad[1])


def conv(x, w_e, w_alpha, w_beta, kh, kw, stride=(1, 1), pad=(0, 0), details=True, sign_inputs=False) -> ConvResult:
    """Binary forward pass I (*) W~ (Section 4.3.2), every patch coded by Algorithm 1 (sign_inputs: by its sign
    pattern and mean magnitude instead, as in the paper's XNOR-structured FBin layers)."""
    x = np.ascontiguousarray(x, np.float32)
    w_e = np.ascontiguousarray(w_e, np.uint8)
    w_alpha = np.ascontiguousarray(w_alpha, np.float32)
    w_beta = np.ascontiguousarray(w_beta, np.float32)
    N, Cc, H, W = x.shape
    Cout, n = w_e.shape
    assert n == Cc * kh * kw
    Ho, Wo = conv_out_hw(H, W, kh, kw, stride, pad)
    d = _desc(x.shape, Cout, kh, kw, stride, pad)
    y = np.zeros((N, Cout, Ho, Wo), np.float32)
    P = N * Ho * Wo
    if details:
        p_e, p_K = np.zeros((P, n), np.uint8), np.zeros(P, np.int32)
        p_g, p_d = np.zeros(P, np.float32), np.zeros(P, np.float32)
        p_f, p_p = np.zeros(P, np.uint32), np.zeros((P, Cout), np.int32)
    else:
        p_e = p_K = p_g = p_d = p_f = p_p = None
    fn = lib().oracle_conv_sign if sign_inputs else lib().oracle_conv
    fn(C.byref(d), _p(x), _p(w_e), _p(w_alpha), _p(w_beta), _p(y), _p(p_e), _p(p_K), _p(p_g), _p(p_d),
                      _p(p_f), _p(p_p))
    return ConvResult(y, p_e, p_K, p_g, p_d, p_f, p_p)


def conv_wbin(x, w_e, w_alpha, w_beta, kh, kw, stride=(1, 1), pad=(0, 0)):
    """I (*) W~ with fp32 activations and two-level filters (Section 4.3.2, weights-only binarization).
    Returns (y fp32, abs_terms fp64), both N x Cout x Ho x Wo."""
    x = np.ascontiguousarray(x, np.float32)
    w_e = np.ascontiguousarray(w_e, np.uint8)
    w_alpha = np.ascontiguousarray(w_alpha, np.float32)
    w_beta = np.ascontiguousarray(w_beta, np.float32)
    N, Cc, H, W = x.shape
    Cout, n = w_e.shape
    assert n == Cc * kh * kw
    Ho, Wo = conv_out_hw(H, W, kh, kw, stride, pad)
    d = _desc(x.shape, Cout, kh, kw, stride, pad)
    y = np.zeros((N, Cout, Ho, Wo), np.float32)
    mag = np.zeros((N, Cout, Ho, Wo), np.float64)
    lib().oracle_conv_wbin(C.byref(d), _p(x), _p(w_e), _p(w_alpha), _p(w_beta), _p(y), _p(mag))
    return y, mag


def train_forward(W: np.ndarray):
    """Algorithm 2, steps 4-13: returns (Wc, Binarized of Wc, Wt dense)."""
    W = np.ascontiguousarray(W, np.float32)
    rows, n = W.shape
    Wc, Wt = np.zeros_like(W), np.zeros_like(W)
    e = np.zeros((rows, n), np.uint8)
    K, flags = np.zeros(rows, np.int32), np.zeros(rows, np.uint32)
    alpha, beta = np.zeros(rows, np.float32), np.zeros(rows, np.float32)
    lib().oracle_train_forward(_p(W), C.c_int64(rows), C.c_int32(n), _p(Wc), _p(e), _p(K), _p(alpha), _p(beta),
                               _p(flags), _p(Wt))
    return Wc, e, K, alpha, beta, flags, Wt


def theorem4(Wc: np.ndarray, e: np.ndarray, K: np.ndarray, grad_Wt: np.ndarray | None = None):
    """Theorem 4: returns (G fp64, grad_W fp32 or None)."""
    Wc = np.ascontiguousarray(Wc, np.float32)
    e = np.ascontiguousarray(e, np.uint8)
    K = np.ascontiguousarray(K, np.int32)
    rows, n = Wc.shape
    G = np.zeros((rows, n), np.float64)
    gw = None
    if grad_Wt is not None:
        grad_Wt = np.ascontiguousarray(grad_Wt, np.float32)
        gw = np.zeros((rows, n), np.float32)
    lib().oracle_theorem4(_p(Wc), _p(e), _p(K), C.c_int64(rows), C.c_int32(n), _p(G), _p(grad_Wt), _p(gw))
    return G, gw


def im2col(x, kh, kw, stride=(1, 1), pad=(0, 0)) -> np.ndarray:
    """Patch rows (N*Ho*Wo) x (C*kh*kw), element order (c, kh, kw), zero padding as 0.0 values."""
    x = np.ascontiguousarray(x, np.float32)
    N, Cc, H, W = x.shape
    Ho, Wo = conv_out_hw(H, W, kh, kw, stride, pad)
    d = _desc(x.shape, 1, kh, kw, stride, pad)
    out = np.zeros((N * Ho * Wo, Cc * kh * kw), np.float32)
    lib().oracle_im2col(C.byref(d), _p(x), _p(out))
    return out


# ------------------------------------------------------------------------------------------------------------
# Whole networks: the full-precision layers around the binarized ones, and the chain
# ------------------------------------------------------------------------------------------------------------
def conv_dense(x, w, kh, kw, stride=(1, 1), pad=(0, 0), bias=None) -> np.ndarray:
    """x (*) W (+ bias) with full-precision filters W [Cout x C*kh*kw]; fp64 sums in (c, kh, kw) order, fp32 out."""
    x = np.ascontiguousarray(x, np.float32)
    w = np.ascontiguousarray(w, np.float32)
    N, Cc, H, W = x.shape
    Cout, n = w.shape
    assert n == Cc * kh * kw
    Ho, Wo = conv_out_hw(H, W, kh, kw, stride, pad)
    d = _desc(x.shape, Cout, kh, kw, stride, pad)
    y = np.zeros((N, Cout, Ho, Wo), np.float32)
    b = None if bias is None else np.ascontiguousarray(bias, np.float32)
    lib().oracle_conv_dense(C.byref(d), _p(x), _p(w), _p(b), _p(y))
    return y


def affine(x, scale, shift) -> np.ndarray:
    x = np.ascontiguousarray(x, np.float32)
    N, Cc = x.shape[0], x.shape[1]
    hw = int(np.prod(x.shape[2:]))
    y = np.zeros_like(x)
    lib().oracle_affine(_p(x), C.c_int64(N), C.c_int32(Cc), C.c_int64(hw), _p(np.ascontiguousarray(scale, np.float32)),
                        _p(np.ascontiguousarray(shift, np.float32)), _p(y))
    return y


def relu(x) -> np.ndarray:
    x = np.ascontiguousarray(x, np.float32)
    y = np.zeros_like(x)
    lib().oracle_relu(_p(x), C.c_int64(x.size), _p(y))
    return y


def maxpool(x, kh, kw, stride=(1, 1), pad=(0, 0)) -> np.ndarray:
    x = np.ascontiguousarray(x, np.float32)
    N, Cc, H, W = x.shape
    Ho, Wo = conv_out_hw(H, W, kh, kw, stride, pad)
    d = _desc(x.shape, Cc, kh, kw, stride, pad)
    y = np.zeros((N, Cc, Ho, Wo), np.float32)
    lib().oracle_maxpool(C.byref(d), _p(x), _p(y))
    return y


def add(a, b) -> np.ndarray:
    a = np.ascontiguousarray(a, np.float32)
    b = np.ascontiguousarray(b, np.float32)
    assert a.shape == b.shape
    y = np.zeros_like(a)
    lib().oracle_add(_p(a), _p(b), C.c_int64(a.size), _p(y))
    return y


def network_layer(layer, x, saved):
    """One layer of a chain (a dict from dab_synth.networks): returns (output, saved).  `saved` is the tensor a
    shortcut holds; layers with on_saved = True transform it instead of the running tensor."""
    kind = layer["kind"]
    src = saved if layer.get("on_saved") else x
    if kind == "conv_dense":
        out = conv_dense(src, layer["w"], layer["kh"], layer["kw"], layer["stride"], layer["pad"], layer.get("bias"))
    elif kind == "conv_binary":
        wb = binarize(layer["w"])
        out = conv(src, wb.e, wb.alpha, wb.beta, layer["kh"], layer["kw"], layer["stride"], layer["pad"], details=False).y
    elif kind == "affine":
        out = affine(src, layer["scale"], layer["shift"])
    elif kind == "relu":
        out = relu(src)
    elif kind == "maxpool":
        out = maxpool(src, layer["kh"], layer["kw"], layer["stride"], layer["pad"])
    elif kind == "save":
        return x, x.copy()
    elif kind == "add":
        return add(x, saved), saved
    else:
        raise ValueError(kind)
    return (x, out) if layer.get("on_saved") else (out, saved)


def network_forward(layers, x, keep=False):
    """The whole chain on the CPU.  keep: also return the running tensor after every layer."""
    saved, outs = None, []
    for layer in layers:
        x, saved = network_layer(layer, x, saved)
        if keep:
            outs.append(x)
    return (x, outs) if keep else x
