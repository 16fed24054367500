"""CPU oracle for the binary convolution hot path (TEST INFRASTRUCTURE ONLY).

Nothing in the product package imports this.  Only the tests, the smoke check and
the CPU-baseline leg of the benchmark may use it.  The arithmetic lives in plain C
(``bcnn_oracle.c``: the definition, on unpacked int8 +-1 tensors; ``bcnn_checker.c``:
a separately written bit-packed checker for full-size coverage, trusted only
through the tests that prove it equal to the definition).  This module compiles
those two files with gcc and marshals numpy arrays; it holds no arithmetic of the
method itself.

Parity pins (see tests/test_oracle_pins.py): closed forms for constant inputs
including the border values that depend on the -1 padding, a one-hot weight case
worked by hand, brute force in pure Python on tiny shapes, the textbook library
convolution of the padded +-1 tensors, the xor/popcount identity against a float
dot product, and the tie rule of the threshold; for the convolution module (batch
norm, identity, PReLU, fp16 store, next sign) a case worked by hand, the fp16
round-to-even ties, the sign-of-the-stored-value rule, the reduction to the integer
threshold and the elementwise numpy restatement.  The paper prints no worked
numeric example of a convolution, so beyond those pins parity is unpinned by the
paper itself.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libbcnn_oracle.so")
_SOURCES = [os.path.join(_HERE, "bcnn_oracle.c"), os.path.join(_HERE, "bcnn_checker.c")]
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle and the checker into one shared object beside the sources."""
    newest = max(os.path.getmtime(s) for s in _SOURCES)
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < newest:
        tmp = _LIB_PATH + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-mpopcnt",
               "-shared", "-fPIC", "-o", tmp] + _SOURCES
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    with _lock:
        if _lib is None:
            _lib = ctypes.CDLL(build())
            _lib.oracle_threads.restype = ctypes.c_int
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def threads() -> int:
    """Number of OpenMP threads the oracle uses."""
    return int(_load().oracle_threads())


def out_hw(H: int, W: int, kh: int, kw: int, stride: int, pad: int):
    """Output extent, floor((H + 2*pad - kh)/stride) + 1."""
    return (H + 2 * pad - kh) // stride + 1, (W + 2 * pad - kw) // stride + 1


def _check_pm1(a: np.ndarray, name: str):
    if a.size and not np.all(np.abs(a) == 1):
        raise ValueError(f"{name} must hold only -1 and +1")


def binarize(x: np.ndarray, bias, R: int = 1) -> np.ndarray:
    """sign(x[..., c mod C_in] + bias[c]) as int8 +-1; x real NHWC fp32 (Section 4.2.1)."""
    x = _c(x, np.float32)
    B, H, W, C_in = x.shape
    C = C_in * R
    out = np.empty((B, H, W, C), dtype=np.int8)
    bptr = None
    if bias is not None:
        bias = _c(bias, np.float32)
        assert bias.shape == (C,)
        bptr = _ptr(bias)
    _load().oracle_binarize(_ptr(x), bptr, _ptr(out), B, H, W, C_in, R)
    return out


def sign_weights(w: np.ndarray) -> np.ndarray:
    """Binary weights = sign of the real weights (Section 5.2)."""
    w = _c(w, np.float32)
    out = np.empty(w.shape, dtype=np.int8)
    _load().oracle_sign_weights(_ptr(w), _ptr(out), ctypes.c_long(w.size))
    return out


def conv2d(x: np.ndarray, w: np.ndarray, stride: int = 1, pad: int = 0) -> np.ndarray:
    """Direct +-1 convolution: x int8 [B,H,W,Cin], w int8 [Cout,kh,kw,Cin] -> int32 [B,OH,OW,Cout]."""
    x = _c(x, np.int8)
    w = _c(w, np.int8)
    _check_pm1(x, "x")
    _check_pm1(w, "w")
    B, H, W, C_in = x.shape
    C_out, kh, kw, C_in2 = w.shape
    assert C_in == C_in2
    OH, OW = out_hw(H, W, kh, kw, stride, pad)
    y = np.empty((B, OH, OW, C_out), dtype=np.int32)
    _load().oracle_conv2d(_ptr(x), _ptr(w), _ptr(y), B, H, W, C_in, C_out, kh, kw, stride, pad)
    return y


def conv2d_pixels(x: np.ndarray, w: np.ndarray, pix, stride: int = 1, pad: int = 0) -> np.ndarray:
    """The convolution at the listed flat output-pixel indices only -> int32 [len(pix), Cout]."""
    x = _c(x, np.int8)
    w = _c(w, np.int8)
    _check_pm1(x, "x")
    _check_pm1(w, "w")
    pix = _c(pix, np.int64)
    B, H, W, C_in = x.shape
    C_out, kh, kw, C_in2 = w.shape
    assert C_in == C_in2
    OH, OW = out_hw(H, W, kh, kw, stride, pad)
    assert pix.size == 0 or (pix.min() >= 0 and pix.max() < B * OH * OW)
    y = np.empty((pix.size, C_out), dtype=np.int32)
    _load().oracle_conv2d_pixels(_ptr(x), _ptr(w), _ptr(pix), ctypes.c_long(pix.size), _ptr(y),
                                 B, H, W, C_in, C_out, kh, kw, stride, pad)
    return y


def gemm(A: np.ndarray, Wt: np.ndarray) -> np.ndarray:
    """C[m,n] = sum_k A[m,k] * Wt[n,k] on int8 +-1 matrices -> int32 [M,N]."""
    A = _c(A, np.int8)
    Wt = _c(Wt, np.int8)
    _check_pm1(A, "A")
    _check_pm1(Wt, "Wt")
    M, K = A.shape
    N, K2 = Wt.shape
    assert K == K2
    C = np.empty((M, N), dtype=np.int32)
    _load().oracle_gemm(_ptr(A), _ptr(Wt), _ptr(C), ctypes.c_long(M), ctypes.c_long(N), ctypes.c_long(K))
    return C


def threshold(acc: np.ndarray, thr: np.ndarray) -> np.ndarray:
    """(acc >= thr[channel]) ? +1 : -1 over the last axis, int8."""
    acc = _c(acc, np.int32)
    thr = _c(thr, np.int32)
    N = acc.shape[-1]
    assert thr.shape == (N,)
    out = np.empty(acc.shape, dtype=np.int8)
    rows = acc.size // N if N else 0
    _load().oracle_threshold(_ptr(acc), _ptr(thr), _ptr(out), ctypes.c_long(rows), ctypes.c_long(N))
    return out


def conv_module(acc: np.ndarray, scale, shift, identity, slope, next_bias=None, want_sign: bool = True):
    """Batch norm (scale, shift) -> + identity (fp16) -> PReLU -> fp16 real map, and the next module's
    sign(stored value + next_bias) as int8 +-1 (Section 4.2.1).  acc int32 [..., N]; per-channel fp32
    vectors of length N; identity float16 [..., N] or None.  Returns (y float16, s int8 or None)."""
    acc = _c(acc, np.int32)
    N = acc.shape[-1]
    scale, shift, slope = _c(scale, np.float32), _c(shift, np.float32), _c(slope, np.float32)
    assert scale.shape == (N,) and shift.shape == (N,) and slope.shape == (N,)
    iptr = None
    if identity is not None:
        identity = _c(identity, np.float16)
        assert identity.shape == acc.shape
        iptr = _ptr(identity)
    nptr = None
    if next_bias is not None:
        next_bias = _c(next_bias, np.float32)
        assert next_bias.shape == (N,)
        nptr = _ptr(next_bias)
    y = np.empty(acc.shape, dtype=np.float16)
    s = np.empty(acc.shape, dtype=np.int8) if want_sign else None
    rows = acc.size // N if N else 0
    _load().oracle_conv_module(_ptr(acc), _ptr(scale), _ptr(shift), iptr, _ptr(slope), nptr, _ptr(y),
                               None if s is None else _ptr(s), ctypes.c_long(rows), ctypes.c_long(N))
    return y, s


# ---- bit-packed checker (not the oracle; proven equal to it by the CPU tests) ----

def checker_conv2d(x_bits: np.ndarray, w_bits: np.ndarray, dims, stride: int, pad: int) -> np.ndarray:
    """x_bits uint8 [B,H,W,Cin/8], w_bits uint8 [Cout,kh,kw,Cin/8]; dims = (B,H,W,Cin,Cout,kh,kw)."""
    B, H, W, C_in, C_out, kh, kw = dims
    x_bits = np.ascontiguousarray(x_bits).view(np.uint8)
    w_bits = np.ascontiguousarray(w_bits).view(np.uint8)
    assert x_bits.size == B * H * W * C_in // 8 and w_bits.size == C_out * kh * kw * C_in // 8
    OH, OW = out_hw(H, W, kh, kw, stride, pad)
    y = np.empty((B, OH, OW, C_out), dtype=np.int32)
    _load().checker_conv2d(_ptr(x_bits), _ptr(w_bits), _ptr(y), B, H, W, C_in, C_out, kh, kw, stride, pad)
    return y


def checker_gemm(A_bits: np.ndarray, W_bits: np.ndarray, M: int, N: int, K: int,
                 rows=None) -> np.ndarray:
    """Packed product; rows=(m0, m1) restricts it to that row range."""
    A_bits = np.ascontiguousarray(A_bits).view(np.uint8)
    W_bits = np.ascontiguousarray(W_bits).view(np.uint8)
    assert A_bits.size == M * K // 8 and W_bits.size == N * K // 8
    if rows is None:
        C = np.empty((M, N), dtype=np.int32)
        _load().checker_gemm(_ptr(A_bits), _ptr(W_bits), _ptr(C),
                             ctypes.c_long(M), ctypes.c_long(N), ctypes.c_long(K))
    else:
        m0, m1 = rows
        C = np.empty((m1 - m0, N), dtype=np.int32)
        _load().checker_gemm_rows(_ptr(A_bits), _ptr(W_bits), _ptr(C), ctypes.c_long(m0),
                                  ctypes.c_long(m1), ctypes.c_long(N), ctypes.c_long(K))
    return C
