"""CPU oracle for the binary convolution hot path (TEST INFRASTRUCTURE ONLY).

Nothing in the product package imports this.  Only the tests, the smoke check and
the CPU-baseline leg of the benchmark may use it.  The arithmetic lives in plain C
(``bcnn_oracle.c``: the definition, on unpacked int8 +-1 tensors; ``bcnn_block_oracle.c``:
the rest of the paper's building block - parallel binary branches, depth-wise 3x3 module,
average pooling, global pooling and the fully connected layer; ``bcnn_checker.c``:
a separately written bit-packed checker for full-size coverage, trusted only
through the tests that prove it equal to the definition).  This module compiles
those files with gcc and marshals numpy arrays; it holds no arithmetic of the
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
paper itself.  The block pieces are pinned in tests/test_block_oracle_pins.py: the branch
module against the single-branch function, a hand-worked two-branch case and the order
of summation; the shifted-branch form of an F x F convolution against the textbook zero-
padded convolution and against the -1-padded one; depth-wise convolution, pooling and the
fully connected layer against closed forms and the float64 library routines.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libbcnn_oracle.so")
_SOURCES = [os.path.join(_HERE, "bcnn_oracle.c"), os.path.join(_HERE, "bcnn_block_oracle.c"),
            os.path.join(_HERE, "bcnn_checker.c")]
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


def conv_module_branches(accs, scales, shifts, identity, slope, next_bias=None, want_sign: bool = True):
    """Module with P parallel binary branches (Section 4.2.1, Figure 4 bottom): accs int32 [P, ..., N], scales and
    shifts fp32 [P, N]; the rest as ``conv_module``.  Returns (y float16, s int8 or None)."""
    accs = _c(accs, np.int32)
    P, N = accs.shape[0], accs.shape[-1]
    scales, shifts, slope = _c(scales, np.float32), _c(shifts, np.float32), _c(slope, np.float32)
    assert scales.shape == (P, N) and shifts.shape == (P, N) and slope.shape == (N,)
    iptr = None
    if identity is not None:
        identity = _c(identity, np.float16)
        assert identity.shape == accs.shape[1:]
        iptr = _ptr(identity)
    nptr = None
    if next_bias is not None:
        next_bias = _c(next_bias, np.float32)
        assert next_bias.shape == (N,)
        nptr = _ptr(next_bias)
    y = np.empty(accs.shape[1:], dtype=np.float16)
    s = np.empty(accs.shape[1:], dtype=np.int8) if want_sign else None
    rows = y.size // N if N else 0
    _load().oracle_conv_module_branches(_ptr(accs), _ptr(scales), _ptr(shifts), iptr, _ptr(slope), nptr, _ptr(y),
                                        None if s is None else _ptr(s), ctypes.c_long(rows), ctypes.c_long(N), P)
    return y, s


def shifted_branch_accs(x_real, biases, ws, kh: int, kw: int, pad_zero_contribution: bool = False):
    """The P = kh*kw branch convolutions that stand for a binary kh x kw convolution (Section 4.2.1, last paragraph):
    branch p = (r, t) sees the real map shifted by (r - (kh-1)/2, t - (kw-1)/2) with ZERO padding, adds its own bias,
    takes the sign and runs its own binary 1x1 convolution.  Steps, in the paper's order, from existing pieces:
    shift + zero pad (array slicing), ``binarize``, ``conv2d`` (1x1).
      x_real float16 [B,H,W,C_in]; biases fp32 [P,C_in]; ws int8 [P,C_out,C_in] (+-1).
    Returns (accs int32 [P,B,H,W,C_out], inside bool [P,H,W]).  With ``pad_zero_contribution`` a branch whose pixel
    lies outside the image contributes 0 instead of the convolution of sign(0 + bias) (the other reading)."""
    x_real = _c(x_real, np.float16)
    B, H, W, C_in = x_real.shape
    P = kh * kw
    biases = _c(biases, np.float32)
    ws = _c(ws, np.int8)
    assert biases.shape == (P, C_in) and ws.shape[0] == P and ws.shape[2] == C_in
    accs, insides = [], []
    for p in range(P):
        r, t = divmod(p, kw)
        dy, dx = r - (kh - 1) // 2, t - (kw - 1) // 2
        shifted = np.zeros_like(x_real)
        inside = np.zeros((H, W), dtype=bool)
        h0, h1 = max(0, -dy), min(H, H - dy)
        w0, w1 = max(0, -dx), min(W, W - dx)
        if h1 > h0 and w1 > w0:
            shifted[:, h0:h1, w0:w1, :] = x_real[:, h0 + dy:h1 + dy, w0 + dx:w1 + dx, :]
            inside[h0:h1, w0:w1] = True
        bits = binarize(shifted.astype(np.float32), biases[p], 1)
        acc = conv2d(bits, ws[p][:, None, None, :], 1, 0)
        if pad_zero_contribution:
            acc = acc * inside[None, :, :, None].astype(np.int32)
        accs.append(acc)
        insides.append(inside)
    return np.stack(accs), np.stack(insides)


def dwconv3x3_module(x, w, scale, shift, slope, R: int = 1, S: int = 1) -> np.ndarray:
    """Real depth-wise 3x3 convolution (stride S, zero padding 1), batch norm, PReLU (Section 4.2.1), with channel
    replication R (Section 4.2.2).  x float16 [B,H,W,C_in]; w fp32 [C,3,3]; per-channel fp32 [C]; C = R*C_in.
    fp64 arithmetic, one rounding to float16."""
    x = _c(x, np.float16)
    B, H, W, C_in = x.shape
    C = C_in * R
    w, scale, shift, slope = _c(w, np.float32), _c(scale, np.float32), _c(shift, np.float32), _c(slope, np.float32)
    assert w.shape == (C, 3, 3) and scale.shape == (C,) and shift.shape == (C,) and slope.shape == (C,)
    OH, OW = (H + 2 - 3) // S + 1, (W + 2 - 3) // S + 1
    y = np.empty((B, OH, OW, C), dtype=np.float16)
    _load().oracle_dwconv3x3_module(_ptr(x), _ptr(w), _ptr(scale), _ptr(shift), _ptr(slope), _ptr(y), B, H, W, C_in, R, S)
    return y


def avgpool(x, S: int, R: int = 1) -> np.ndarray:
    """S x S / S average pooling (Section 4.2.3) with channel replication R; float16 in and out, fp64 mean."""
    x = _c(x, np.float16)
    B, H, W, C_in = x.shape
    assert H % S == 0 and W % S == 0
    y = np.empty((B, H // S, W // S, C_in * R), dtype=np.float16)
    _load().oracle_avgpool(_ptr(x), _ptr(y), B, H, W, C_in, R, S)
    return y


def gap(x) -> np.ndarray:
    """Global average pooling (Section 4.1): float16 [B,H,W,C] -> float64 [B,C]."""
    x = _c(x, np.float16)
    B, H, W, C = x.shape
    out = np.empty((B, C), dtype=np.float64)
    _load().oracle_gap(_ptr(x), _ptr(out), B, ctypes.c_long(H * W), C)
    return out


def fc(pooled, w, bias=None) -> np.ndarray:
    """Fully connected layer (Section 4.1): pooled float64 [B,C], w fp32 [N,C], bias fp32 [N] -> float64 [B,N]."""
    pooled = _c(pooled, np.float64)
    w = _c(w, np.float32)
    B, C = pooled.shape
    N = w.shape[0]
    assert w.shape == (N, C)
    bptr = None
    if bias is not None:
        bias = _c(bias, np.float32)
        assert bias.shape == (N,)
        bptr = _ptr(bias)
    out = np.empty((B, N), dtype=np.float64)
    _load().oracle_fc(_ptr(pooled), _ptr(w), bptr, _ptr(out), B, C, N)
    return out


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
