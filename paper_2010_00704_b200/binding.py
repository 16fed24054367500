"""Thin ctypes binding of the C ABI in include/bcnn.h.

Argument marshalling only: every step of the path runs in the CUDA kernels.  Tensors
are torch CUDA tensors used purely as device buffers; the functions take their
``data_ptr()`` and the current torch stream.  There is no CPU fallback: if the shared
library is missing or does not load, importing the symbols raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libbcnn.so")

ENGINE_AUTO, ENGINE_LOP3, ENGINE_MMA_B1, ENGINE_TC_I8, ENGINE_MMA_S8, ENGINE_TC_WS, ENGINE_TC_PW, ENGINE_TC_C3, ENGINE_TC_PN = 0, 1, 2, 3, 4, 5, 6, 7, 8
ENGINES = {"auto": ENGINE_AUTO, "lop3": ENGINE_LOP3, "mma_b1": ENGINE_MMA_B1, "tc_i8": ENGINE_TC_I8,
           "mma_s8": ENGINE_MMA_S8, "tc_ws": ENGINE_TC_WS, "tc_pw": ENGINE_TC_PW, "tc_c3": ENGINE_TC_C3, "tc_pn": ENGINE_TC_PN}

EXPORTS = (
    "bcnn_pack", "bcnn_stem_fused", "bcnn_gemm_b1", "bcnn_gemm_b1_fused", "bcnn_conv2d_b1", "bcnn_conv2d_b1_fused", "bcnn_conv2d_b1_module",
    "bcnn_conv2d_b1_branches", "bcnn_dwconv3x3_module", "bcnn_avgpool", "bcnn_gap", "bcnn_fc",
    "bcnn_prepared_weights_bytes", "bcnn_prepare_weights", "bcnn_conv2d_b1_prepared", "bcnn_gemm_b1_prepared", "bcnn_prepared_preferred",
    "bcnn_conv2d_b1_fused_noalloc",
    "bcnn_conv2d_b1_engine", "bcnn_gemm_b1_engine", "bcnn_auto_engine", "bcnn_device_error", "bcnn_device_status",
    "bcnn_workspace_bytes", "bcnn_selftest_wait_timeout", "bcnn_status_string", "bcnn_version",
)

# bcnn_status values
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_CUDA, ERR_WORKSPACE, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5, -6
SELFTEST_TIMEOUT_CODE = 120

_lib = None


class BcnnError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} ({status})")


def load() -> ctypes.CDLL:
    """Load libbcnn.so (built in-tree by ``build.py``); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not built: run python -m paper_2010_00704_b200.build")
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
        lib.bcnn_pack.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp]
        lib.bcnn_stem_fused.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp]
        lib.bcnn_gemm_b1.argtypes = [vp, vp, vp, i64, i32, i32, vp]
        lib.bcnn_gemm_b1_fused.argtypes = [vp, vp, vp, vp, i64, i32, i32, vp]
        lib.bcnn_conv2d_b1.argtypes = [vp, vp, vp] + [i32] * 9 + [vp]
        lib.bcnn_conv2d_b1_fused.argtypes = [vp, vp, vp, vp] + [i32] * 9 + [vp]
        lib.bcnn_conv2d_b1_module.argtypes = [vp] * 9 + [i32] * 9 + [vp]
        lib.bcnn_conv2d_b1_branches.argtypes = [vp] * 10 + [i32] * 8 + [vp]
        lib.bcnn_dwconv3x3_module.argtypes = [vp] * 8 + [i32] * 6 + [vp]
        lib.bcnn_avgpool.argtypes = [vp, vp] + [i32] * 6 + [vp]
        lib.bcnn_gap.argtypes = [vp, vp] + [i32] * 4 + [vp]
        lib.bcnn_fc.argtypes = [vp] * 4 + [i32] * 3 + [vp]
        lib.bcnn_prepared_weights_bytes.argtypes = [i32, i32]
        lib.bcnn_prepared_weights_bytes.restype = ctypes.c_size_t
        lib.bcnn_prepare_weights.argtypes = [vp, vp, i32, i32, vp]
        lib.bcnn_conv2d_b1_prepared.argtypes = [vp, vp, vp, vp] + [i32] * 9 + [vp]
        lib.bcnn_gemm_b1_prepared.argtypes = [vp, vp, vp, vp, i64, i32, i32, vp]
        lib.bcnn_prepared_preferred.argtypes = [i32] * 10
        lib.bcnn_conv2d_b1_fused_noalloc.argtypes = [vp, vp, vp, vp] + [i32] * 9 + [vp]
        lib.bcnn_conv2d_b1_engine.argtypes = [i32, vp, vp, vp, vp] + [i32] * 9 + [vp]
        lib.bcnn_gemm_b1_engine.argtypes = [i32, vp, vp, vp, vp, i64, i32, i32, vp]
        lib.bcnn_auto_engine.argtypes = [i32] * 10
        lib.bcnn_device_error.argtypes = []
        lib.bcnn_device_status.argtypes = [ctypes.POINTER(ctypes.c_int)]
        lib.bcnn_workspace_bytes.argtypes = [i32] * 10
        lib.bcnn_workspace_bytes.restype = ctypes.c_size_t
        lib.bcnn_selftest_wait_timeout.argtypes = [i32, vp]
        lib.bcnn_status_string.argtypes = [i32]
        lib.bcnn_status_string.restype = ctypes.c_char_p
        for name in EXPORTS:
            if name not in ("bcnn_status_string", "bcnn_workspace_bytes", "bcnn_prepared_weights_bytes"):
                getattr(lib, name).restype = i32
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load().bcnn_status_string(int(status)).decode()


def version() -> int:
    return load().bcnn_version()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _p(t) -> int | None:
    return None if t is None else t.data_ptr()


def _check(status: int, what: str):
    if status != 0:
        raise BcnnError(status, what)


def out_hw(H, W, kh, kw, stride, pad):
    return (H + 2 * pad - kh) // stride + 1, (W + 2 * pad - kw) // stride + 1


def bcnn_pack(x: torch.Tensor, bias, out_bits: torch.Tensor, B, H, W, C_in, R=1):
    """x fp32 NHWC device tensor -> packed sign bits written into ``out_bits``."""
    _check(load().bcnn_pack(_p(x), _p(bias), _p(out_bits), B, H, W, C_in, R, _stream()), "bcnn_pack")
    return out_bits


def bcnn_stem_fused(x, bias, w_bits, thr, y_bits, B, H, W, C_in, R, C_out):
    """fp32 NHWC input -> (bias, sign, replication) -> binary 1x1 convolution -> threshold -> packed bits."""
    if thr is None:
        raise BcnnError(-1, "bcnn_stem_fused")
    _check(load().bcnn_stem_fused(_p(x), _p(bias), _p(w_bits), _p(thr), _p(y_bits), B, H, W, C_in, R, C_out,
                                  _stream()), "bcnn_stem_fused")
    return y_bits


def bcnn_gemm_b1(A_bits, W_bits, C, M, N, K, engine=ENGINE_AUTO):
    _check(load().bcnn_gemm_b1_engine(engine, _p(A_bits), _p(W_bits), None, _p(C), M, N, K, _stream()),
           "bcnn_gemm_b1")
    return C


def bcnn_gemm_b1_fused(A_bits, W_bits, thr, out_bits, M, N, K, engine=ENGINE_AUTO):
    if thr is None:
        raise BcnnError(-1, "bcnn_gemm_b1_fused")
    _check(load().bcnn_gemm_b1_engine(engine, _p(A_bits), _p(W_bits), _p(thr), _p(out_bits), M, N, K, _stream()),
           "bcnn_gemm_b1_fused")
    return out_bits


def bcnn_conv2d_b1(x_bits, w_bits, y, B, H, W, C_in, C_out, kh, kw, stride, pad, engine=ENGINE_AUTO):
    _check(load().bcnn_conv2d_b1_engine(engine, _p(x_bits), _p(w_bits), None, _p(y), B, H, W, C_in, C_out,
                                        kh, kw, stride, pad, _stream()), "bcnn_conv2d_b1")
    return y


def bcnn_conv2d_b1_fused(x_bits, w_bits, thr, y_bits, B, H, W, C_in, C_out, kh, kw, stride, pad,
                         engine=ENGINE_AUTO):
    if thr is None:
        raise BcnnError(-1, "bcnn_conv2d_b1_fused")
    _check(load().bcnn_conv2d_b1_engine(engine, _p(x_bits), _p(w_bits), _p(thr), _p(y_bits), B, H, W, C_in,
                                        C_out, kh, kw, stride, pad, _stream()), "bcnn_conv2d_b1_fused")
    return y_bits


def bcnn_conv2d_b1_module(x_bits, w_bits, bn_scale, bn_shift, identity, prelu_slope, next_bias, y_real, y_bits,
                          B, H, W, C_in, C_out, kh, kw, stride, pad):
    """Binary conv -> batch norm -> + identity (fp16) -> PReLU -> fp16 map and the next module's packed signs."""
    _check(load().bcnn_conv2d_b1_module(_p(x_bits), _p(w_bits), _p(bn_scale), _p(bn_shift), _p(identity),
                                        _p(prelu_slope), _p(next_bias), _p(y_real), _p(y_bits), B, H, W, C_in, C_out,
                                        kh, kw, stride, pad, _stream()), "bcnn_conv2d_b1_module")
    return y_real, y_bits


def bcnn_conv2d_b1_branches(x_bits, w_bits, bn_scale, bn_shift, pad_dot, identity, prelu_slope, next_bias, y_real, y_bits,
                            B, H, W, C_in, C_out, P, kh=1, kw=1):
    """Module with P parallel binary branches (kh*kw > 1: the P = kh*kw shifted taps of a binary kh x kw convolution)."""
    _check(load().bcnn_conv2d_b1_branches(_p(x_bits), _p(w_bits), _p(bn_scale), _p(bn_shift), _p(pad_dot), _p(identity),
                                          _p(prelu_slope), _p(next_bias), _p(y_real), _p(y_bits), B, H, W, C_in, C_out, P,
                                          kh, kw, _stream()), "bcnn_conv2d_b1_branches")
    return y_real, y_bits


def bcnn_dwconv3x3_module(x, w, bn_scale, bn_shift, prelu_slope, next_bias, y_real, y_bits, B, H, W, C_in, R=1, S=1):
    """Real depth-wise 3x3 convolution (stride S, replication R) -> batch norm -> PReLU -> fp16 map (+ next signs)."""
    _check(load().bcnn_dwconv3x3_module(_p(x), _p(w), _p(bn_scale), _p(bn_shift), _p(prelu_slope), _p(next_bias), _p(y_real),
                                        _p(y_bits), B, H, W, C_in, R, S, _stream()), "bcnn_dwconv3x3_module")
    return y_real, y_bits


def bcnn_avgpool(x, y, B, H, W, C_in, R=1, S=1):
    _check(load().bcnn_avgpool(_p(x), _p(y), B, H, W, C_in, R, S, _stream()), "bcnn_avgpool")
    return y


def bcnn_gap(x, pooled, B, H, W, C):
    _check(load().bcnn_gap(_p(x), _p(pooled), B, H, W, C, _stream()), "bcnn_gap")
    return pooled


def bcnn_fc(pooled, w, bias, logits, B, C, N):
    _check(load().bcnn_fc(_p(pooled), _p(w), _p(bias), _p(logits), B, C, N, _stream()), "bcnn_fc")
    return logits


def bcnn_prepared_weights_bytes(C_out, K) -> int:
    return int(load().bcnn_prepared_weights_bytes(C_out, K))


def bcnn_prepare_weights(w_bits, prepared, C_out, K):
    """Expand a layer's packed weights once into the caller's buffer ``prepared`` (256-byte aligned)."""
    _check(load().bcnn_prepare_weights(_p(w_bits), _p(prepared), C_out, K, _stream()), "bcnn_prepare_weights")
    return prepared


def bcnn_conv2d_b1_prepared(x_bits, prepared, thr, out, B, H, W, C_in, C_out, kh, kw, stride, pad):
    _check(load().bcnn_conv2d_b1_prepared(_p(x_bits), _p(prepared), _p(thr), _p(out), B, H, W, C_in, C_out, kh, kw, stride, pad,
                                          _stream()), "bcnn_conv2d_b1_prepared")
    return out


def bcnn_gemm_b1_prepared(A_bits, prepared, thr, out, M, N, K):
    _check(load().bcnn_gemm_b1_prepared(_p(A_bits), _p(prepared), _p(thr), _p(out), M, N, K, _stream()), "bcnn_gemm_b1_prepared")
    return out


STATIC_SCRATCH_BYTES = 4 << 20


def bcnn_conv2d_b1_fused_noalloc(x_bits, w_bits, thr, y_bits, B, H, W, C_in, C_out, kh, kw, stride, pad):
    """``bcnn_conv2d_b1_fused`` for callers that cannot allocate: the prepared weights live in a static array of the
    library (4 MiB per GPU); layers whose prepared form is larger raise BCNN_ERR_WORKSPACE."""
    if thr is None:
        raise BcnnError(-1, "bcnn_conv2d_b1_fused_noalloc")
    _check(load().bcnn_conv2d_b1_fused_noalloc(_p(x_bits), _p(w_bits), _p(thr), _p(y_bits), B, H, W, C_in, C_out, kh, kw,
                                               stride, pad, _stream()), "bcnn_conv2d_b1_fused_noalloc")
    return y_bits


def bcnn_prepared_preferred(B, H, W, C_in, C_out, kh, kw, stride, pad, fused=True) -> bool:
    return bool(load().bcnn_prepared_preferred(B, H, W, C_in, C_out, kh, kw, stride, pad, 1 if fused else 0))


def bcnn_auto_engine(B, H, W, C_in, C_out, kh, kw, stride, pad, fused=True) -> str:
    """Name of the engine BCNN_ENGINE_AUTO picks for this shape."""
    e = load().bcnn_auto_engine(B, H, W, C_in, C_out, kh, kw, stride, pad, 1 if fused else 0)
    if e < 0:
        raise BcnnError(e, "bcnn_auto_engine")
    return {v: k for k, v in ENGINES.items()}[e]


def bcnn_device_error() -> int:
    return load().bcnn_device_error()


def bcnn_device_status():
    """(status, code): BCNN_OK / BCNN_ERR_TIMEOUT / BCNN_ERR_CUDA and the raw device error code."""
    code = ctypes.c_int(0)
    st = load().bcnn_device_status(ctypes.byref(code))
    return st, code.value


def bcnn_workspace_bytes(B, H, W, C_in, C_out, kh, kw, stride, pad, fused=True) -> int:
    return int(load().bcnn_workspace_bytes(B, H, W, C_in, C_out, kh, kw, stride, pad, 1 if fused else 0))


def bcnn_selftest_wait_timeout(polls: int = 256):
    """Enqueue the self-test kernel whose bounded wait runs out (see include/bcnn.h)."""
    _check(load().bcnn_selftest_wait_timeout(int(polls), _stream()), "bcnn_selftest_wait_timeout")
