"""The C-ABI library loads and exports every symbol include/bcnn.h declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "bcnn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bcnn_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported():
    from paper_2010_00704_b200 import build, binding
    lib = ctypes.CDLL(build.build())
    names = _declared()
    assert "bcnn_pack" in names and "bcnn_conv2d_b1_fused" in names and "bcnn_gemm_b1" in names
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.EXPORTS) <= set(names)


def test_status_strings_and_version():
    from paper_2010_00704_b200 import build, binding
    build.build()
    assert binding.version() >= 100
    assert binding.status_string(0) == "ok"
    assert "align" in binding.status_string(-3)
    assert "workspace" in binding.status_string(binding.ERR_WORKSPACE)
    assert "wait" in binding.status_string(binding.ERR_TIMEOUT)
    # the device error codes name the engine and the role whose wait gave up
    for code in (101, 102, 103, 111, 112, 113, 121, 122, 123, 124, 125, 126, 131, 132, 133, 134, 141, 142, 143, 144, 145, 146, 151, 152, 153, 154, 155, 156,
                 binding.SELFTEST_TIMEOUT_CODE):
        assert "timed out" in binding.status_string(code)
    assert binding.status_string(77) == "device-side error code"


def test_workspace_bytes_is_zero_for_every_shape():
    # no kernel uses scratch memory: the query exists so that callers can size one buffer per model anyway
    from paper_2010_00704_b200 import build, binding, workloads as wl
    build.build()
    for l in wl.BACKBONE18 + wl.BLOCK_STACK + wl.STEM_DOWN:
        for fused in (False, True):
            assert binding.bcnn_workspace_bytes(256, l.H, l.W, l.C_in, l.C_out, l.k, l.k, l.stride, l.pad, fused) == 0
    assert binding.bcnn_workspace_bytes(1, 16384, 1, 9216, 16384, 1, 1, 1, 0) == 0      # a GEMM of the sweep
    assert binding.bcnn_workspace_bytes(1, 4, 4, 48, 32, 1, 1, 1, 0) == 0                # invalid shape: still 0


def test_argument_validation_needs_no_device():
    # validation runs before any CUDA call, so bad arguments are reported on a CPU-only box too
    from paper_2010_00704_b200 import build, binding
    build.build()
    lib = binding.load()
    a = ctypes.c_void_p(4096)
    assert lib.bcnn_gemm_b1(None, a, a, 8, 8, 32, None) == -1
    assert lib.bcnn_gemm_b1(a, a, a, 8, 8, 48, None) == -2          # K not a multiple of 32
    assert lib.bcnn_gemm_b1(a, a, a, 0, 8, 32, None) == -1
    assert lib.bcnn_gemm_b1(ctypes.c_void_p(4100), a, a, 8, 8, 32, None) == -3
    assert lib.bcnn_gemm_b1_fused(a, a, None, a, 8, 32, 32, None) == -1
    assert lib.bcnn_gemm_b1_fused(a, a, a, a, 8, 40, 32, None) == -2  # N not a multiple of 32
    assert lib.bcnn_conv2d_b1(a, a, a, 1, 4, 4, 48, 8, 3, 3, 1, 1, None) == -2
    assert lib.bcnn_conv2d_b1(a, a, a, 1, 2, 2, 32, 8, 5, 5, 1, 0, None) == -1   # kernel larger than image
    assert lib.bcnn_conv2d_b1(a, a, a, 1, 4, 4, 32, 8, 3, 3, 0, 1, None) == -1
    assert lib.bcnn_pack(a, None, a, 1, 2, 2, 12, 2, None) == -2
    assert lib.bcnn_pack(None, None, a, 1, 2, 2, 32, 1, None) == -1
    assert lib.bcnn_conv2d_b1_engine(99, a, a, None, a, 1, 4, 4, 32, 8, 3, 3, 1, 1, None) == -2
    assert lib.bcnn_selftest_wait_timeout(0, None) == -1
    assert lib.bcnn_selftest_wait_timeout(1 << 20, None) == -1
