"""Pins for the CPU oracle: it is checked against things other than itself.

Closed forms, a hand-worked one-hot case, pure-Python brute force, the textbook
library convolution, the xor/popcount identity, numpy's integer matmul, special
floating-point values for the sign, and the threshold tie rule.  Shapes are
deliberately lopsided (H != W, kh != kw, C_in != C_out, stride 2, pad 0/1/2) so that a
swapped index, a transposed operand, a dropped tap or a wrong padding value fails.
"""
import itertools

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from paper_2010_00704_b200 import synth


def _rng(i):
    return np.random.default_rng(7000 + i)


# ---------------------------------------------------------------- closed forms

@pytest.mark.parametrize("stride,pad,kh,kw", [(1, 1, 3, 3), (2, 1, 3, 3), (1, 0, 1, 1), (2, 2, 3, 5), (1, 2, 5, 3)])
def test_constant_inputs_give_plus_minus_K_everywhere(oracle, stride, pad, kh, kw):
    B, H, W, Ci, Co = 2, 7, 9, 32, 5
    K = kh * kw * Ci
    xm = -np.ones((B, H, W, Ci), np.int8)
    wp = np.ones((Co, kh, kw, Ci), np.int8)
    # padding is -1 as well, so borders are no exception
    assert np.all(oracle.conv2d(xm, wp, stride, pad) == -K)
    assert np.all(oracle.conv2d(xm, -wp, stride, pad) == K)


def test_all_plus_one_shows_the_minus_one_padding(oracle):
    B, H, W, Ci, Co = 1, 6, 8, 32, 3
    K = 9 * Ci
    y = oracle.conv2d(np.ones((B, H, W, Ci), np.int8), np.ones((Co, 3, 3, Ci), np.int8), 1, 1)
    expect = np.full((H, W), K, np.int32)
    expect[0, :] = expect[-1, :] = K - 6 * Ci      # 3 of 9 taps padded: (6 - 3) * Ci
    expect[:, 0] = expect[:, -1] = K - 6 * Ci
    for i, j in itertools.product((0, -1), (0, -1)):
        expect[i, j] = K - 10 * Ci                 # 5 of 9 taps padded: (4 - 5) * Ci
    for co in range(Co):
        assert np.array_equal(y[0, :, :, co], expect)


def test_stride2_even_size_touches_only_top_left_padding(oracle):
    # H even, k 3, stride 2, pad 1: the last window starts at H-3 and ends at H-1, inside.
    H = W = 8
    Ci = 32
    y = oracle.conv2d(np.ones((1, H, W, Ci), np.int8), np.ones((1, 3, 3, Ci), np.int8), 2, 1)[0, :, :, 0]
    K = 9 * Ci
    assert y.shape == (4, 4)
    expect = np.full((4, 4), K)
    expect[0, :] = K - 6 * Ci
    expect[:, 0] = K - 6 * Ci
    expect[0, 0] = K - 10 * Ci
    assert np.array_equal(y, expect)


def test_one_hot_weight_hand_worked(oracle):
    # all weights -1 except one +1 at (co=1, r=0, t=2, ci=5):
    # y = -(sum of the padded window) + 2 * x_padded[tap (0,2), channel 5]
    rng = _rng(1)
    B, H, W, Ci, Co, kh, kw, s, p = 2, 5, 7, 32, 3, 3, 3, 1, 1
    x = synth.pm1(rng, (B, H, W, Ci))
    w = -np.ones((Co, kh, kw, Ci), np.int8)
    w[1, 0, 2, 5] = 1
    y = oracle.conv2d(x, w, s, p)
    xp = np.pad(x.astype(np.int64), ((0, 0), (p, p), (p, p), (0, 0)), constant_values=-1)
    for b, oh, ow in itertools.product(range(B), range(H), range(W)):
        win = xp[b, oh:oh + kh, ow:ow + kw, :]
        assert y[b, oh, ow, 0] == -win.sum()
        assert y[b, oh, ow, 2] == -win.sum()
        assert y[b, oh, ow, 1] == -win.sum() + 2 * win[0, 2, 5]


# ---------------------------------------------------------------- brute force, library routine

def _brute_conv(x, w, stride, pad):
    B, H, W, Ci = x.shape
    Co, kh, kw, _ = w.shape
    OH = (H + 2 * pad - kh) // stride + 1
    OW = (W + 2 * pad - kw) // stride + 1
    y = np.zeros((B, OH, OW, Co), np.int64)
    for b, oh, ow, co in itertools.product(range(B), range(OH), range(OW), range(Co)):
        acc = 0
        for r, t, ci in itertools.product(range(kh), range(kw), range(Ci)):
            ih, iw = oh * stride - pad + r, ow * stride - pad + t
            v = int(x[b, ih, iw, ci]) if (0 <= ih < H and 0 <= iw < W) else -1
            acc += v * int(w[co, r, t, ci])
        y[b, oh, ow, co] = acc
    return y


@pytest.mark.parametrize("case", range(12))
def test_brute_force_tiny(oracle, case):
    rng = _rng(100 + case)
    B = int(rng.integers(1, 3))
    H, W = int(rng.integers(1, 5)), int(rng.integers(1, 5))
    Ci = 8 * int(rng.integers(1, 5))
    Co = int(rng.integers(1, 4))
    kh, kw = int(rng.integers(1, 4)), int(rng.integers(1, 4))
    stride = int(rng.integers(1, 3))
    pad = int(rng.integers(0, 3))
    if H + 2 * pad < kh or W + 2 * pad < kw:
        pad = 2
    x = synth.pm1(rng, (B, H, W, Ci))
    w = synth.pm1(rng, (Co, kh, kw, Ci))
    assert np.array_equal(oracle.conv2d(x, w, stride, pad), _brute_conv(x, w, stride, pad))


def _torch_conv(x, w, stride, pad):
    xt = torch.from_numpy(x.astype(np.float32)).permute(0, 3, 1, 2)
    wt = torch.from_numpy(w.astype(np.float32)).permute(0, 3, 1, 2)
    xt = F.pad(xt, (pad, pad, pad, pad), value=-1.0)
    y = F.conv2d(xt, wt, stride=stride)
    return y.permute(0, 2, 3, 1).numpy().astype(np.int64)


@pytest.mark.parametrize("shape", [
    (2, 9, 13, 32, 40, 3, 3, 1, 1),
    (1, 12, 10, 64, 24, 3, 3, 2, 1),
    (3, 5, 6, 96, 16, 1, 1, 1, 0),
    (1, 8, 8, 32, 8, 3, 1, 2, 0),
    (2, 7, 11, 32, 8, 1, 3, 1, 2),
    (1, 32, 32, 128, 128, 3, 3, 1, 1),          # the single 3x3 workload, K = 1152
])
def test_against_library_convolution(oracle, shape):
    B, H, W, Ci, Co, kh, kw, s, p = shape
    rng = _rng(sum(shape))
    x = synth.pm1(rng, (B, H, W, Ci))
    w = synth.pm1(rng, (Co, kh, kw, Ci))
    y = oracle.conv2d(x, w, s, p)
    assert y.dtype == np.int32
    assert np.array_equal(y, _torch_conv(x, w, s, p))      # exact: |sums| < 2**24
    # sampled entry point returns the same rows
    pix = rng.choice(y.shape[0] * y.shape[1] * y.shape[2], size=min(17, y[..., 0].size), replace=False)
    assert np.array_equal(oracle.conv2d_pixels(x, w, pix, s, p), y.reshape(-1, Co)[pix])


def test_conv_invariants(oracle):
    rng = _rng(5)
    B, H, W, Ci, Co = 2, 10, 9, 64, 48
    x = synth.pm1(rng, (B, H, W, Ci))
    w = synth.pm1(rng, (Co, 3, 3, Ci))
    y = oracle.conv2d(x, w, 2, 1).astype(np.int64)
    K = 9 * Ci
    assert np.all((y - K) % 2 == 0)
    assert np.all(np.abs(y) <= K)
    # summing over output channels = the patch against the summed filter
    wsum = w.astype(np.float32).sum(axis=0, keepdims=True)
    xt = F.pad(torch.from_numpy(x.astype(np.float32)).permute(0, 3, 1, 2), (1, 1, 1, 1), value=-1.0)
    ysum = F.conv2d(xt, torch.from_numpy(wsum).permute(0, 3, 1, 2), stride=2).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(y.sum(axis=-1, keepdims=True), ysum.astype(np.int64))
    # i.i.d. inputs: mean ~ 0, variance ~ K
    assert abs(y.mean()) < 1.0
    assert 0.8 * K < y.var() < 1.2 * K


# ---------------------------------------------------------------- GEMM

def test_gemm_against_numpy_matmul_and_operand_order(oracle):
    rng = _rng(9)
    M, N, K = 37, 19, 96
    A = synth.pm1(rng, (M, K))
    Wt = synth.pm1(rng, (N, K))
    C = oracle.gemm(A, Wt)
    assert C.shape == (M, N)
    assert np.array_equal(C, A.astype(np.int64) @ Wt.astype(np.int64).T)
    assert np.array_equal(oracle.gemm(Wt, A), C.T)


def test_xor_popcount_identity(oracle):
    rng = _rng(10)
    M, N, K = 11, 13, 160
    A = synth.pm1(rng, (M, K))
    Wt = synth.pm1(rng, (N, K))
    C = oracle.gemm(A, Wt)
    Ab, Wb = synth.pack_bits(A), synth.pack_bits(Wt)
    fl = A.astype(np.float32) @ Wt.astype(np.float32).T
    for m in range(M):
        for n in range(N):
            a = int.from_bytes(Ab[m].tobytes(), "little")
            g = int.from_bytes(Wb[n].tobytes(), "little")
            v = K - 2 * bin(a ^ g).count("1")
            assert v == C[m, n] == int(fl[m, n])


def test_1x1_conv_is_the_gemm(oracle):
    rng = _rng(11)
    B, H, W, Ci, Co = 2, 5, 3, 64, 24
    x = synth.pm1(rng, (B, H, W, Ci))
    w = synth.pm1(rng, (Co, 1, 1, Ci))
    y = oracle.conv2d(x, w, 1, 0)
    assert np.array_equal(y.reshape(-1, Co), oracle.gemm(x.reshape(-1, Ci), w.reshape(Co, Ci)))


def test_3x3_conv_is_the_gemm_of_the_patch_matrix(oracle):
    # lowering (Section 1): rows = output pixels, columns ordered (r, t, ci)
    rng = _rng(12)
    B, H, W, Ci, Co, s, p = 1, 6, 5, 32, 8, 2, 1
    x = synth.pm1(rng, (B, H, W, Ci))
    w = synth.pm1(rng, (Co, 3, 3, Ci))
    xp = np.pad(x, ((0, 0), (p, p), (p, p), (0, 0)), constant_values=-1)
    OH, OW = oracle.out_hw(H, W, 3, 3, s, p)
    rows = [xp[0, oh * s:oh * s + 3, ow * s:ow * s + 3, :].reshape(-1) for oh in range(OH) for ow in range(OW)]
    A = np.stack(rows)
    assert np.array_equal(oracle.conv2d(x, w, s, p).reshape(-1, Co), oracle.gemm(A, w.reshape(Co, -1)))


# ---------------------------------------------------------------- sign / binarize / threshold

def test_binarize_special_values_and_replication(oracle):
    tiny = np.float32(1e-45)
    x = np.array([0.0, -0.0, tiny, -tiny, np.inf, -np.inf, np.nan, -1.5], np.float32).reshape(1, 1, 2, 4)
    out = oracle.binarize(x, None, R=1)
    assert out.reshape(-1).tolist() == [1, 1, 1, -1, 1, -1, -1, -1]
    # replication: output channel c reads input channel c mod C_in, bias indexed by c
    x = np.array([0.25, -0.25, 1.0, -1.0], np.float32).reshape(1, 1, 1, 4)
    bias = np.array([0, 0, 0, 0, -0.5, 0.5, -2.0, 2.0], np.float32)
    assert oracle.binarize(x, bias, R=2).reshape(-1).tolist() == [1, -1, 1, -1, -1, 1, -1, 1]
    # x + bias rounds in fp32: 1 + 2**-25 == 1 exactly, so (-1) + that is 0 -> +1
    x = np.array([-1.0] * 4, np.float32).reshape(1, 1, 1, 4)
    bias = np.array([1.0, np.float32(1.0) - np.float32(2.0 ** -24), 1.0, 1.0], np.float32)
    assert oracle.binarize(x, bias, 1).reshape(-1).tolist() == [1, -1, 1, 1]


def test_binarize_against_numpy(oracle):
    rng = _rng(13)
    x = synth.real_input(rng, (2, 5, 7, 12))
    bias = synth.real_input(rng, (36,))
    got = oracle.binarize(x, bias, R=3)
    want = np.where(np.tile(x, (1, 1, 1, 3)) + bias >= 0, 1, -1)
    assert np.array_equal(got, want)
    assert np.array_equal(oracle.sign_weights(x), np.where(x >= 0, 1, -1))


def test_threshold_tie_rule(oracle):
    acc = np.array([[4, -2, 0], [6, -2, -2]], np.int32)
    thr = np.array([5, -2, 1], np.int32)          # acc-1 / tie / acc+1 patterns
    assert oracle.threshold(acc, thr).tolist() == [[-1, 1, -1], [1, 1, -1]]


# ---------------------------------------------------------------- packed checker == oracle

@pytest.mark.parametrize("shape", [
    (2, 9, 13, 32, 40, 3, 3, 1, 1),
    (1, 12, 10, 64, 24, 3, 3, 2, 1),
    (3, 5, 6, 96, 16, 1, 1, 1, 0),
    (2, 7, 11, 32, 8, 1, 3, 1, 2),
    (1, 32, 32, 128, 128, 3, 3, 1, 1),
])
def test_checker_conv_equals_oracle(oracle, shape):
    B, H, W, Ci, Co, kh, kw, s, p = shape
    rng = _rng(31 + sum(shape))
    x = synth.pm1(rng, (B, H, W, Ci))
    w = synth.pm1(rng, (Co, kh, kw, Ci))
    got = oracle.checker_conv2d(synth.pack_bits(x), synth.pack_bits(w), (B, H, W, Ci, Co, kh, kw), s, p)
    assert np.array_equal(got, oracle.conv2d(x, w, s, p))


def test_checker_gemm_equals_oracle(oracle):
    rng = _rng(40)
    M, N, K = 70, 45, 320
    A = synth.pm1(rng, (M, K))
    Wt = synth.pm1(rng, (N, K))
    want = oracle.gemm(A, Wt)
    Ab, Wb = synth.pack_bits(A), synth.pack_bits(Wt)
    assert np.array_equal(oracle.checker_gemm(Ab, Wb, M, N, K), want)
    assert np.array_equal(oracle.checker_gemm(Ab, Wb, M, N, K, rows=(13, 29)), want[13:29])


def test_pack_unpack_layout():
    v = -np.ones((1, 40), np.int8)
    v[0, 0] = 1
    v[0, 9] = 1
    v[0, 39] = 1
    b = synth.pack_bits(v)
    assert b.tolist() == [[0x01, 0x02, 0x00, 0x00, 0x80]]
    assert b[:, :4].copy().view("<u4").tolist() == [[0x00000201]]
    assert np.array_equal(synth.unpack_bits(b), v)
