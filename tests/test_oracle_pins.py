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


# ---- convolution module: batch norm -> + identity -> PReLU -> fp16 store -> next sign (Section 4.2.1) ----

def test_conv_module_hand_worked(oracle):
    # four channels worked by hand with exactly representable numbers:
    #   c0: 3*0.5 + 0.25 = 1.75, + 1 = 2.75 (>= 0 stays);           sign(2.75 - 3) = -1
    #   c1: -3*0.5 + 0.25 = -1.25, + 1 = -0.25, * 0.25 = -0.0625;   sign(-0.0625 + 0.0625 = 0) = +1 (tie goes up)
    #   c2: 0*2 - 1 = -1, + 0.5 = -0.5, * 0.125 = -0.0625;          sign(-0.0625 + 0.0625) = +1
    #   c3: 5*(-1) + 1 = -4, - 10 = -14, * 0.5 = -7;                sign(-7 + 7) = +1
    acc = np.array([[3, -3, 0, 5]], np.int32)
    y, s = oracle.conv_module(acc, [0.5, 0.5, 2, -1], [0.25, 0.25, -1, 1], np.array([[1, 1, 0.5, -10]], np.float16),
                              [0.25, 0.25, 0.125, 0.5], [-3, 0.0625, 0.0625, 7])
    assert y.dtype == np.float16 and y.tolist() == [[2.75, -0.0625, -0.0625, -7.0]]
    assert s.tolist() == [[-1, 1, 1, 1]]


def test_conv_module_pass_through_and_relu(oracle):
    # scale 1, shift 0, no identity, slope 1: the stored map is the integer sum itself (exact in fp16 up to 2048);
    # slope 0 makes the PReLU a ReLU
    acc = np.arange(-2048, 2049, dtype=np.int32).reshape(-1, 1)
    one, zero = np.ones(1, np.float32), np.zeros(1, np.float32)
    y, _ = oracle.conv_module(acc, one, zero, None, one, None, want_sign=False)
    assert np.array_equal(y.astype(np.int32), acc)
    y, _ = oracle.conv_module(acc, one, zero, None, zero, None, want_sign=False)
    assert np.array_equal(y.astype(np.int32), np.maximum(acc, 0))


def test_conv_module_fp16_ties_and_sign_of_stored_value(oracle):
    # 2049 and 2051 lie halfway between fp16 neighbours: round to even gives 2048 and 2052;
    # the next sign looks at the STORED value: 2049 -> 2048, and 2048 - 2048.5 < 0 although 2049 - 2048.5 > 0
    acc = np.array([[2049], [2051], [2050]], np.int32)
    one, zero = np.ones(1, np.float32), np.zeros(1, np.float32)
    y, s = oracle.conv_module(acc, one, zero, None, one, np.array([-2048.5], np.float32))
    assert y.astype(np.float32).ravel().tolist() == [2048.0, 2052.0, 2050.0]
    assert s.ravel().tolist() == [-1, 1, 1]
    # overflow of the fp16 range stores infinity, a NaN scale stores NaN whose sign is -1
    y, s = oracle.conv_module(np.array([[70000]], np.int32), one, zero, None, one, zero)
    assert np.isinf(y[0, 0]) and s[0, 0] == 1
    y, s = oracle.conv_module(np.array([[1]], np.int32), np.array([np.nan], np.float32), zero, None, one, zero)
    assert np.isnan(y[0, 0]) and s[0, 0] == -1
    # negative zero (0 * -1 = -0, -0 + -0 = -0) is >= 0: it passes the PReLU unchanged and its sign is +1
    y, s = oracle.conv_module(np.array([[0]], np.int32), np.array([-1.0], np.float32), np.array([-0.0], np.float32), None,
                              np.array([7.0], np.float32), zero)
    assert np.signbit(y[0, 0]) and y[0, 0] == 0 and s[0, 0] == 1


def test_conv_module_reduces_to_the_integer_threshold(oracle):
    # unit scale, integer shift and next bias, no identity, slope 1: sign(acc + b + nb >= 0) is the integer
    # threshold acc >= -(b + nb) of the fused path (sums stay below 2048, exact in fp16)
    rng = np.random.default_rng(31)
    N = 24
    acc = rng.integers(-900, 901, size=(50, N)).astype(np.int32)
    b = rng.integers(-100, 101, size=N).astype(np.float32)
    nb = rng.integers(-100, 101, size=N).astype(np.float32)
    _, s = oracle.conv_module(acc, np.ones(N, np.float32), b, None, np.ones(N, np.float32), nb)
    assert np.array_equal(s, oracle.threshold(acc, (-(b + nb)).astype(np.int32)))


def test_conv_module_against_elementwise_numpy(oracle):
    # numpy restatement, one IEEE fp32 operation per step (numpy never fuses), fp16 conversion by astype;
    # the sign is the already pinned binarize() of the stored map
    rng = np.random.default_rng(32)
    N = 40
    acc = rng.integers(-1152, 1153, size=(3, 5, 7, N)).astype(np.int32)
    scale = rng.standard_normal(N).astype(np.float32) * np.float32(0.05)
    shift = rng.standard_normal(N).astype(np.float32)
    slope = rng.uniform(-0.5, 1.5, N).astype(np.float32)
    ident = rng.standard_normal(acc.shape).astype(np.float16)
    nb = rng.standard_normal(N).astype(np.float32)
    y, s = oracle.conv_module(acc, scale, shift, ident, slope, nb)
    t = acc.astype(np.float32) * scale
    t = t + shift
    u = t + ident.astype(np.float32)
    r = np.where(u >= 0, u, slope * u).astype(np.float32)
    want = r.astype(np.float16)
    assert np.array_equal(y.view(np.uint16), want.view(np.uint16))
    assert np.array_equal(s, oracle.binarize(want.astype(np.float32), nb, 1))
    # planting a mistake must show: sign of the unrounded value differs somewhere on a finer grid
    y2, _ = oracle.conv_module(acc, scale, shift, None, slope, None, want_sign=False)
    assert not np.array_equal(y2.view(np.uint16), y.view(np.uint16))
