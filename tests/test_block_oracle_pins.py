"""Pins for the oracle of the rest of the building block (oracle/bcnn_block_oracle.c): parallel binary branches and
the shifted-branch form of an F x F convolution, the depth-wise 3x3 module, average pooling, global pooling and the
fully connected layer.  Each function is checked against something other than itself: the single-branch function,
cases worked by hand, closed forms, the float64 library routines, and the already pinned -1-padded convolution."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from paper_2010_00704_b200 import synth


def _rng(i):
    return np.random.default_rng(8100 + i)


# ---------------------------------------------------------------- parallel branches (Section 4.2.1, Figure 4 bottom)

def test_one_branch_is_the_plain_module(oracle):
    rng = _rng(1)
    rows, N = 37, 40
    acc = rng.integers(-64, 65, (1, rows, N)).astype(np.int32)
    sc, sh, sl, nb = (rng.standard_normal(N).astype(np.float32) for _ in range(4))
    ident = rng.standard_normal((rows, N)).astype(np.float16)
    y1, s1 = oracle.conv_module(acc[0], sc, sh, ident, sl, nb)
    yp, sp = oracle.conv_module_branches(acc, sc[None], sh[None], ident, sl, nb)
    assert np.array_equal(y1.view(np.uint16), yp.view(np.uint16)) and np.array_equal(s1, sp)


def test_two_branches_hand_worked(oracle):
    # one row, four channels; every number below is exact in fp32 and fp16, so the expected values are the real ones
    acc = np.array([[[4, -2, 6, 0]], [[-8, 2, 1, 3]]], np.int32)                 # [P=2][rows=1][N=4]
    scale = np.array([[0.5, 1.0, 0.25, 2.0], [0.25, -1.0, 2.0, 0.5]], np.float32)
    shift = np.array([[1.0, 0.0, -0.5, 0.0], [0.0, 0.5, 0.0, -1.0]], np.float32)
    ident = np.array([[0.5, -4.0, 0.0, -2.0]], np.float16)
    slope = np.array([0.5, 0.25, 0.5, 0.5], np.float32)
    nbias = np.array([-1.0, 2.0, -4.0, 0.75], np.float32)
    # branch terms: p=0: 3, -2, 1, 0;  p=1: -2, -1.5, 2, 0.5;  sum: 1, -3.5, 3, 0.5;  + identity: 1.5, -7.5, 3, -1.5
    # PReLU: 1.5, -1.875, 3, -0.75;  + next bias: 0.5, 0.125, -1, 0 -> signs + + - +
    y, s = oracle.conv_module_branches(acc, scale, shift, ident, slope, nbias)
    assert y.tolist() == [[1.5, -1.875, 3.0, -0.75]]
    assert s.tolist() == [[1, 1, -1, 1]]


def test_branches_are_summed_left_to_right_in_fp32(oracle):
    # 2^24 + 1 is not an fp32 number: (2^24 + 1) + (-2^24) = 0 when the first two terms are added first,
    # but 2^24 + (1 - 2^24) = 1 in the other order; the stated order is left to right
    acc = np.array([[[1]], [[1]], [[1]]], np.int32)
    scale = np.array([[16777216.0], [1.0], [-16777216.0]], np.float32)
    shift = np.zeros((3, 1), np.float32)
    one = np.ones(1, np.float32)
    y, _ = oracle.conv_module_branches(acc, scale, shift, None, one, None)
    assert float(y[0, 0]) == 0.0
    y, _ = oracle.conv_module_branches(acc[[0, 2, 1]], scale[[0, 2, 1]], shift, None, one, None)
    assert float(y[0, 0]) == 1.0


def test_branches_against_elementwise_numpy(oracle):
    rng = _rng(2)
    P, rows, N = 3, 50, 24
    acc = rng.integers(-200, 201, (P, rows, N)).astype(np.int32)
    sc = (rng.standard_normal((P, N)) / 8).astype(np.float32)
    sh = rng.standard_normal((P, N)).astype(np.float32)
    sl = rng.uniform(-0.5, 1, N).astype(np.float32)
    nb = rng.standard_normal(N).astype(np.float32)
    ident = rng.standard_normal((rows, N)).astype(np.float16)
    t = None
    for p in range(P):                                    # numpy never fuses: one fp32 operation per step
        tp = acc[p].astype(np.float32) * sc[p][None, :]
        tp = tp + sh[p][None, :]
        t = tp if t is None else t + tp
    u = t + ident.astype(np.float32)
    r = np.where(u >= 0, u, sl[None, :] * u).astype(np.float32)
    want_y = r.astype(np.float16)
    want_s = np.where(want_y.astype(np.float32) + nb[None, :] >= 0, 1, -1)
    y, s = oracle.conv_module_branches(acc, sc, sh, ident, sl, nb)
    assert np.array_equal(y.view(np.uint16), want_y.view(np.uint16)) and np.array_equal(s, want_s)


# ---------------------------------------------------------------- F x F convolution as F*F shifted 1x1 branches

def _fxf_inputs(rng, B, H, W, Ci, Co, k):
    x = rng.standard_normal((B, H, W, Ci)).astype(np.float16)
    x[x == 0] = np.float16(0.5)                          # keep sign(x) two-valued
    w = synth.pm1(rng, (k * k, Co, Ci))
    return x, w


@pytest.mark.parametrize("k,H,W", [(3, 6, 7), (3, 1, 4), (5, 7, 5), (1, 3, 3)])
def test_shifted_branches_with_zero_contribution_are_the_zero_padded_convolution(oracle, k, H, W):
    # no bias, taps outside the image contribute nothing, unit scales: the sum of the branches is the textbook
    # zero-padded convolution of sign(x) with the k x k weights
    rng = _rng(10 + k + H)
    B, Ci, Co = 2, 32, 5
    x, w = _fxf_inputs(rng, B, H, W, Ci, Co, k)
    accs, inside = oracle.shifted_branch_accs(x, np.zeros((k * k, Ci), np.float32), w, k, k, pad_zero_contribution=True)
    total = accs.sum(axis=0)
    xs = torch.from_numpy(np.where(x.astype(np.float32) >= 0, 1.0, -1.0)).permute(0, 3, 1, 2).double()
    wt = torch.from_numpy(w.reshape(k, k, Co, Ci).astype(np.float64)).permute(2, 3, 0, 1)      # [Co][Ci][r][t]
    want = F.conv2d(xs, wt, padding=(k - 1) // 2).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(total, want.astype(np.int32))
    # the inside masks: tap (r, t) of pixel (h, w) lies inside iff the shifted pixel does
    for p in range(k * k):
        r, t = divmod(p, k)
        hh, ww = np.meshgrid(np.arange(H) + r - (k - 1) // 2, np.arange(W) + t - (k - 1) // 2, indexing="ij")
        assert np.array_equal(inside[p], (hh >= 0) & (hh < H) & (ww >= 0) & (ww < W))


def test_shifted_branches_with_negative_bias_are_the_minus_one_padded_convolution(oracle):
    # the paper pads the REAL map with zeros before the branch's bias and sign: with a small negative bias that
    # changes no sign inside the image the padding binarizes to -1, and the sum of the nine branches must be the
    # (separately pinned) 3x3 convolution with -1 padding; with a small positive bias the padding is +1
    rng = _rng(20)
    B, H, W, Ci, Co, k = 2, 5, 6, 32, 4, 3
    x, w = _fxf_inputs(rng, B, H, W, Ci, Co, k)
    bits = np.where(x.astype(np.float32) >= 0, 1, -1).astype(np.int8)
    w4 = np.ascontiguousarray(w.reshape(k, k, Co, Ci).transpose(2, 0, 1, 3))                   # [Co][r][t][Ci]
    tiny = np.full((k * k, Ci), 1e-4, np.float32)
    accs, _ = oracle.shifted_branch_accs(x, -tiny, w, k, k)
    assert np.array_equal(accs.sum(axis=0), oracle.conv2d(bits, w4, 1, 1))
    accs, _ = oracle.shifted_branch_accs(x, tiny, w, k, k)
    xp = torch.from_numpy(bits.astype(np.float64)).permute(0, 3, 1, 2)
    want = F.conv2d(F.pad(xp, (1, 1, 1, 1), value=1.0), torch.from_numpy(w4.astype(np.float64)).permute(0, 3, 1, 2))
    assert np.array_equal(accs.sum(axis=0), want.permute(0, 2, 3, 1).numpy().astype(np.int32))


def test_shifted_branch_padding_is_the_convolution_of_the_bias_signs(oracle):
    # where a branch looks outside the image its result is sum_ci sign(0 + bias[ci]) * w[co][ci], whatever x holds
    rng = _rng(21)
    B, H, W, Ci, Co, k = 1, 4, 4, 32, 6, 3
    x, w = _fxf_inputs(rng, B, H, W, Ci, Co, k)
    biases = rng.standard_normal((k * k, Ci)).astype(np.float32)
    biases[3, :4] = [0.0, -0.0, 1.0, -1.0]
    accs, inside = oracle.shifted_branch_accs(x, biases, w, k, k)
    for p in range(k * k):
        pad_dot = (np.where(biases[p] >= 0, 1, -1)[None, :] * w[p].astype(np.int32)).sum(axis=1)
        out = ~inside[p]
        assert np.all(accs[p][:, out, :] == pad_dot[None, None, :])


# ---------------------------------------------------------------- depth-wise 3x3 module, pooling, head

def test_dwconv_delta_kernel_is_the_pointwise_module(oracle):
    rng = _rng(30)
    B, H, W, C = 2, 5, 6, 16
    x = rng.standard_normal((B, H, W, C)).astype(np.float16)
    w = np.zeros((C, 3, 3), np.float32)
    w[:, 1, 1] = 1.0
    sc, sh = rng.standard_normal(C).astype(np.float32), rng.standard_normal(C).astype(np.float32)
    sl = rng.uniform(0, 0.5, C).astype(np.float32)
    t = x.astype(np.float64) * sc.astype(np.float64) + sh.astype(np.float64)
    want = np.where(t >= 0, t, sl.astype(np.float64) * t).astype(np.float16)
    assert np.array_equal(oracle.dwconv3x3_module(x, w, sc, sh, sl).view(np.uint16), want.view(np.uint16))


def test_dwconv_constant_input_counts_the_taps_inside(oracle):
    # all-ones input and weights, unit batch norm: interior 9, edges 6, corners 4 (zero padding); stride 2 keeps
    # the windows centred on even pixels
    B, H, W, C = 1, 6, 8, 8
    one = np.ones(C, np.float32)
    y = oracle.dwconv3x3_module(np.ones((B, H, W, C), np.float16), np.ones((C, 3, 3), np.float32), one, 0 * one, one)
    expect = np.full((H, W), 9.0)
    expect[0, :] = expect[-1, :] = 6.0
    expect[:, 0] = expect[:, -1] = 6.0
    expect[0, 0] = expect[0, -1] = expect[-1, 0] = expect[-1, -1] = 4.0
    assert np.array_equal(y[0, :, :, 3].astype(np.float64), expect)
    y2 = oracle.dwconv3x3_module(np.ones((B, H, W, C), np.float16), np.ones((C, 3, 3), np.float32), one, 0 * one, one, S=2)
    assert y2.shape == (1, 3, 4, C)
    assert np.array_equal(y2[0, :, :, 0].astype(np.float64), expect[::2, ::2])


@pytest.mark.parametrize("S,R", [(1, 1), (2, 1), (1, 2), (2, 4)])
def test_dwconv_against_library_depthwise_convolution(oracle, S, R):
    rng = _rng(31 + S + R)
    B, H, W, Ci = 2, 7, 9, 6
    C = Ci * R
    x = rng.standard_normal((B, H, W, Ci)).astype(np.float16)
    w = rng.standard_normal((C, 3, 3)).astype(np.float32)
    sc, sh = rng.standard_normal(C).astype(np.float32), rng.standard_normal(C).astype(np.float32)
    sl = rng.uniform(-0.25, 0.5, C).astype(np.float32)
    xr = torch.from_numpy(np.tile(x.astype(np.float64), (1, 1, 1, R))).permute(0, 3, 1, 2)     # channel c <- c mod Ci
    conv = F.conv2d(xr, torch.from_numpy(w.astype(np.float64))[:, None], stride=S, padding=1, groups=C)
    t = conv.permute(0, 2, 3, 1).numpy() * sc.astype(np.float64) + sh.astype(np.float64)
    want = np.where(t >= 0, t, sl.astype(np.float64) * t).astype(np.float16)
    got = oracle.dwconv3x3_module(x, w, sc, sh, sl, R=R, S=S)
    assert got.shape == want.shape
    # the library may sum the nine products in another order: equal up to one float16 unit in the last place
    diff = np.abs(got.view(np.int16).astype(np.int32) - want.view(np.int16).astype(np.int32))
    assert diff.max() <= 1 and (diff > 0).mean() < 0.01


def test_avgpool_hand_values_library_and_replication(oracle):
    x = np.arange(16, dtype=np.float16).reshape(1, 4, 4, 1)
    assert oracle.avgpool(x, 2)[0, :, :, 0].tolist() == [[2.5, 4.5], [10.5, 12.5]]
    rng = _rng(40)
    x = rng.standard_normal((2, 6, 9, 5)).astype(np.float16)
    want = F.avg_pool2d(torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2), 3).permute(0, 2, 3, 1).numpy()
    got = oracle.avgpool(x, 3, R=2)
    assert got.shape == (2, 2, 3, 10)
    assert np.array_equal(got[..., :5].view(np.uint16), want.astype(np.float16).view(np.uint16))
    assert np.array_equal(got[..., 5:], got[..., :5])                 # channel c reads channel c mod C_in
    assert np.array_equal(oracle.avgpool(x, 1).view(np.uint16), x.view(np.uint16))


def test_gap_and_fc_against_numpy(oracle):
    rng = _rng(50)
    B, H, W, C, N = 3, 7, 7, 24, 10
    x = rng.standard_normal((B, H, W, C)).astype(np.float16)
    pooled = oracle.gap(x)
    assert np.allclose(pooled, x.astype(np.float64).mean(axis=(1, 2)), rtol=0, atol=1e-15)
    assert np.array_equal(oracle.gap(np.full((1, 2, 3, 4), 1.5, np.float16)), np.full((1, 4), 1.5))
    w = rng.standard_normal((N, C)).astype(np.float32)
    b = rng.standard_normal(N).astype(np.float32)
    want = pooled @ w.astype(np.float64).T + b.astype(np.float64)
    assert np.allclose(oracle.fc(pooled, w, b), want, rtol=1e-14, atol=1e-14)
    # operand order: a one-hot weight row picks one pooled channel
    w1 = np.zeros((2, C), np.float32)
    w1[1, 5] = 2.0
    assert np.allclose(oracle.fc(pooled, w1, None), np.stack([0 * pooled[:, 0], 2 * pooled[:, 5]], axis=1))
