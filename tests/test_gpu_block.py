"""GPU parity of the building-block pieces beyond the single binary convolution: the module with P parallel binary
branches (bit-exact), the F x F convolution as F*F shifted branches (bit-exact, both padding readings), the depth-wise
3x3 module, average pooling, global pooling and the fully connected layer (fp32 on the GPU against the fp64 oracle,
within the stated tolerance).  Everything goes through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2010_00704_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bk():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2010_00704_b200 import build, binding
    build.build()
    binding.load()
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def dev_f16(a):
    return dev(np.ascontiguousarray(a, dtype=np.float16).view(np.uint8).reshape(-1))


def _branch_case(rng, B, H, W, Ci, Co, P):
    x = rng.standard_normal((B, H, W, Ci)).astype(np.float16)
    biases = (rng.standard_normal((P, Ci)) * 0.5).astype(np.float32)
    ws = synth.pm1(rng, (P, Co, Ci))
    sc = (rng.standard_normal((P, Co)) / np.sqrt(Ci)).astype(np.float32)
    sc[:, ::5] *= -1
    sh = rng.standard_normal((P, Co)).astype(np.float32)
    sl = rng.uniform(-0.25, 1.0, Co).astype(np.float32)
    nb = rng.standard_normal(Co).astype(np.float32)
    ident = rng.standard_normal((B, H, W, Co)).astype(np.float16)
    return x, biases, ws, sc, sh, sl, nb, ident


def _run_branches(bk, x, biases, ws, sc, sh, sl, nb, ident, pad_dot, kh, kw, in_place=False, want_bits=True):
    B, H, W, Ci = x.shape
    P, Co, _ = ws.shape
    # the P binarizations are ONE pack call with R = P and the branch biases concatenated
    xbits = torch.empty(B * H * W * P * Ci // 8, dtype=torch.uint8, device="cuda")
    bk.bcnn_pack(dev(x.astype(np.float32)), dev(biases.reshape(-1)), xbits, B, H, W, Ci, P)
    n = B * H * W * Co
    yreal = torch.full((2 * n + 512,), 0xA5, dtype=torch.uint8, device="cuda")
    ybits = torch.full((n // 8 + 512,), 0xA5, dtype=torch.uint8, device="cuda")
    yv, bv = yreal[256:256 + 2 * n], ybits[256:256 + n // 8]
    id_dev = None
    if ident is not None:
        if in_place:
            yv.copy_(dev_f16(ident))
            id_dev = yv
        else:
            id_dev = dev_f16(ident)
    bk.bcnn_conv2d_b1_branches(xbits, dev(synth.pack_bits(ws)), dev(sc), dev(sh), None if pad_dot is None else dev(pad_dot),
                               id_dev, dev(sl), dev(nb) if nb is not None else None, yv, bv if want_bits else None,
                               B, H, W, Ci, Co, P, kh, kw)
    torch.cuda.synchronize()
    for raw, m in ((yreal, 2 * n), (ybits, n // 8)):
        r = raw.cpu().numpy()
        assert np.all(r[:256] == 0xA5) and np.all(r[256 + m:] == 0xA5), "write outside the output buffer"
    y = yv.cpu().numpy().view(np.uint16).reshape(B, H, W, Co)
    s = synth.unpack_bits(bv.cpu().numpy().reshape(B, H, W, Co // 8)) if want_bits else None
    return y, s


BRANCH_SHAPES = [
    # B, H, W, Ci, Co, P
    (2, 9, 13, 64, 64, 2),        # the paper's P = 2 on its 64-channel module
    (1, 20, 21, 32, 32, 2),
    (2, 7, 11, 128, 128, 2),
    (1, 5, 6, 256, 320, 3),       # sliced output channels, ragged last slice
    (3, 4, 5, 96, 64, 1),         # P = 1: the plain module
    (1, 3, 3, 512, 1024, 2),      # wide: several slices
]


@pytest.mark.parametrize("variant", ["full", "no_identity", "in_place", "no_bits"])
@pytest.mark.parametrize("shape", BRANCH_SHAPES)
def test_parallel_branches(bk, oracle, shape, variant):
    B, H, W, Ci, Co, P = shape
    rng = np.random.default_rng(8800 + sum(shape))
    x, biases, ws, sc, sh, sl, nb, ident = _branch_case(rng, B, H, W, Ci, Co, P)
    accs = np.stack([oracle.conv2d(oracle.binarize(x.astype(np.float32), biases[p], 1), ws[p][:, None, None, :], 1, 0)
                     for p in range(P)])
    use_id = None if variant == "no_identity" else ident
    want_y, want_s = oracle.conv_module_branches(accs, sc, sh, use_id, sl, nb)
    y, s = _run_branches(bk, x, biases, ws, sc, sh, sl, nb, use_id, None, 1, 1, in_place=variant == "in_place",
                         want_bits=variant != "no_bits")
    assert np.array_equal(y, want_y.view(np.uint16))
    if s is not None:
        assert np.array_equal(s, want_s)
    if P == 1 and variant == "full":
        # ... and for one branch the tensor-core module call gives the same bits
        yreal = torch.empty(B * H * W * Co * 2, dtype=torch.uint8, device="cuda")
        ybits = torch.empty(B * H * W * Co // 8, dtype=torch.uint8, device="cuda")
        xb = torch.empty(B * H * W * Ci // 8, dtype=torch.uint8, device="cuda")
        bk.bcnn_pack(dev(x.astype(np.float32)), dev(biases[0]), xb, B, H, W, Ci, 1)
        bk.bcnn_conv2d_b1_module(xb, dev(synth.pack_bits(ws[0])), dev(sc[0]), dev(sh[0]), dev_f16(ident), dev(sl), dev(nb),
                                 yreal, ybits, B, H, W, Ci, Co, 1, 1, 1, 0)
        torch.cuda.synchronize()
        assert np.array_equal(yreal.cpu().numpy().view(np.uint16).reshape(B, H, W, Co), y)
    assert bk.bcnn_device_error() == 0


@pytest.mark.parametrize("reading", ["paper", "zero"])
@pytest.mark.parametrize("shape", [(2, 9, 11, 64, 64, 3), (1, 6, 5, 32, 96, 3), (1, 4, 4, 32, 32, 5), (1, 1, 7, 64, 32, 3)])
def test_fxf_as_shifted_branches(bk, oracle, shape, reading):
    # binary k x k convolution as k*k shifted 1x1 branches with a real scale per tap (Section 4.2.1, last paragraph):
    # "paper" pads the real map with zeros before each branch's bias and sign (pad_dot = the convolution of the bias
    # signs), "zero" lets a tap outside the image contribute nothing (pad_dot = NULL)
    B, H, W, Ci, Co, k = shape
    P = k * k
    rng = np.random.default_rng(8900 + sum(shape))
    x, biases, ws, sc, sh, sl, nb, ident = _branch_case(rng, B, H, W, Ci, Co, P)
    accs, _ = oracle.shifted_branch_accs(x, biases, ws, k, k, pad_zero_contribution=reading == "zero")
    want_y, want_s = oracle.conv_module_branches(accs, sc, sh, ident, sl, nb)
    pad_dot = None
    if reading == "paper":
        pad_dot = np.stack([(np.where(biases[p] >= 0, 1, -1)[None, :] * ws[p].astype(np.int32)).sum(axis=1) for p in range(P)]).astype(np.int32)
    y, s = _run_branches(bk, x, biases, ws, sc, sh, sl, nb, ident, pad_dot, k, k)
    assert np.array_equal(y, want_y.view(np.uint16))
    assert np.array_equal(s, want_s)
    assert bk.bcnn_device_error() == 0


def test_branches_errors(bk):
    a = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    f = torch.zeros(4096, dtype=torch.float32, device="cuda")
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_conv2d_b1_branches(a, a, f, f, None, None, f, None, a, None, 1, 4, 4, 32, 32, 2, 3, 3)   # P != kh * kw
    assert e.value.status == -1
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_conv2d_b1_branches(a, a, f, f, None, None, f, None, a, None, 1, 4, 4, 48, 32, 2, 1, 1)
    assert e.value.status == -2
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_conv2d_b1_branches(a, a, f[1:], f, None, None, f, None, a, None, 1, 4, 4, 32, 32, 2, 1, 1)
    assert e.value.status == -3
    torch.cuda.synchronize()
    assert int(a.sum()) == 0


def _ulp_distance(got_u16, want_f16):
    def key(u):                                                   # monotone integer key of a float16 bit pattern
        s = u.astype(np.int32)
        return np.where(s & 0x8000, -(s & 0x7FFF), s & 0x7FFF)
    return np.abs(key(got_u16) - key(want_f16.view(np.uint16)))


# Tolerance of the real-valued vector operations: the GPU sums at most nine products (or S*S values) in fp32, each
# step within 2^-24 relative, then rounds once to float16 (2^-11): against the fp64 oracle's single rounding the
# stored value can land on the neighbouring float16 only when the exact value lies within about 2^-20 relative of
# a rounding boundary, i.e. for well under 1 % of the elements, and never by more than one unit in the last place.
@pytest.mark.parametrize("shape", [(2, 9, 11, 16, 1, 1), (2, 12, 10, 32, 1, 2), (1, 7, 7, 8, 4, 1), (3, 8, 8, 32, 2, 2),
                                   (1, 1, 1, 64, 1, 1), (1, 56, 56, 64, 2, 2)])
def test_dwconv3x3_module(bk, oracle, shape):
    B, H, W, Ci, R, S = shape
    C = Ci * R
    rng = np.random.default_rng(9200 + sum(shape))
    x = rng.standard_normal((B, H, W, Ci)).astype(np.float16)
    w = (rng.standard_normal((C, 3, 3)) / 3).astype(np.float32)
    sc, sh = rng.standard_normal(C).astype(np.float32), rng.standard_normal(C).astype(np.float32)
    sl = rng.uniform(-0.25, 0.5, C).astype(np.float32)
    nb = rng.standard_normal(C).astype(np.float32)
    want = oracle.dwconv3x3_module(x, w, sc, sh, sl, R=R, S=S)
    OH, OW = want.shape[1:3]
    n = B * OH * OW * C
    y = torch.empty(2 * n, dtype=torch.uint8, device="cuda")
    bits = torch.empty(n // 8, dtype=torch.uint8, device="cuda") if C % 32 == 0 else None
    bk.bcnn_dwconv3x3_module(dev_f16(x), dev(w), dev(sc), dev(sh), dev(sl), dev(nb), y, bits, B, H, W, Ci, R, S)
    torch.cuda.synchronize()
    got = y.cpu().numpy().view(np.uint16).reshape(B, OH, OW, C)
    d = _ulp_distance(got, want)
    assert d.max() <= 1 and (d > 0).mean() < 0.01
    if bits is not None:
        # the sign is taken of the STORED value (both sides in fp32 on the same float16 input): bit-exact given the map
        want_s = oracle.binarize(got.view(np.float16).astype(np.float32), nb, 1)
        assert np.array_equal(synth.unpack_bits(bits.cpu().numpy().reshape(B, OH, OW, C // 8)), want_s)


@pytest.mark.parametrize("shape", [(2, 8, 12, 16, 1, 2), (1, 9, 6, 8, 2, 3), (2, 5, 7, 32, 4, 1), (1, 56, 56, 64, 2, 2)])
def test_avgpool(bk, oracle, shape):
    B, H, W, Ci, R, S = shape
    rng = np.random.default_rng(9300 + sum(shape))
    x = rng.standard_normal((B, H, W, Ci)).astype(np.float16)
    want = oracle.avgpool(x, S, R)
    y = torch.empty(2 * want.size, dtype=torch.uint8, device="cuda")
    bk.bcnn_avgpool(dev_f16(x), y, B, H, W, Ci, R, S)
    torch.cuda.synchronize()
    got = y.cpu().numpy().view(np.uint16).reshape(want.shape)
    d = _ulp_distance(got, want)
    assert d.max() <= 1 and (d > 0).mean() < 0.01
    if S == 1:
        assert np.array_equal(got, want.view(np.uint16))           # pure replication: exact


def test_gap_and_fc(bk, oracle):
    # head of the paper's network: 7 x 7 x 1024 -> 1024 -> 1000 (Table 1), batch 9 (not a multiple of the images a CTA
    # takes); fp32 sums of 49 / 1024 terms against fp64: relative to the sum of magnitudes within 1024 * 2^-24
    rng = np.random.default_rng(9400)
    B, H, W, C, N = 9, 7, 7, 1024, 1000
    x = rng.standard_normal((B, H, W, C)).astype(np.float16)
    wfc = (rng.standard_normal((N, C)) / 32).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    pooled = torch.empty(B * C, dtype=torch.float32, device="cuda")
    logits = torch.empty(B * N, dtype=torch.float32, device="cuda")
    bk.bcnn_gap(dev_f16(x), pooled, B, H, W, C)
    bk.bcnn_fc(pooled, dev(wfc), dev(bias), logits, B, C, N)
    torch.cuda.synchronize()
    want_p = oracle.gap(x)
    got_p = pooled.cpu().numpy().reshape(B, C).astype(np.float64)
    mag_p = np.abs(x.astype(np.float64)).mean(axis=(1, 2))
    assert np.all(np.abs(got_p - want_p) <= 64 * 2.0 ** -24 * mag_p + 1e-30)
    want_l = oracle.fc(got_p, wfc, bias)                             # the layer on the GPU's own pooled values
    mag_l = np.abs(got_p) @ np.abs(wfc.astype(np.float64)).T + np.abs(bias.astype(np.float64))
    got_l = logits.cpu().numpy().reshape(B, N).astype(np.float64)
    assert np.all(np.abs(got_l - want_l) <= 1100 * 2.0 ** -24 * mag_l)
    # and end to end against the oracle's own pooling
    assert np.allclose(got_l, oracle.fc(want_p, wfc, bias), rtol=0, atol=1e-4 * mag_l.max())


def test_block_ops_errors(bk):
    a = torch.zeros(1 << 14, dtype=torch.uint8, device="cuda")
    f = torch.zeros(1024, dtype=torch.float32, device="cuda")
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_avgpool(a, a, 1, 5, 4, 8, 1, 2)                      # H not a multiple of S
    assert e.value.status == -1
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_dwconv3x3_module(a, f, f, f, f, None, a, None, 1, 4, 4, 12, 1, 1)   # C_in % 8 != 0
    assert e.value.status == -2
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_gap(a[2:], f, 1, 2, 2, 8)
    assert e.value.status == -3
    with pytest.raises(bk.BcnnError):
        bk.bcnn_fc(f, None, None, f, 1, 8, 4)
    torch.cuda.synchronize()
    assert int(a.sum()) == 0
