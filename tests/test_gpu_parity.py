"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

from paper_2010_00704_b200 import synth, workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bk():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2010_00704_b200 import build, binding
    build.build()
    binding.load()
    return binding


ENGINES = ["auto", "lop3", "mma_b1", "tc_i8", "mma_s8", "tc_ws", "tc_pw", "tc_c3", "tc_pn"]


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def guard_alloc(nbytes, dtype=torch.uint8):
    """Device buffer with 256 guard bytes on both sides, filled with 0xA5."""
    raw = torch.full((nbytes + 512,), 0xA5, dtype=torch.uint8, device="cuda")
    return raw, raw[256:256 + nbytes]


def check_guards(raw, nbytes):
    r = raw.cpu().numpy()
    assert np.all(r[:256] == 0xA5) and np.all(r[256 + nbytes:] == 0xA5), "write outside the output buffer"


class Declined(Exception):
    """An explicitly chosen engine returned BCNN_ERR_UNSUPPORTED for the shape or output kind."""


def call_or_skip(bk, engine, fn):
    """An explicitly chosen engine may decline a shape (BCNN_ERR_UNSUPPORTED); "auto" may not."""
    try:
        fn()
    except bk.BcnnError as e:
        if e.status == -2 and engine != "auto":
            raise Declined(engine)
        raise


def skip_if_all_declined(engine, ran):
    if not ran:
        pytest.skip(f"engine {engine} does not take this shape")


def run_conv(bk, x, w, thr, stride, pad, engine):
    """x int8 [B,H,W,Ci] +-1, w int8 [Co,kh,kw,Ci] +-1 -> numpy result (int32 or +-1 int8)."""
    B, H, W, Ci = x.shape
    Co, kh, kw, _ = w.shape
    OH, OW = bk.out_hw(H, W, kh, kw, stride, pad)
    xb, wb = dev(synth.pack_bits(x)), dev(synth.pack_bits(w))
    eng = bk.ENGINES[engine]
    if thr is None:
        n = B * OH * OW * Co * 4
        raw, buf = guard_alloc(n)
        call_or_skip(bk, engine, lambda: bk.bcnn_conv2d_b1(xb, wb, buf, B, H, W, Ci, Co, kh, kw, stride, pad, engine=eng))
        torch.cuda.synchronize()
        check_guards(raw, n)
        return buf.cpu().numpy().view(np.int32).reshape(B, OH, OW, Co)
    n = B * OH * OW * Co // 8
    raw, buf = guard_alloc(n)
    call_or_skip(bk, engine, lambda: bk.bcnn_conv2d_b1_fused(xb, wb, dev(thr), buf, B, H, W, Ci, Co, kh, kw, stride, pad, engine=eng))
    torch.cuda.synchronize()
    check_guards(raw, n)
    return synth.unpack_bits(buf.cpu().numpy().reshape(B, OH, OW, Co // 8))


CONV_SHAPES = [
    # B, H, W, Ci, Co, kh, kw, stride, pad
    (1, 32, 32, 128, 128, 3, 3, 1, 1),     # the single 3x3 workload
    (2, 9, 13, 32, 64, 3, 3, 1, 1),        # ragged M, one-word pixels
    (3, 12, 10, 64, 96, 3, 3, 2, 1),       # stride 2, two-word pixels
    (2, 7, 11, 96, 32, 1, 1, 1, 0),        # 1x1, three-word pixels
    (1, 17, 5, 32, 160, 3, 1, 2, 0),       # kh != kw, ragged N tile
    (2, 6, 9, 160, 224, 1, 3, 1, 2),       # pad larger than needed, wide N
    (1, 40, 40, 256, 256, 3, 3, 2, 1),     # several M and N tiles, K = 2304
    (5, 14, 14, 512, 64, 3, 3, 1, 1),      # K = 4608
    (1, 3, 3, 32, 32, 5, 5, 1, 2),         # kernel larger than the image interior
    (3, 20, 19, 32, 32, 1, 1, 1, 0),       # pointwise layer with one word of K, M % 4 == 0
    (1, 21, 27, 32, 32, 1, 1, 1, 0),       # the same with a tail of three pixels
    (2, 23, 15, 64, 64, 1, 1, 1, 0),       # 1x1 with 64 channels
    (1, 2, 2, 32, 32, 1, 1, 1, 0),         # a single group of four pixels
    (2, 301, 333, 32, 32, 1, 1, 1, 0),     # pointwise engine: several blocks per CTA, ragged last chunk (M = 200466)
    (1, 257, 301, 64, 64, 1, 1, 1, 0),     # ... two words of K, M = 77357 (odd: the last block's bytes are no multiple of 16)
    (1, 129, 203, 128, 128, 1, 1, 1, 0),   # ... four words of K, one tile per chunk
    (1, 97, 101, 96, 96, 1, 1, 1, 0),      # ... three words of K, 96 of 128 accumulator columns used
    (1, 55, 77, 32, 128, 1, 1, 1, 0),      # ... narrow K, wide N
    (1, 66, 51, 128, 32, 1, 1, 1, 0),      # ... wide K, narrow N
    (3, 37, 44, 32, 32, 3, 3, 1, 1),       # halo-tile 3x3 engine: 8 x 16 output tiles, ragged in both directions
    (2, 61, 52, 32, 64, 3, 3, 2, 1),       # ... stride 2, packed 16-bit epilogue with two output words
    (2, 45, 30, 64, 64, 3, 3, 1, 1),       # ... two-word pixels: both producer groups fill every tile
    (1, 70, 66, 64, 32, 3, 3, 2, 0),       # ... stride 2 without padding
    (1, 50, 40, 32, 96, 3, 3, 1, 0),       # ... 96 of 128 accumulator columns, no padding
    (1, 41, 48, 64, 128, 3, 3, 2, 1),      # ... two-word pixels, 128 channels: one accumulator
    (1, 30, 34, 64, 64, 3, 3, 1, 1),       # ... image rows of 68 words: W * C_in / 32 is a multiple of 4, W is not
    (2, 29, 31, 256, 256, 1, 1, 1, 0),     # wide pointwise engine: K = 256, two parts per tile, ragged last tile
    (1, 37, 41, 256, 128, 1, 1, 1, 0),     # ... one part per tile (one of the two issuers idles)
    (1, 23, 19, 256, 512, 1, 1, 1, 0),     # ... four resident slices
    (1, 33, 35, 512, 512, 1, 1, 1, 0),     # ... K = 512: two units per tile, four CTA groups of one slice
    (1, 21, 22, 512, 256, 1, 1, 1, 0),     # ... two CTA groups
    (1, 11, 13, 512, 128, 1, 1, 1, 0),     # ... one group, two parts of 64 channels
]


def plant_extreme_thresholds(thr, K):
    """Thresholds at and beyond the reachable sums, up to the ends of int32 (a batch norm whose scale vanishes
    folds to an unbounded threshold: INT_MAX = the channel never fires, INT_MIN = it always does)."""
    ext = np.array([-2**31, 2**31 - 1, -K - 2, -K - 1, -K, K, K + 1, K + 2, 2**26, -2**26, 2**30, -2**30,
                    2**26 + K, -(2**26) - K, 2**31 - 1 - K, -2**31 + K], dtype=np.int64).astype(np.int32)
    n = min(len(ext), max(1, len(thr) // 2))
    thr[1:2 * n:2] = ext[:n]                      # odd channels (the even ones keep ties / uniform draws)
    return thr


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("shape", CONV_SHAPES)
def test_conv_int32_and_fused(bk, oracle, shape, engine):
    B, H, W, Ci, Co, kh, kw, s, p = shape
    rng = np.random.default_rng(900 + sum(shape))
    x = synth.pm1(rng, (B, H, W, Ci))
    w = synth.pm1(rng, (Co, kh, kw, Ci))
    want = oracle.conv2d(x, w, s, p)
    ran = 0
    try:                                              # (an engine may take one output kind only)
        got = run_conv(bk, x, w, None, s, p, engine)
        assert np.array_equal(got, want)
        ran += 1
    except Declined:
        pass
    K = kh * kw * Ci
    thr = synth.thresholds(rng, K, Co)
    thr[::3] = want.reshape(-1, Co)[0, ::3]           # exact ties on some channels
    try:
        got_bits = run_conv(bk, x, w, thr, s, p, engine)
        assert np.array_equal(got_bits, oracle.threshold(want, thr))
        thr = plant_extreme_thresholds(thr, K)
        got_bits = run_conv(bk, x, w, thr, s, p, engine)
        assert np.array_equal(got_bits, oracle.threshold(want, thr))
        ran += 1
    except Declined:
        pass
    skip_if_all_declined(engine, ran)


@pytest.mark.parametrize("engine", ENGINES)
def test_conv_int32_any_channel_count(bk, oracle, engine):
    # int32 output accepts C_out that is not a multiple of 32 (or even)
    for Co in (1, 7, 30, 33):
        rng = np.random.default_rng(50 + Co)
        x = synth.pm1(rng, (1, 6, 7, 64))
        w = synth.pm1(rng, (Co, 3, 3, 64))
        try:
            assert np.array_equal(run_conv(bk, x, w, None, 1, 1, engine), oracle.conv2d(x, w, 1, 1))
        except Declined:
            pytest.skip(f"engine {engine} has no int32 output")


@pytest.mark.parametrize("engine", ENGINES)
def test_conv_constant_inputs(bk, engine):
    # closed forms straight on the GPU: all -1 activations -> -+K everywhere, borders included
    B, H, W, Ci, Co = 1, 9, 9, 64, 32
    K = 9 * Ci
    xm = -np.ones((B, H, W, Ci), np.int8)
    wp = np.ones((Co, 3, 3, Ci), np.int8)
    if engine in ("tc_pw", "tc_c3", "tc_pn"):
        pytest.skip("the pointwise and halo-tile engines have packed output only")
    assert np.all(run_conv(bk, xm, wp, None, 1, 1, engine) == -K)
    assert np.all(run_conv(bk, xm, -wp, None, 2, 1, engine) == K)
    y = run_conv(bk, -xm, wp, None, 1, 1, engine)[0, :, :, 0]
    assert y[4, 4] == K and y[0, 4] == K - 6 * Ci and y[0, 0] == K - 10 * Ci


@pytest.mark.parametrize("shape", [
    (8, 160, 176, 32, 32, 1, 1),      # 1760 tiles: twelve per CTA - every ring (halo tiles, activation stages, "done" barriers) wraps
    (6, 161, 180, 32, 64, 2, 1),      # stride 2, ragged: 81 x 90 outputs
    (16, 128, 128, 64, 64, 1, 1),     # two-word pixels, 2048 tiles
    (7, 100, 90, 64, 32, 2, 0),       # ... stride 2, no padding (image rows of 180 words)
])
def test_tc_c3_many_tiles_sampled(bk, oracle, shape):
    """The halo-tile 3x3 engine over many tiles per CTA, against the oracle at sampled output pixels (image corners and
    borders, the pixels around tile borders, and random ones) and against the weight-stationary engine everywhere."""
    B, H, W, Ci, Co, s, p = shape
    rng = np.random.default_rng(77 + sum(shape))
    x = synth.pm1(rng, (B, H, W, Ci))
    w = synth.pm1(rng, (Co, 3, 3, Ci))
    K = 9 * Ci
    OH, OW = bk.out_hw(H, W, 3, 3, s, p)
    thr = plant_extreme_thresholds(synth.thresholds(rng, K, Co), K)
    xb, wb, dthr = dev(synth.pack_bits(x)), dev(synth.pack_bits(w)), dev(thr)
    n = B * OH * OW * Co // 8
    raw, buf = guard_alloc(n)
    bk.bcnn_conv2d_b1_fused(xb, wb, dthr, buf, B, H, W, Ci, Co, 3, 3, s, p, engine=bk.ENGINES["tc_c3"])
    torch.cuda.synchronize()
    assert bk.bcnn_device_error() == 0
    check_guards(raw, n)
    got = synth.unpack_bits(buf.cpu().numpy().reshape(B * OH * OW, Co // 8))
    pix = set()
    for b in (0, B // 2, B - 1):
        for oh in (0, 1, 7, 8, 9, OH // 2, OH - 9, OH - 2, OH - 1):
            for ow in (0, 1, 15, 16, 17, OW // 2, OW - 17, OW - 2, OW - 1):
                pix.add((b * OH + oh) * OW + ow)
    pix.update(int(v) for v in rng.integers(0, B * OH * OW, 3000))
    pix = np.array(sorted(pix), dtype=np.int64)
    want = oracle.threshold(oracle.conv2d_pixels(x, w, pix, s, p), thr)
    assert np.array_equal(got[pix], want)
    ref = torch.zeros(n, dtype=torch.uint8, device="cuda")
    bk.bcnn_conv2d_b1_fused(xb, wb, dthr, ref, B, H, W, Ci, Co, 3, 3, s, p, engine=bk.ENGINES["tc_ws"])
    torch.cuda.synchronize()
    assert torch.equal(ref, buf)                       # (the other engine is itself checked against the oracle above)


@pytest.mark.parametrize("shape", [
    (333 * 128 + 77, 512, 512),       # nine and ten row tiles per CTA (four groups of 37): every ring and barrier ring wraps
    (148 * 9 * 128 + 5, 256, 256),    # K = 256: ten tiles per CTA
    (50000, 128, 512),
    (70001, 512, 256),
])
def test_tc_pn_many_tiles_sampled(bk, oracle, shape):
    """The wide pointwise engine over many tiles per CTA, against the oracle on sampled rows (the first and last ones,
    the rows around tile borders, random ones) and against the weight-stationary engine everywhere."""
    M, N, K = shape
    rng = np.random.default_rng(31 + sum(shape))
    Ab = synth.random_bits(rng, (M, K // 8))
    Wb = synth.random_bits(rng, (N, K // 8))
    thr = plant_extreme_thresholds(synth.thresholds(rng, K, N), K)
    dA, dW, dthr = dev(Ab), dev(Wb), dev(thr)
    raw, ob = guard_alloc(M * N // 8)
    bk.bcnn_gemm_b1_fused(dA, dW, dthr, ob, M, N, K, engine=bk.ENGINES["tc_pn"])
    torch.cuda.synchronize()
    assert bk.bcnn_device_error() == 0
    check_guards(raw, M * N // 8)
    got = synth.unpack_bits(ob.cpu().numpy().reshape(M, N // 8))
    rows = {0, 1, 127, 128, 129, M - 130, M - 129, M - 128, M - 2, M - 1}
    rows.update(int(v) for v in rng.integers(0, M, 1500))
    rows = np.array(sorted(rows), dtype=np.int64)
    want = oracle.threshold(oracle.gemm(synth.unpack_bits(Ab[rows]), synth.unpack_bits(Wb)), thr)
    assert np.array_equal(got[rows], want)
    ref = torch.zeros(M * N // 8, dtype=torch.uint8, device="cuda")
    bk.bcnn_gemm_b1_fused(dA, dW, dthr, ref, M, N, K, engine=bk.ENGINES["tc_ws"])
    torch.cuda.synchronize()
    assert torch.equal(ref, ob)                        # (the other engine is itself checked against the oracle above)


GEMM_SHAPES = [(1024, 1024, 512), (1024, 1024, 2304), (300, 200, 96), (129, 33, 1056), (64, 512, 4608), (1, 32, 32),
               (3000, 256, 256), (1, 128, 512), (2049, 512, 256)]


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("shape", GEMM_SHAPES)
def test_gemm_int32_and_fused(bk, oracle, shape, engine):
    M, N, K = shape
    rng = np.random.default_rng(1000 + sum(shape))
    A = synth.pm1(rng, (M, K))
    Wt = synth.pm1(rng, (N, K))
    want = oracle.gemm(A, Wt)
    Ab, Wb = dev(synth.pack_bits(A)), dev(synth.pack_bits(Wt))
    ran = 0
    raw, C = guard_alloc(M * N * 4)
    try:
        call_or_skip(bk, engine, lambda: bk.bcnn_gemm_b1(Ab, Wb, C, M, N, K, engine=bk.ENGINES[engine]))
        torch.cuda.synchronize()
        check_guards(raw, M * N * 4)
        assert np.array_equal(C.cpu().numpy().view(np.int32).reshape(M, N), want)
        ran += 1
    except Declined:
        pass
    if N % 32 == 0:
        thr = synth.thresholds(rng, K, N)
        raw, ob = guard_alloc(M * N // 8)
        try:
            call_or_skip(bk, engine, lambda: bk.bcnn_gemm_b1_fused(Ab, Wb, dev(thr), ob, M, N, K, engine=bk.ENGINES[engine]))
        except Declined:
            skip_if_all_declined(engine, ran)
            return
        torch.cuda.synchronize()
        check_guards(raw, M * N // 8)
        assert np.array_equal(synth.unpack_bits(ob.cpu().numpy().reshape(M, N // 8)), oracle.threshold(want, thr))
        thr = plant_extreme_thresholds(thr, K)
        thr[::4] = want[M // 2, ::4]                    # ties
        raw, ob = guard_alloc(M * N // 8)
        bk.bcnn_gemm_b1_fused(Ab, Wb, dev(thr), ob, M, N, K, engine=bk.ENGINES[engine])
        torch.cuda.synchronize()
        check_guards(raw, M * N // 8)
        assert np.array_equal(synth.unpack_bits(ob.cpu().numpy().reshape(M, N // 8)), oracle.threshold(want, thr))


PACK_SHAPES = [
    # B, H, W, C_in, R, bias
    (2, 5, 7, 32, 1, False), (2, 5, 7, 64, 1, True), (1, 33, 9, 96, 1, True), (3, 8, 8, 4, 8, True),
    (3, 8, 8, 4, 8, False), (1, 4, 5, 8, 4, True), (2, 3, 3, 16, 6, True), (1, 2, 2, 3, 32, True),
    (1, 64, 64, 128, 1, True),
]


@pytest.mark.parametrize("shape", PACK_SHAPES)
def test_pack(bk, oracle, shape):
    B, H, W, Ci, R, has_bias = shape
    rng = np.random.default_rng(300 + sum(shape[:5]))
    x = synth.real_input(rng, (B, H, W, Ci))
    C = Ci * R
    bias = synth.real_input(rng, (C,)) if has_bias else None
    # plant ties and special values
    flat = x.reshape(-1)
    flat[:8] = [0.0, -0.0, np.inf, -np.inf, np.nan, 1e-45, -1e-45, 0.0]
    if has_bias:
        flat[8] = -bias[8 % Ci] if R == 1 else flat[8]
    want = oracle.binarize(x, bias, R)
    n = B * H * W * C // 8
    raw, out = guard_alloc(n)
    bk.bcnn_pack(dev(x), None if bias is None else dev(bias), out, B, H, W, Ci, R)
    torch.cuda.synchronize()
    check_guards(raw, n)
    assert np.array_equal(synth.unpack_bits(out.cpu().numpy().reshape(B, H, W, C // 8)), want)


def test_pack_stem_nonfinite_and_tied_biases(bk, oracle):
    # stem shape (4 real channels x 8): infinite / NaN biases take the per-channel path
    # (inf + -inf = NaN -> -1), equal biases exercise ties in the sorted-threshold path
    rng = np.random.default_rng(4242)
    B, H, W = 2, 9, 11
    x = synth.real_input(rng, (B, H, W, 4))
    x.reshape(-1)[:12] = [0.0, -0.0, np.inf, -np.inf, np.nan, 1e-45, -1e-45, 0.5, -0.5, 1.0, -1.0, 2.0]
    for kind in ("inf", "nan", "ties", "zeros"):
        bias = synth.real_input(rng, (32,))
        if kind == "inf":
            bias[3], bias[10] = np.inf, -np.inf
        elif kind == "nan":
            bias[7] = np.nan
        elif kind == "ties":
            bias[:] = np.repeat(np.array([0.5, -0.5, 0.0, -0.0], np.float32), 8)
            bias[5] = -x.reshape(-1)[21]           # exact tie x + b == 0 on one channel
        else:
            bias[:] = 0.0
        want = oracle.binarize(x, bias, 8)
        out = torch.empty(B * H * W * 4, dtype=torch.uint8, device="cuda")
        bk.bcnn_pack(dev(x), dev(bias), out, B, H, W, 4, 8)
        torch.cuda.synchronize()
        assert np.array_equal(synth.unpack_bits(out.cpu().numpy().reshape(B, H, W, 4)), want), kind


def _stem_want(oracle, x, bias, w, thr):
    """pack (bias, sign, 8x replication) -> binary 1x1 convolution -> threshold, all by the oracle."""
    return oracle.threshold(oracle.conv2d(oracle.binarize(x, bias, 8), w, 1, 0), thr)


def _run_stem(bk, x, bias, w, thr):
    B, H, W, _ = x.shape
    n = B * H * W * 4
    raw, out = guard_alloc(n)
    bk.bcnn_stem_fused(dev(x), None if bias is None else dev(bias), dev(synth.pack_bits(w)), dev(thr), out,
                       B, H, W, 4, 8, 32)
    torch.cuda.synchronize()
    check_guards(raw, n)
    return synth.unpack_bits(out.cpu().numpy().reshape(B, H, W, 4))


@pytest.mark.parametrize("case", ["normal", "no_bias", "ties", "inf_bias", "nan_bias", "extreme_thr", "one_pixel"])
def test_stem_fused(bk, oracle, case):
    # fused pack + first binary 1x1 layer against the oracle's three steps; special inputs, tied and
    # non-finite biases (the plain path), thresholds at and beyond the reachable sums
    rng = np.random.default_rng(9100 + len(case))
    B, H, W = (1, 1, 1) if case == "one_pixel" else (3, 37, 29)      # more pixels than one grid-stride pass of a CTA
    x = synth.real_input(rng, (B, H, W, 4))
    flat = x.reshape(-1)
    if flat.size >= 12:
        flat[:12] = [0.0, -0.0, np.inf, -np.inf, np.nan, 1e-45, -1e-45, 0.5, -0.5, 1.0, -1.0, 2.0]
    bias = synth.real_input(rng, (32,))
    w = synth.pm1(rng, (32, 1, 1, 32))
    thr = synth.thresholds(rng, 32, 32)
    if case == "no_bias":
        bias = None
    elif case == "ties":
        bias[:] = np.repeat(np.array([0.5, -0.5, 0.0, -0.0], np.float32), 8)
        if flat.size > 21:
            bias[5] = -flat[21]                     # exact tie x + b == 0 on one channel
        thr[:] = np.arange(-32, 32, 2, dtype=np.int32)          # every even sum is hit exactly by some output
    elif case == "inf_bias":
        bias[3], bias[10] = np.inf, -np.inf
    elif case == "nan_bias":
        bias[7] = np.nan
    elif case == "extreme_thr":
        thr[:8] = [-2**31, 2**31 - 1, -33, -32, 32, 33, 34, -34]
        thr[8:16] = np.arange(-7, 9, 2)             # odd thresholds: never a tie
    got = _run_stem(bk, x, bias, w, thr)
    assert np.array_equal(got, _stem_want(oracle, x, bias, w, thr)), case
    assert bk.bcnn_device_error() == 0


def test_stem_fused_errors(bk):
    a = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    f = torch.zeros(1024, dtype=torch.float32, device="cuda")
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_stem_fused(f, None, a, a, a, 1, 4, 4, 8, 4, 32)      # not the stem shape
    assert e.value.status == -2
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_stem_fused(f, None, a[4:], a, a, 1, 4, 4, 4, 8, 32)
    assert e.value.status == -3
    with pytest.raises(bk.BcnnError):
        bk.bcnn_stem_fused(f, None, a, None, a, 1, 4, 4, 4, 8, 32)
    torch.cuda.synchronize()
    assert int(a.sum()) == 0


def test_pack_weights_layout(bk, oracle):
    # packing real weights [C_out][kh][kw][C_in] with the same call gives the conv weight layout
    rng = np.random.default_rng(77)
    wr = synth.real_input(rng, (64, 3, 3, 32))
    out = torch.empty(64 * 9 * 32 // 8, dtype=torch.uint8, device="cuda")
    bk.bcnn_pack(dev(wr), None, out, 64, 3, 3, 32, 1)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().reshape(64, 3, 3, 4), synth.pack_bits(oracle.sign_weights(wr)))


def test_errors_launch_nothing(bk):
    a = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_conv2d_b1(a, a, a, 1, 4, 4, 48, 32, 3, 3, 1, 1)
    assert e.value.status == -2
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_gemm_b1(a[4:], a, a, 8, 8, 32)
    assert e.value.status == -3
    with pytest.raises(bk.BcnnError):
        bk.bcnn_gemm_b1_fused(a, a, None, a, 8, 32, 32)
    torch.cuda.synchronize()
    assert int(a.sum()) == 0
    assert bk.bcnn_device_error() == 0


PREPARED_SHAPES = [
    # B, H, W, Ci, Co, kh, kw, stride, pad
    (1, 40, 40, 256, 256, 3, 3, 2, 1),     # several M tiles, K = 2304, one 256-wide tile column
    (5, 14, 14, 512, 64, 3, 3, 1, 1),      # K = 4608, narrow N (128-wide tile, half of it padding)
    (2, 6, 9, 160, 224, 1, 3, 1, 2),       # ragged N, K = 480 (not a multiple of 128), pad 2
    (1, 32, 32, 128, 128, 3, 3, 1, 1),     # the single 3x3 workload
    (2, 9, 13, 32, 64, 3, 3, 1, 1),        # one-word pixels, K = 288
    (1, 17, 5, 32, 160, 3, 1, 2, 0),       # kh != kw
    (3, 7, 11, 96, 32, 1, 1, 1, 0),        # 1x1, K = 96
    (1, 13, 17, 512, 512, 1, 1, 1, 0),     # wide 1x1: two 256-wide tile columns, several M tiles
]


@pytest.mark.parametrize("shape", PREPARED_SHAPES)
def test_conv_prepared_weights(bk, oracle, shape):
    # weights expanded once into a caller-owned buffer, then streamed by TMA: int32 and packed outputs against the
    # oracle, thresholds with ties and out-of-range values, guard bytes around outputs and the prepared buffer
    B, H, W, Ci, Co, kh, kw, s, p = shape
    rng = np.random.default_rng(1900 + sum(shape))
    x = synth.pm1(rng, (B, H, W, Ci))
    w = synth.pm1(rng, (Co, kh, kw, Ci))
    want = oracle.conv2d(x, w, s, p)
    K = kh * kw * Ci
    OH, OW = bk.out_hw(H, W, kh, kw, s, p)
    nbytes = bk.bcnn_prepared_weights_bytes(Co, K)
    assert nbytes >= Co * K
    raw_p, prep = guard_alloc(nbytes)
    assert prep.data_ptr() % 256 == 0
    xb = dev(synth.pack_bits(x))
    bk.bcnn_prepare_weights(dev(synth.pack_bits(w)), prep, Co, K)
    n32 = B * OH * OW * Co * 4
    raw, buf = guard_alloc(n32)
    bk.bcnn_conv2d_b1_prepared(xb, prep, None, buf, B, H, W, Ci, Co, kh, kw, s, p)
    torch.cuda.synchronize()
    check_guards(raw, n32)
    check_guards(raw_p, nbytes)
    assert np.array_equal(buf.cpu().numpy().view(np.int32).reshape(B, OH, OW, Co), want)
    if Co % 32 == 0:
        thr = synth.thresholds(rng, K, Co)
        thr[::3] = want.reshape(-1, Co)[0, ::3]
        thr = plant_extreme_thresholds(thr, K)
        nb = B * OH * OW * Co // 8
        raw, bits = guard_alloc(nb)
        bk.bcnn_conv2d_b1_prepared(xb, prep, dev(thr), bits, B, H, W, Ci, Co, kh, kw, s, p)
        torch.cuda.synchronize()
        check_guards(raw, nb)
        assert np.array_equal(synth.unpack_bits(bits.cpu().numpy().reshape(B, OH, OW, Co // 8)), oracle.threshold(want, thr))
    assert bk.bcnn_device_error() == 0


@pytest.mark.parametrize("shape", [(1024, 1024, 512), (300, 200, 96), (129, 33, 1056), (64, 512, 4608), (1, 32, 32), (2000, 384, 2304)])
def test_gemm_prepared_weights(bk, oracle, shape):
    M, N, K = shape
    rng = np.random.default_rng(2900 + sum(shape))
    A, Wt = synth.pm1(rng, (M, K)), synth.pm1(rng, (N, K))
    want = oracle.gemm(A, Wt)
    prep = torch.empty(bk.bcnn_prepared_weights_bytes(N, K), dtype=torch.uint8, device="cuda")
    bk.bcnn_prepare_weights(dev(synth.pack_bits(Wt)), prep, N, K)
    raw, C = guard_alloc(M * N * 4)
    bk.bcnn_gemm_b1_prepared(dev(synth.pack_bits(A)), prep, None, C, M, N, K)
    torch.cuda.synchronize()
    check_guards(raw, M * N * 4)
    assert np.array_equal(C.cpu().numpy().view(np.int32).reshape(M, N), want)
    if N % 32 == 0:
        thr = plant_extreme_thresholds(synth.thresholds(rng, K, N), K)
        thr[::4] = want[M // 2, ::4]
        raw, ob = guard_alloc(M * N // 8)
        bk.bcnn_gemm_b1_prepared(dev(synth.pack_bits(A)), prep, dev(thr), ob, M, N, K)
        torch.cuda.synchronize()
        check_guards(raw, M * N // 8)
        assert np.array_equal(synth.unpack_bits(ob.cpu().numpy().reshape(M, N // 8)), oracle.threshold(want, thr))
    assert bk.bcnn_device_error() == 0


def test_prepared_errors(bk):
    a = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    assert bk.bcnn_prepared_weights_bytes(64, 48) == 0                 # K not a multiple of 32
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_prepare_weights(a, a[16:], 32, 64)                     # buffer not 256-byte aligned
    assert e.value.status == -3
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_conv2d_b1_prepared(a, a, a, a, 1, 4, 4, 32, 48, 1, 1, 1, 0)   # packed output needs C_out % 32 == 0
    assert e.value.status == -2
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_gemm_b1_prepared(a, None, None, a, 8, 32, 32)
    assert e.value.status == -1
    torch.cuda.synchronize()
    assert int(a.sum()) == 0


def test_bounded_wait_runs_out_and_is_reported(bk, oracle):
    # failure detection without a fault: a wait that nothing satisfies gives up after its poll limit, the kernel
    # frees its tensor memory and ends normally, the error word carries the code until it is read, and the context
    # (tensor memory included: the next tcgen05 kernel allocates all of it) stays usable
    assert bk.bcnn_device_error() == 0
    bk.bcnn_selftest_wait_timeout(256)
    torch.cuda.synchronize()                               # the kernel ended by itself
    st, code = bk.bcnn_device_status()
    assert st == bk.ERR_TIMEOUT and code == bk.SELFTEST_TIMEOUT_CODE
    assert "self-test" in bk.status_string(code)
    assert bk.bcnn_device_status() == (bk.OK, 0)           # reading cleared it
    bk.bcnn_selftest_wait_timeout(1)
    assert bk.bcnn_device_error() == bk.SELFTEST_TIMEOUT_CODE and bk.bcnn_device_error() == 0
    # a normal convolution on both tcgen05 engines right after: bit-exact, no error
    rng = np.random.default_rng(31337)
    x, w = synth.pm1(rng, (2, 12, 12, 64)), synth.pm1(rng, (64, 3, 3, 64))
    want = oracle.conv2d(x, w, 1, 1)
    for engine in ("tc_ws", "tc_i8"):
        assert np.array_equal(run_conv(bk, x, w, None, 1, 1, engine), want)
    assert bk.bcnn_device_error() == 0


MODULE_SHAPES = [
    # B, H, W, Ci, Co, k, stride, pad
    (2, 9, 13, 64, 64, 1, 1, 0),       # weight-stationary engine, the paper's 1x1 module shape
    (1, 20, 20, 128, 128, 1, 1, 0),
    (2, 12, 10, 64, 96, 3, 2, 1),      # 3x3 stride 2, ragged N tile
    (3, 7, 11, 32, 32, 1, 1, 0),       # one-word K: streaming engine
    (1, 14, 14, 256, 256, 1, 1, 0),    # streaming engine, 256-wide tile
    (2, 7, 7, 512, 1024, 1, 1, 0),     # several N tiles
    (1, 10, 10, 128, 320, 3, 1, 1),    # ragged N tile of the streaming engine, K = 1152
]


@pytest.mark.parametrize("variant", ["full", "no_identity", "no_bits", "in_place"])
@pytest.mark.parametrize("shape", MODULE_SHAPES)
def test_conv_module(bk, oracle, shape, variant):
    # binary conv -> batch norm -> + identity -> PReLU -> fp16 map + next signs, bit for bit against the oracle
    B, H, W, Ci, Co, k, stride, pad = shape
    rng = np.random.default_rng(7000 + sum(shape))
    x, w = synth.pm1(rng, (B, H, W, Ci)), synth.pm1(rng, (Co, k, k, Ci))
    K = k * k * Ci
    scale = (rng.standard_normal(Co) / np.sqrt(K)).astype(np.float32)
    scale[::7] *= -1                                       # negative batch-norm scales need no folding here
    shift = rng.standard_normal(Co).astype(np.float32)
    slope = rng.uniform(-0.25, 1.0, Co).astype(np.float32)
    nbias = rng.standard_normal(Co).astype(np.float32)
    OH, OW = bk.out_hw(H, W, k, k, stride, pad)
    ident = rng.standard_normal((B, OH, OW, Co)).astype(np.float16)
    acc = oracle.conv2d(x, w, stride, pad)
    # plant exact zeros and sign ties: channel 0 passes acc through and its next bias cancels a value that occurs
    scale[0], shift[0], slope[0] = 1.0, 0.0, 1.0
    ident[..., 0] = 0
    nbias[0] = -float(acc[0, 0, 0, 0])
    has_id = variant != "no_identity"
    has_bits = variant != "no_bits"
    want_y, want_s = oracle.conv_module(acc, scale, shift, ident if has_id else None, slope, nbias if has_bits else None)
    n = B * OH * OW * Co
    raw_y, ybuf = guard_alloc(2 * n)
    raw_b, bbuf = guard_alloc(n // 8)
    id_dev = None
    if has_id:
        if variant == "in_place":
            ybuf.copy_(dev(ident.view(np.uint8).reshape(-1)))
            id_dev = ybuf
        else:
            id_dev = dev(ident.view(np.uint8).reshape(-1))
    bk.bcnn_conv2d_b1_module(dev(synth.pack_bits(x)), dev(synth.pack_bits(w)), dev(scale), dev(shift), id_dev, dev(slope),
                             dev(nbias) if has_bits else None, ybuf, bbuf if has_bits else None,
                             B, H, W, Ci, Co, k, k, stride, pad)
    torch.cuda.synchronize()
    check_guards(raw_y, 2 * n)
    check_guards(raw_b, n // 8)
    got_y = ybuf.cpu().numpy().view(np.uint16).reshape(B, OH, OW, Co)
    assert np.array_equal(got_y, want_y.view(np.uint16))
    if has_bits:
        assert np.array_equal(synth.unpack_bits(bbuf.cpu().numpy().reshape(B, OH, OW, Co // 8)), want_s)
    assert bk.bcnn_device_error() == 0


def test_conv_module_errors(bk):
    a = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    f = torch.zeros(1024, dtype=torch.float32, device="cuda")
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_conv2d_b1_module(a, a, f, f, None, f, None, a, None, 1, 4, 4, 32, 48, 1, 1, 1, 0)   # C_out % 32 != 0
    assert e.value.status == -2
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_conv2d_b1_module(a, a, None, f, None, f, None, a, None, 1, 4, 4, 32, 32, 1, 1, 1, 0)
    assert e.value.status == -1
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_conv2d_b1_module(a, a, f[1:], f, None, f, None, a, None, 1, 4, 4, 32, 32, 1, 1, 1, 0)
    assert e.value.status == -3
    torch.cuda.synchronize()
    assert int(a.sum()) == 0
