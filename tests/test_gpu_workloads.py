"""GPU parity on the benchmark workloads at their full sizes.

Where the definition oracle finishes in seconds it covers every output; above that the
oracle covers sampled rows / the first images of the batch (images are independent), and
the bit-packed CPU checker (proven equal to the oracle in the CPU tests) covers all outputs.
"""
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


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def test_single_3x3_workload(bk, oracle):
    l = wl.SINGLE_3X3
    rng = synth.rng_for(1)
    x = synth.pm1(rng, (1, l.H, l.W, l.C_in))
    w = synth.pm1(rng, (l.C_out, 3, 3, l.C_in))
    y = torch.empty(l.M(1) * l.C_out, dtype=torch.int32, device="cuda")
    bk.bcnn_conv2d_b1(dev(synth.pack_bits(x)), dev(synth.pack_bits(w)), y, 1, l.H, l.W, l.C_in, l.C_out, 3, 3, 1, 1)
    assert np.array_equal(y.cpu().numpy().reshape(1, 32, 32, 128), oracle.conv2d(x, w, 1, 1))


@pytest.mark.parametrize("MN", wl.GEMM_SWEEP_MN)
@pytest.mark.parametrize("K", wl.GEMM_SWEEP_K)
def test_gemm_sweep(bk, oracle, MN, K):
    M = N = MN
    rng = synth.rng_for(2, MN + K)
    Ab = synth.random_bits(rng, (M, K // 8))
    Wb = synth.random_bits(rng, (N, K // 8))
    thr = synth.thresholds(rng, K, N)
    dA, dW = dev(Ab), dev(Wb)
    C = torch.empty(M * N, dtype=torch.int32, device="cuda")
    bits = torch.empty(M * N // 8, dtype=torch.uint8, device="cuda")
    bk.bcnn_gemm_b1(dA, dW, C, M, N, K)
    bk.bcnn_gemm_b1_fused(dA, dW, dev(thr), bits, M, N, K)
    got = C.cpu().numpy().reshape(M, N)
    got_bits = bits.cpu().numpy().reshape(M, N // 8)
    # definition oracle: all rows at M = 1024, else sampled rows (tile edges + random)
    if M <= 1024:
        rows = np.arange(M)
    else:
        edge = np.array([0, 1, 127, 128, 129, 255, 256, M // 2 - 1, M // 2, M - 129, M - 128, M - 1])
        rows = np.unique(np.concatenate([edge, rng.choice(M, size=36, replace=False)]))
    Wpm = synth.unpack_bits(Wb)
    want = oracle.gemm(synth.unpack_bits(Ab[rows]), Wpm)
    assert np.array_equal(got[rows], want)
    assert np.array_equal(synth.unpack_bits(got_bits[rows]), oracle.threshold(want, thr))
    # every output: packed checker
    full = oracle.checker_gemm(Ab, Wb, M, N, K)
    assert np.array_equal(got, full)
    assert np.array_equal(got_bits, synth.pack_bits(np.where(full >= thr[None, :], 1, -1).astype(np.int8)))


def _chain_inputs(config, layers, B):
    rng = synth.rng_for(config)
    l0 = layers[0]
    x_bits = synth.random_bits(rng, (B, l0.H, l0.W, l0.C_in // 8))
    ws = [synth.random_bits(synth.rng_for(config, i + 1), (l.C_out, l.k, l.k, l.C_in // 8)) for i, l in enumerate(layers)]
    ts = [synth.thresholds(synth.rng_for(config, 100 + i), l.K, l.C_out) for i, l in enumerate(layers)]
    return x_bits, ws, ts


def _check_chain(bk, oracle, config, layers, B, b_oracle):
    from paper_2010_00704_b200.chain import FusedChain
    x_bits, ws, ts = _chain_inputs(config, layers, B)
    ch = FusedChain(layers, B, ws, ts, keep_all=True)
    ch.in_bits.copy_(dev(x_bits).reshape(-1))
    ch.run()
    torch.cuda.synchronize()
    outs = [o.cpu().numpy() for o in ch.outs]
    # (i) definition oracle, from scratch, on the first b_oracle images
    cur = synth.unpack_bits(x_bits[:b_oracle])
    for l, w, t, o in zip(layers, ws, ts, outs):
        acc = oracle.conv2d(cur, synth.unpack_bits(w), l.stride, l.pad)
        cur = oracle.threshold(acc, t)
        got = synth.unpack_bits(o.reshape(B, l.OH, l.OW, l.C_out // 8)[:b_oracle])
        assert np.array_equal(got, cur), l.name
    # (ii) every output of every layer: packed checker, each layer fed the GPU's (checked) input
    cur_bits = x_bits
    for l, w, t, o in zip(layers, ws, ts, outs):
        acc = oracle.checker_conv2d(cur_bits, w, (B, l.H, l.W, l.C_in, l.C_out, l.k, l.k), l.stride, l.pad)
        want = synth.pack_bits(np.where(acc >= t, 1, -1).astype(np.int8))
        got = o.reshape(B, l.OH, l.OW, l.C_out // 8)
        assert np.array_equal(got, want), l.name
        cur_bits = got


def test_stem_downsample_layers(bk, oracle):
    # two independent layers, each in full against the definition oracle
    B = wl.STEM_DOWN_BATCH
    for i, l in enumerate(wl.STEM_DOWN):
        rng = synth.rng_for(3, i)
        x = synth.pm1(rng, (B, l.H, l.W, l.C_in))
        w = synth.pm1(rng, (l.C_out, 3, 3, l.C_in))
        thr = synth.thresholds(rng, l.K, l.C_out)
        out = torch.empty(l.out_bits_bytes(B), dtype=torch.uint8, device="cuda")
        bk.bcnn_conv2d_b1_fused(dev(synth.pack_bits(x)), dev(synth.pack_bits(w)), dev(thr), out,
                                B, l.H, l.W, l.C_in, l.C_out, 3, 3, l.stride, l.pad)
        want = oracle.threshold(oracle.conv2d(x, w, l.stride, l.pad), thr)
        assert np.array_equal(synth.unpack_bits(out.cpu().numpy().reshape(B, l.OH, l.OW, l.C_out // 8)), want)


def test_block_stack_chain(bk, oracle):
    _check_chain(bk, oracle, 4, wl.BLOCK_STACK, wl.BLOCK_STACK_BATCH, b_oracle=4)


def test_backbone18_chain(bk, oracle):
    _check_chain(bk, oracle, 5, wl.BACKBONE18, wl.BACKBONE18_BATCH, b_oracle=2)


def test_backbone18_with_pack_stage_and_graph(bk, oracle):
    # fp32 input -> pack (bias + sign, 4 channels replicated 8x) -> 18 fused layers, replayed from a CUDA graph
    from paper_2010_00704_b200.chain import FusedChain
    B = 8
    layers = wl.BACKBONE18
    H, W, C, R = wl.BACKBONE18_INPUT
    rng = synth.rng_for(5, 999)
    x = synth.real_input(rng, (B, H, W, C))
    bias = synth.real_input(rng, (C * R,))
    _, ws, ts = _chain_inputs(5, layers, 1)
    ch = FusedChain(layers, B, ws, ts, real_input_shape=(H, W, C), bias=bias, replicate=R)
    ch.x_real.copy_(dev(x).reshape(-1))
    ch.capture()
    for _ in range(2):
        ch.run()
    torch.cuda.synchronize()
    got = synth.unpack_bits(ch.outs[-1].cpu().numpy().reshape(B, 7, 7, 512 // 8))
    b = 2
    cur = oracle.binarize(x[:b], bias, R)
    for l, w, t in zip(layers, ws, ts):
        cur = oracle.threshold(oracle.conv2d(cur, synth.unpack_bits(w), l.stride, l.pad), t)
    assert np.array_equal(got[:b], cur)
    assert bk.bcnn_device_error() == 0


def test_backbone18_stem_fused_full_batch(bk, oracle):
    # the fused stem (pack + L1) at the benchmark's size, batch 256: the oracle's three steps on 300000
    # sampled pixels plus the first and last 4096 (a 1x1 layer: every pixel is independent)
    B = wl.BACKBONE18_BATCH
    H, W, C, R = wl.BACKBONE18_INPUT
    rng = synth.rng_for(5, 4321)
    x = synth.real_input(rng, (B, H, W, C))
    bias = synth.real_input(rng, (C * R,))
    _, ws, ts = _chain_inputs(5, wl.BACKBONE18[:1], 1)
    out = torch.empty(B * H * W * 4, dtype=torch.uint8, device="cuda")
    bk.bcnn_stem_fused(dev(x), dev(bias), dev(ws[0]), dev(ts[0]), out, B, H, W, C, R, 32)
    torch.cuda.synchronize()
    got = out.cpu().numpy().reshape(-1, 4)
    npix = B * H * W
    idx = np.unique(np.concatenate([np.arange(4096), np.arange(npix - 4096, npix), rng.integers(0, npix, 300000)]))
    xs = x.reshape(-1, C)[idx].reshape(1, -1, 1, C)
    want = oracle.threshold(oracle.conv2d(oracle.binarize(xs, bias, R), synth.unpack_bits(ws[0]), 1, 0), ts[0])
    assert np.array_equal(synth.unpack_bits(got[idx]), want.reshape(-1, 32))
    assert bk.bcnn_device_error() == 0


def test_backbone18_from_host_pipeline(bk, oracle):
    # the host-input entry of the chain: three different inputs in a row through the double-buffered
    # copy stream; every result must be the one of its own input (checked against the oracle)
    from paper_2010_00704_b200.chain import FusedChain
    B = 4
    layers = wl.BACKBONE18
    H, W, C, R = wl.BACKBONE18_INPUT
    rng = synth.rng_for(5, 1234)
    bias = synth.real_input(rng, (C * R,))
    _, ws, ts = _chain_inputs(5, layers, 1)
    ch = FusedChain(layers, B, ws, ts, real_input_shape=(H, W, C), bias=bias, replicate=R)
    ch.capture()
    xs = [synth.real_input(rng, (B, H, W, C)) for _ in range(3)]
    x_hosts = [torch.from_numpy(x.reshape(-1)).pin_memory() for x in xs]
    out_hosts = [torch.empty(ch.outs[-1].numel(), dtype=torch.uint8).pin_memory() for _ in xs]
    for xh, oh in zip(x_hosts, out_hosts):
        ch.run_from_host(xh, oh)
    torch.cuda.synchronize()
    for x, oh in zip(xs, out_hosts):
        cur = oracle.binarize(x[:1], bias, R)
        for l, w, t in zip(layers, ws, ts):
            cur = oracle.threshold(oracle.conv2d(cur, synth.unpack_bits(w), l.stride, l.pad), t)
        got = synth.unpack_bits(oh.numpy().reshape(B, 7, 7, 512 // 8))
        assert np.array_equal(got[:1], cur)
    assert bk.bcnn_device_error() == 0


@pytest.mark.parametrize("li", range(14))
def test_paper_1x1_convs(bk, oracle, li):
    # every distinct binary 1x1 convolution of the paper's own network (Table 1) at batch 4, fused and int32:
    # the definition oracle on 512 sampled pixels plus the first and last 128, the packed checker on every output
    l, _count = wl.paper_binary_1x1_convs(1)[li]
    B = 4
    rng = synth.rng_for(6, li)
    xb = synth.random_bits(rng, (B, l.H, l.W, l.C_in // 8))
    wb = synth.random_bits(rng, (l.C_out, 1, 1, l.C_in // 8))
    thr = synth.thresholds(rng, l.K, l.C_out)
    M, N = l.M(B), l.C_out
    y = torch.empty(M * N, dtype=torch.int32, device="cuda")
    yb = torch.empty(M * N // 8, dtype=torch.uint8, device="cuda")
    bk.bcnn_conv2d_b1(dev(xb), dev(wb), y, B, l.H, l.W, l.C_in, N, 1, 1, 1, 0)
    bk.bcnn_conv2d_b1_fused(dev(xb), dev(wb), dev(thr), yb, B, l.H, l.W, l.C_in, N, 1, 1, 1, 0)
    torch.cuda.synchronize()
    got = y.cpu().numpy().reshape(M, N)
    got_bits = yb.cpu().numpy().reshape(M, N // 8)
    full = oracle.checker_conv2d(xb, wb, (B, l.H, l.W, l.C_in, N, 1, 1), 1, 0).reshape(M, N)
    assert np.array_equal(got, full)
    assert np.array_equal(got_bits, synth.pack_bits(np.where(full >= thr[None, :], 1, -1).astype(np.int8)))
    rows = np.unique(np.concatenate([np.arange(min(128, M)), np.arange(max(0, M - 128), M), rng.integers(0, M, 512)]))
    xs = synth.unpack_bits(xb.reshape(M, l.C_in // 8)[rows]).reshape(1, -1, 1, l.C_in)
    want = oracle.conv2d(xs, synth.unpack_bits(wb), 1, 0).reshape(-1, N)
    assert np.array_equal(got[rows], want)
    assert np.array_equal(synth.unpack_bits(got_bits[rows]), oracle.threshold(want, thr))
    assert bk.bcnn_device_error() == 0
