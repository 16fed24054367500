"""The entry point that allocates nothing (bcnn_conv2d_b1_fused_noalloc), through the C ABI.

Some callers of the library cannot allocate device memory where they call it - they run inside a memory plan they do
not own, or at a point where an allocation is forbidden - so this call keeps its scratch (the layer's prepared weights)
in a static array inside the library.  The array is shared by all calls and keeps whatever the last call left there;
the test therefore makes two calls in a row with different layers and checks each against the ordinary entry point,
bit for bit (the tolerance of every packed-output test here).  Collected last on purpose: a failure here must not
keep the other tests from running under `pytest -x`."""
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


def _layer(rng, B, H, W, Ci, Co, k, stride, pad):
    x = synth.random_bits(rng, (B * H * W * Ci // 8,))
    w = synth.random_bits(rng, (Co * k * k * Ci // 8,))
    thr = synth.thresholds(rng, k * k * Ci, Co)
    thr[3], thr[10], thr[17] = 2**31 - 1, -2**31, 0          # a channel that never fires, one that always does, a tie-prone one
    return dev(x), dev(w), dev(thr)


def test_noalloc_matches_the_ordinary_call_twice_in_a_row(bk):
    rng = np.random.default_rng(424242)
    # the second layer is smaller in every dimension than the first: whatever the first call left in the static
    # array beyond the second layer's own prepared weights must not matter
    layers = [(2, 14, 14, 256, 512, 3, 1, 1), (3, 9, 11, 64, 96, 3, 2, 1)]
    for (B, H, W, Ci, Co, k, s, p) in layers:
        x, w, thr = _layer(rng, B, H, W, Ci, Co, k, s, p)
        OH, OW = bk.out_hw(H, W, k, k, s, p)
        n = B * OH * OW * Co // 8
        want = torch.empty(n, dtype=torch.uint8, device="cuda")
        bk.bcnn_conv2d_b1_fused(x, w, thr, want, B, H, W, Ci, Co, k, k, s, p)
        raw = torch.full((n + 512,), 0xA5, dtype=torch.uint8, device="cuda")
        got = raw[256:256 + n]
        assert bk.bcnn_prepared_weights_bytes(Co, k * k * Ci) <= bk.STATIC_SCRATCH_BYTES
        bk.bcnn_conv2d_b1_fused_noalloc(x, w, thr, got, B, H, W, Ci, Co, k, k, s, p)
        torch.cuda.synchronize()
        r = raw.cpu().numpy()
        assert np.all(r[:256] == 0xA5) and np.all(r[256 + n:] == 0xA5), "write outside the output buffer"
        assert torch.equal(got, want)
    assert bk.bcnn_device_error() == 0


def test_noalloc_rejects_layers_beyond_its_array(bk):
    a = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    # 1024 output channels x 9216 bits: 9 MiB of prepared weights, more than the 4 MiB array
    assert bk.bcnn_prepared_weights_bytes(1024, 9216) > bk.STATIC_SCRATCH_BYTES
    with pytest.raises(bk.BcnnError) as e:
        bk.bcnn_conv2d_b1_fused_noalloc(a, a, a, a, 1, 4, 4, 1024, 1024, 3, 3, 1, 1)
    assert e.value.status == bk.ERR_WORKSPACE
    assert "scratch" in bk.status_string(bk.ERR_WORKSPACE)
    with pytest.raises(bk.BcnnError):
        bk.bcnn_conv2d_b1_fused_noalloc(a, a, None, a, 1, 4, 4, 32, 32, 3, 3, 1, 1)
    torch.cuda.synchronize()
    assert int(a.sum()) == 0
