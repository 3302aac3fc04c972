"""GPU: every tensor-core pass must repeat itself bit for bit and finish without a device-side timeout.
The pipelines hand work between asynchronous agents (TMA, several issuing threads, epilogue warps); a missing
ordering shows up as results that differ between identical launches long before it shows up as a parity
failure, so each shape is launched several times and compared with itself."""
import pytest
import torch

import gpu_helpers as G

pytestmark = pytest.mark.gpu

SHAPES = [
    # name, N, C, K, H, R, pad: the VGG-A layer shapes at a reduced minibatch, a 5x5 96->256 layer, FC-like GEMMs
    ("first", 32, 3, 64, 224, 3, 1), ("narrow", 32, 64, 128, 112, 3, 1), ("mid", 32, 128, 256, 56, 3, 1),
    ("wide", 32, 256, 256, 56, 3, 1), ("deep", 64, 512, 512, 14, 3, 1), ("five", 64, 96, 256, 24, 5, 0),
    ("fc_big", 256, 4096, 1000, 1, 1, 0), ("fc_odd", 96, 440, 2048, 1, 1, 0),
]


@pytest.mark.parametrize("name,N,C,K,H,R,pad", SHAPES)
def test_passes_repeat_bit_for_bit(name, N, C, K, H, R, pad):
    from paper_1602_06709_b200 import binding as B
    d = B.conv_desc(N, C, K, H, H, R, R, 1, pad)
    P, Q = B.conv_out_dims(d)
    g = torch.Generator(device="cuda").manual_seed(1602)
    x = torch.rand(N, H, H, C, device="cuda", generator=g)
    w = torch.randn(K, R, R, C, device="cuda", generator=g) * 0.05
    dy = torch.randn(N, P, Q, K, device="cuda", generator=g) * 1e-2
    b = torch.zeros(K, device="cuda")
    ws = torch.empty(max(256, max(B.conv_workspace_bytes(d, i) for i in range(3))), dtype=torch.uint8, device="cuda")
    ref = None
    for _ in range(6):
        y = torch.empty(N, P, Q, K, device="cuda")
        dx = torch.empty_like(x)
        dw = torch.empty_like(w)
        B.conv_fwd(d, x, w, b, y, B.ACT_RELU, ws)
        if C >= 4:
            B.conv_bwd_data(d, dy, w, x, dx, ws)
        B.conv_bwd_weights(d, x, dy, dw, None, True, ws)
        B.check_device_status()
        outs = (y, dx if C >= 4 else None, dw)
        if ref is None:
            ref = outs
        else:
            for a, o in zip(ref, outs):
                assert a is None or torch.equal(a, o)


@pytest.mark.parametrize("name,N,C,K,H", [("first", 32, 3, 64, 224), ("narrow", 32, 64, 128, 112), ("wide", 32, 256, 256, 56)])
def test_forward_with_pool_repeats_bit_for_bit(name, N, C, K, H):
    """conv -> ReLU -> 2x2 pool in one launch, with and without the full-resolution output stored (the first layer
    runs the sixteen-epilogue-warp variant): pooled tensor and position codes identical across launches and
    between the two forms."""
    from paper_1602_06709_b200 import binding as B
    d = B.conv_desc(N, C, K, H, H, 3, 3, 1, 1)
    assert B.conv_fwd_pool_is_fused(d)
    g = torch.Generator(device="cuda").manual_seed(709)
    x = torch.rand(N, H, H, C, device="cuda", generator=g)
    w = torch.randn(K, 3, 3, C, device="cuda", generator=g) * 0.05
    b = torch.randn(K, device="cuda", generator=g) * 0.1
    ws = torch.empty(max(256, B.conv_workspace_bytes(d, B.PASS_FWD)), dtype=torch.uint8, device="cuda")
    ref = None
    for i in range(8):
        yp = G.guarded((N, H // 2, H // 2, K))
        codes = G.guarded((N, H // 2, H // 2, K), torch.uint8, fill=255)
        y = torch.empty(N, H, H, K, device="cuda") if i % 2 else None
        B.conv_fwd_pool(d, x, w, b, y, yp, B.ACT_RELU, ws, pool_codes=codes)
        B.check_device_status()
        if ref is None:
            ref = (yp, codes)
        else:
            assert torch.equal(ref[0], yp) and torch.equal(ref[1], codes)
    assert int(ref[1].max()) <= 7 and not torch.isnan(ref[0]).any()


def test_first_layer_weight_gradient_from_pooled_gradient_repeats_bit_for_bit():
    """The weight-gradient kernel whose epilogue warps build the dy tiles in shared memory (generic-proxy stores handed
    to the tensor core through fence.proxy.async and the slot's barrier): identical results over repeated launches."""
    from paper_1602_06709_b200 import binding as B
    N, C, K, H = 32, 3, 64, 224
    d = B.conv_desc(N, C, K, H, H, 3, 3, 1, 1)
    assert B.conv_bwd_weights_pooled_is_fused(d)
    g = torch.Generator(device="cuda").manual_seed(16)
    x = torch.rand(N, H, H, C, device="cuda", generator=g)
    dyp = torch.randn(N, H // 2, H // 2, K, device="cuda", generator=g) * 1e-2
    codes = torch.randint(0, 8, (N, H // 2, H // 2, K), dtype=torch.uint8, device="cuda", generator=g)
    ws = torch.empty(max(256, B.conv_bwd_weights_pooled_workspace_bytes(d)), dtype=torch.uint8, device="cuda")
    ref = None
    for _ in range(10):
        dw = G.guarded((K, 3, 3, C))
        db = G.guarded((K,))
        B.conv_bwd_weights_pooled(d, x, dyp, codes, True, dw, db, ws)
        B.check_device_status()
        if ref is None:
            ref = (dw, db)
        else:
            assert torch.equal(ref[0], dw) and torch.equal(ref[1], db)
    assert not torch.isnan(ref[0]).any() and not torch.isnan(ref[1]).any()
