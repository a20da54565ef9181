"""Parity of the fp32 interface (sdwino_filter_transform_f32 / sdwino_conv3x3_f32) with the fp64 oracle.

Bar: max|gpu - ref| <= 1e-2 * max|ref| per layer, ref = fp64 direct convolution of the fp32 inputs; the
operands of the contraction are rounded to fp16 (the significand of TF32), accumulation and output are fp32.
On inputs that fp16 represents exactly the fp32 calls must reproduce the fp16 calls bit for bit once their
output is rounded to fp16: both interfaces share every arithmetic step between the loads and the stores.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_05781_b200 import workloads
from paper_2412_05781_b200.workloads import ConvLayer

pytestmark = pytest.mark.gpu

TOL = 1e-2
TOL_F2_REGRESSION = 2.5e-3
F4_POINTS = (0, 0.75, -0.75, 1.5, -1.5)


@pytest.fixture(scope="module")
def B():
    from paper_2412_05781_b200 import build_library
    build_library()
    from paper_2412_05781_b200 import binding
    assert torch.cuda.is_available()
    return binding


def _run32(B, layer, tile, x, w, b, ws_bytes=None):
    wT = B.sdwino_filter_transform_f32(w.cuda(), tile)
    if ws_bytes is None:
        ws_bytes = B.sdwino_workspace_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, tile)
    ws = B.alloc_workspace(ws_bytes)
    y = B.sdwino_conv3x3_f32(x.cuda(), wT, None if b is None else b.cuda(), layer.K, tile, workspace=ws)
    assert B.sdwino_last_device_status() == B.OK
    assert y.dtype == torch.float32
    return y.cpu()


def _rel_err(y, ref):
    return float(np.abs(y.double().numpy() - ref).max() / np.abs(ref).max())


SHAPES = [
    # C, K, H, W, N: scalar kernels (odd widths), vector kernels (W % 8 == 0), few channels, ragged everything
    (1, 1, 4, 4, 1), (3, 4, 5, 7, 2), (7, 33, 2, 9, 1), (33, 3, 13, 1, 2), (4, 40, 16, 16, 1), (40, 4, 24, 32, 2),
    (64, 128, 16, 16, 1), (65, 129, 17, 19, 1), (96, 160, 18, 24, 2), (130, 257, 33, 40, 1), (16, 16, 40, 56, 3),
    (72, 200, 50, 48, 2),
]


@pytest.mark.parametrize("tile", [2, 4])
@pytest.mark.parametrize("shape", SHAPES)
def test_fp32_interface_elementwise(B, shape, tile):
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=sum(shape), dtype=torch.float32)
    assert x.dtype == torch.float32 and not torch.equal(x, x.half().float())   # values fp16 cannot hold
    y = _run32(B, layer, tile, x, w, b)
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    err = _rel_err(y, ref)
    assert err <= (TOL_F2_REGRESSION if tile == 2 else TOL), err
    # the edge tiles alone (padding and tile-index logic)
    m = tile
    TH, TW = -(-H // m), -(-W // m)
    mask = np.zeros((H, W), dtype=bool)
    mask[:m, :] = mask[:, :m] = True
    mask[(TH - 1) * m:, :] = mask[:, (TW - 1) * m:] = True
    assert np.abs(y.double().numpy() - ref)[:, :, mask].max() <= TOL * np.abs(ref).max()
    # and the three-step fp64 Winograd route with the same interpolation points
    wino = oracle.winograd_conv3x3(x.numpy(), w.numpy(), b.numpy(), m=tile, points=None if tile == 2 else F4_POINTS)
    assert _rel_err(y, wino) <= TOL


@pytest.mark.parametrize("tile", [2, 4])
@pytest.mark.parametrize("shape", [(32, 48, 16, 16, 2), (20, 24, 9, 11, 1), (64, 48, 64, 64, 2), (24, 32, 100, 64, 1)])
def test_fp32_interface_reproduces_fp16_interface_on_fp16_values(B, shape, tile):
    # more than 8 channels on both sides: the fp16 call takes the same three kernels (its single-kernel paths
    # for very few channels keep V unrounded and differ in the last bits)
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=11 + C)
    wT16 = B.sdwino_filter_transform(w.cuda(), tile)
    wT32 = B.sdwino_filter_transform_f32(w.float().cuda(), tile)
    a, Kb, Cb = tile + 2, -(-K // 16), -(-C // 64)
    payload = a * a * Kb * Cb * 1024 * 2               # U[a*a][Cb][Kb][16][64] fp16 behind the 1 KB header
    assert torch.equal(wT16[:16], wT32[:16])           # magic, K, C, tile
    assert torch.equal(wT16[1024:1024 + payload], wT32[1024:1024 + payload])   # every transformed filter value
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(N, C, H, W, K, tile))
    y16 = B.sdwino_conv3x3(x.cuda(), wT16, b.cuda(), K, tile, workspace=ws).cpu()
    y32 = B.sdwino_conv3x3_f32(x.float().cuda(), wT16, b.float().cuda(), K, tile, workspace=ws).cpu()
    assert B.sdwino_last_device_status() == B.OK
    assert torch.equal(y32.half(), y16)
    # the fp32 result is the unrounded one: closer to the oracle than (or as close as) its fp16 rounding
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    assert _rel_err(y32, ref) <= _rel_err(y16, ref) + 1e-4


@pytest.mark.parametrize("tile", [2, 4])
@pytest.mark.parametrize("KC", [(320, 320), (3, 128), (130, 7)])
def test_fp32_filter_transform_matches_oracle(B, KC, tile):
    K, C = KC
    a = tile + 2
    g = torch.Generator().manual_seed(K + C)
    w = torch.randn(K, C, 3, 3, generator=g) / (9 * C) ** 0.5
    wT = B.sdwino_filter_transform_f32(w.cuda(), tile)
    Kb, Cb = -(-K // 16), -(-C // 64)
    assert wT[:16].view(torch.int32).cpu().tolist() == [0x55574453, K, C, tile]
    U = wT[1024:].view(torch.float16)[:a * a * Kb * Cb * 1024].view(a * a, Cb, Kb, 16, 64).permute(0, 2, 3, 1, 4)
    U = U.reshape(a * a, Kb * 16, Cb * 64).cpu()
    Uo = oracle.filter_transform(w.numpy(), tile, points=None if tile == 2 else F4_POINTS)
    Uo = torch.from_numpy(Uo.reshape(K, C, a * a).transpose(2, 0, 1).copy())
    ref16 = Uo.half()
    ulp = torch.maximum((torch.nextafter(ref16, torch.full_like(ref16, float("inf"))) - ref16).double().abs(),
                        (ref16 - torch.nextafter(ref16, torch.full_like(ref16, -float("inf")))).double().abs())
    assert bool(((U[:, :K, :C].double() - ref16.double()).abs() <= ulp).all())
    assert float(U[:, :, C:].abs().max() if Cb * 64 > C else 0) == 0
    assert float(U[:, K:, :].abs().max() if Kb * 16 > K else 0) == 0


@pytest.mark.parametrize("tile", [2, 4])
def test_fp32_interface_several_passes_no_bias_and_delta_filter(B, tile):
    layer = ConvLayer(C=24, K=32, H=96, W=64, N=2)
    x, w, _ = workloads.make_inputs(layer, seed=3, with_bias=False, dtype=torch.float32)
    full = _run32(B, layer, tile, x, w, None)
    # a workspace of a quarter of the layer: four passes, the same bits
    small = B.sdwino_workspace_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, tile) // 4
    small = max(small, B.sdwino_workspace_min_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, tile))
    assert torch.equal(_run32(B, layer, tile, x, w, None, ws_bytes=small), full)
    assert _rel_err(full, oracle.direct_conv3x3(x.numpy(), w.numpy(), None)) <= TOL
    # a filter that is 1 at the centre tap of channel k = c copies x up to the fp16 rounding of V and M
    C = 16
    lay = ConvLayer(C=C, K=C, H=21, W=24, N=1)
    xd, _, _ = workloads.make_inputs(lay, seed=8, dtype=torch.float32)
    wd = torch.zeros(C, C, 3, 3)
    for k in range(C):
        wd[k, k, 1, 1] = 1.0
    yd = _run32(B, lay, tile, xd, wd, None)
    assert float((yd - xd).abs().max()) <= TOL * float(xd.abs().max())


def test_fp32_interface_argument_errors(B):
    layer = ConvLayer(C=16, K=16, H=8, W=8, N=1)
    x, w, b = workloads.make_inputs(layer, seed=1, dtype=torch.float32)
    lib = B.lib
    wT = B.sdwino_filter_transform_f32(w.cuda(), 2)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(1, 16, 8, 8, 16, 2))
    xd, bd = x.cuda(), b.cuda()
    y = torch.empty(1, 16, 8, 8, device="cuda")
    nb = ws.numel()
    call = lambda xp, wp, bp, yp, tile=2, wsp=ws.data_ptr(), n=nb: lib.sdwino_conv3x3_f32(  # noqa: E731
        xp, wp, bp, yp, 1, 16, 8, 8, 16, tile, wsp, n, None)
    assert call(xd.data_ptr(), wT.data_ptr(), bd.data_ptr(), y.data_ptr()) == B.OK
    assert call(None, wT.data_ptr(), bd.data_ptr(), y.data_ptr()) == B.ERR_INVALID_ARG
    assert call(xd.data_ptr(), wT.data_ptr(), bd.data_ptr(), None) == B.ERR_INVALID_ARG
    assert call(xd.data_ptr() + 2, wT.data_ptr(), bd.data_ptr(), y.data_ptr()) == B.ERR_MISALIGNED
    assert call(xd.data_ptr(), wT.data_ptr(), bd.data_ptr() + 2, y.data_ptr()) == B.ERR_MISALIGNED
    assert call(xd.data_ptr(), wT.data_ptr(), bd.data_ptr(), y.data_ptr(), tile=3) == B.ERR_UNSUPPORTED
    assert call(xd.data_ptr(), wT.data_ptr(), bd.data_ptr(), y.data_ptr(), wsp=None, n=0) == B.ERR_WORKSPACE
    assert lib.sdwino_filter_transform_f32(None, wT.data_ptr(), 16, 16, 2, None) == B.ERR_INVALID_ARG
    assert lib.sdwino_filter_transform_f32(w.cuda().data_ptr(), wT.data_ptr(), 16, 16, 6, None) == B.ERR_UNSUPPORTED
    torch.cuda.synchronize()
    # a 4-byte aligned but not 16-byte aligned x takes the scalar kernel: same result
    buf = torch.empty(x.numel() + 1, device="cuda")
    buf[1:].copy_(xd.flatten())
    y2 = torch.empty_like(y)
    assert call(buf[1:].data_ptr(), wT.data_ptr(), bd.data_ptr(), y2.data_ptr()) == B.OK
    torch.cuda.synchronize()
    assert B.sdwino_last_device_status() == B.OK
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    assert _rel_err(y2.cpu(), ref) <= TOL_F2_REGRESSION and _rel_err(y.cpu(), ref) <= TOL_F2_REGRESSION


@pytest.mark.parametrize("idx", [1, 5, 7, 12])
def test_fp32_interface_sd15_layers_sampled_channels(B, idx):
    layer = workloads.sd15_unet()[idx]
    tile = B.sdwino_choose_tile(layer.N, layer.C, layer.H, layer.W, layer.K)
    x, w, b = workloads.make_inputs(layer, seed=idx, dtype=torch.float32)
    y = _run32(B, layer, tile, x, w, b)
    rng = np.random.default_rng(idx)
    ks = np.sort(rng.choice(layer.K, size=16, replace=False))
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy()[ks], b.numpy()[ks])
    got = y[:, ks].double().numpy()
    assert np.abs(got - ref).max() <= TOL * np.abs(ref).max()


@pytest.mark.parametrize("shape", [(48, 3, 16, 16, 2), (128, 3, 64, 64, 1), (20, 8, 24, 40, 3), (70, 5, 40, 24, 2)])
def test_fp32_interface_few_output_channels_fused_kernel(B, shape):
    # F(2x2) layers with at most 8 output channels take the single tcgen05 kernel (one launch, no workspace
    # traffic); it rounds the fp32 pixels to fp16 as it loads them.  Same result as the three-kernel path.
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=sum(shape), dtype=torch.float32)
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    B.sdwino_set_fused_min_tiles(1)
    try:
        n0 = B.sdwino_launch_count()
        y = _run32(B, layer, 2, x, w, b)
        assert B.sdwino_launch_count() - n0 == 2          # filter transform + the fused kernel
    finally:
        B.sdwino_set_fused_min_tiles(0)
    assert _rel_err(y, ref) <= TOL_F2_REGRESSION
    B.sdwino_set_gemm_shape(1, 16)                         # forcing a GEMM shape takes the three kernels
    try:
        n0 = B.sdwino_launch_count()
        y3 = _run32(B, layer, 2, x, w, b)
        assert B.sdwino_launch_count() - n0 == 4
    finally:
        B.sdwino_set_gemm_shape(0, 0)
    assert _rel_err(y3, ref) <= TOL_F2_REGRESSION
    assert float((y - y3).abs().max()) <= 2 * TOL_F2_REGRESSION * float(np.abs(ref).max())
    # an 8-byte aligned y is needed for the fused kernel's stores; a 4-byte aligned one takes the three kernels
    buf = torch.empty(N * K * H * W + 1, device="cuda")
    yv = buf[1:].view(N, K, H, W)
    wT = B.sdwino_filter_transform_f32(w.cuda(), 2)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(N, C, H, W, K, 2))
    xd, bd = x.cuda(), b.cuda()
    rc = B.lib.sdwino_conv3x3_f32(xd.data_ptr(), wT.data_ptr(), bd.data_ptr(), yv.data_ptr(), N, C, H, W, K, 2,
                                  ws.data_ptr(), ws.numel(), None)
    assert rc == B.OK and B.sdwino_last_device_status() == B.OK
    assert _rel_err(yv.cpu(), ref) <= TOL_F2_REGRESSION


@pytest.mark.parametrize("shape", [(4, 40, 16, 16, 2), (3, 17, 21, 26, 2), (8, 8, 9, 11, 1), (1, 5, 13, 2, 3), (4, 320, 64, 64, 2)])
def test_fp32_interface_few_input_channels_fused_kernel(B, shape):
    # F(2x2) layers with at most 8 input channels take the single warp-MMA kernel: one launch, same result as the
    # three kernels; widths that are multiples of 4 (16-byte stores), even (8-byte) and odd (4-byte)
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=sum(shape), dtype=torch.float32)
    ks = list(range(K)) if K <= 64 else sorted(np.random.default_rng(0).choice(K, 16, replace=False).tolist())
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy()[ks], b.numpy()[ks])
    n0 = B.sdwino_launch_count()
    y = _run32(B, layer, 2, x, w, b)
    assert B.sdwino_launch_count() - n0 == 2              # filter transform + the fused kernel
    assert _rel_err(y[:, ks], ref) <= TOL_F2_REGRESSION
    B.sdwino_set_gemm_shape(1, 16)
    try:
        y3 = _run32(B, layer, 2, x, w, b)
    finally:
        B.sdwino_set_gemm_shape(0, 0)
    assert _rel_err(y3[:, ks], ref) <= TOL_F2_REGRESSION
    assert float((y - y3).abs().max()) <= 2 * TOL_F2_REGRESSION * float(np.abs(ref).max())
    # y 4-byte aligned only: the scalar stores
    buf = torch.empty(N * K * H * W + 1, device="cuda")
    yv = buf[1:].view(N, K, H, W)
    wT = B.sdwino_filter_transform_f32(w.cuda(), 2)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(N, C, H, W, K, 2))
    xd, bd = x.cuda(), b.cuda()
    rc = B.lib.sdwino_conv3x3_f32(xd.data_ptr(), wT.data_ptr(), bd.data_ptr(), yv.data_ptr(), N, C, H, W, K, 2,
                                  ws.data_ptr(), ws.numel(), None)
    assert rc == B.OK and B.sdwino_last_device_status() == B.OK
    assert torch.equal(yv.cpu(), y)


@pytest.mark.parametrize("act", ["none", "silu"])
@pytest.mark.parametrize("shape,tile", [((32, 48, 16, 16, 2), 2), ((32, 48, 16, 16, 2), 4), ((20, 24, 9, 11, 1), 2),
                                        ((20, 24, 9, 11, 1), 4), ((4, 40, 12, 16, 1), 2), ((40, 4, 12, 16, 2), 2),
                                        ((64, 64, 64, 64, 1), 4), ((17, 33, 13, 24, 3), 4)])
def test_fp32_interface_fused_residual_and_activation(B, shape, tile, act):
    # y = act(conv + bias + residual), all fp32: vector, scalar and TMA-staged output kernels, both tiles, layers that
    # would otherwise take a single-kernel path, the residual aliasing y
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=sum(shape) + tile, dtype=torch.float32)
    g = torch.Generator().manual_seed(99)
    res = torch.randn((N, K, H, W), generator=g)
    name = "silu" if act == "silu" else None
    ref = oracle.epilogue(oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy()), res.numpy(), name)
    wT = B.sdwino_filter_transform_f32(w.cuda(), tile)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(N, C, H, W, K, tile))
    flag = B.ACT_SILU if act == "silu" else B.ACT_NONE
    xd, bd = x.cuda(), b.cuda()
    y = B.sdwino_conv3x3_f32_ex(xd, wT, bd, res.cuda(), K, tile, flag, ws)
    assert B.sdwino_last_device_status() == B.OK and y.dtype == torch.float32
    assert _rel_err(y.cpu(), ref) <= TOL
    y2 = res.cuda().clone()                                  # in place: the residual is y
    B.sdwino_conv3x3_f32_ex(xd, wT, bd, y2, K, tile, flag, ws, y=y2)
    assert torch.equal(y2, y)
    y3 = B.sdwino_conv3x3_f32_ex(xd, wT, None, None, K, tile, flag, ws)      # no residual, no bias
    ref3 = oracle.epilogue(oracle.direct_conv3x3(x.numpy(), w.numpy(), None), None, name)
    assert _rel_err(y3.cpu(), ref3) <= TOL
    if act == "none":
        # the epilogue adds exactly the residual to what the three kernels of the plain call compute
        B.sdwino_set_gemm_shape(1, 0)      # keeps the plain call off the single-kernel paths
        try:
            plain = B.sdwino_conv3x3_f32(xd, wT, bd, K, tile, ws)
        finally:
            B.sdwino_set_gemm_shape(0, 0)
        assert torch.equal(y, plain + res.cuda())
    with pytest.raises(B.SdwinoError) as e:
        B.sdwino_conv3x3_f32_ex(xd, wT, bd, None, K, tile, 7, ws)
    assert e.value.status == B.ERR_UNSUPPORTED


@pytest.mark.parametrize("tile", [2, 4])
@pytest.mark.parametrize("scale", [1.0e4, 3.0e7, 2.0e-6])
@pytest.mark.parametrize("shape", [(64, 96, 24, 32, 2), (33, 40, 13, 17, 1), (4, 24, 16, 16, 1), (160, 8, 40, 40, 1)])
def test_fp32_range_safe_entry_on_magnitudes_fp16_cannot_hold(B, shape, scale, tile):
    # activations far outside (or far below) the fp16 range: V would overflow to infinity (or flush to zero) in the
    # plain fp32 call; the range-safe call scales by a power of two around the fp16 operands
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=7 + C, dtype=torch.float32)
    x = x * scale
    b = b * scale
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    wT = B.sdwino_filter_transform_f32(w.cuda(), tile)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(N, C, H, W, K, tile))
    y = B.sdwino_conv3x3_f32(x.cuda(), wT, b.cuda(), K, tile, workspace=ws, scaled=True)
    assert B.sdwino_last_device_status() == B.OK
    assert torch.isfinite(y).all()
    assert _rel_err(y.cpu(), ref) <= (TOL_F2_REGRESSION if tile == 2 else TOL)
    if scale >= 1.0e4 and tile == 4:
        # where the plain call breaks down: its V exceeds the fp16 range
        y_plain = B.sdwino_conv3x3_f32(x.cuda(), wT, b.cuda(), K, tile, workspace=ws)
        assert B.sdwino_last_device_status() == B.OK
        assert (not torch.isfinite(y_plain).all()) or _rel_err(y_plain.cpu(), ref) > TOL


@pytest.mark.parametrize("tile", [2, 4])
def test_fp32_range_safe_entry_changes_nothing_on_moderate_inputs_and_handles_zero(B, tile):
    layer = ConvLayer(C=48, K=64, H=32, W=40, N=2)
    x, w, b = workloads.make_inputs(layer, seed=5, dtype=torch.float32)
    x = x * 16.0      # max|x| lands in [64, 128): the exponent is zero and the call reproduces the plain one
    assert 64.0 <= float(x.abs().max()) < 128.0
    wT = B.sdwino_filter_transform_f32(w.cuda(), tile)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, tile))
    y_plain = B.sdwino_conv3x3_f32(x.cuda(), wT, b.cuda(), layer.K, tile, workspace=ws).clone()
    y_safe = B.sdwino_conv3x3_f32(x.cuda(), wT, b.cuda(), layer.K, tile, workspace=ws, scaled=True)
    assert torch.equal(y_plain, y_safe)
    # an all-zero input has no maximum to scale by: the result is the bias
    y0 = B.sdwino_conv3x3_f32(torch.zeros_like(x).cuda(), wT, b.cuda(), layer.K, tile, workspace=ws, scaled=True)
    assert B.sdwino_last_device_status() == B.OK
    assert torch.equal(y0.cpu(), b.view(1, -1, 1, 1).expand_as(y0).contiguous())


@pytest.mark.parametrize("tile", [2, 4])
def test_fp32_host_entry_matches_the_device_entry(B, tile):
    layers = [ConvLayer(C=64, K=96, H=32, W=32, N=2), ConvLayer(C=20, K=24, H=17, W=23, N=1)]
    for seed, layer in enumerate(layers):
        x, w, b = workloads.make_inputs(layer, seed=seed, dtype=torch.float32, pin=True)
        dims = (layer.N, layer.C, layer.H, layer.W, layer.K, tile)
        wT = B.sdwino_filter_transform_f32(w.cuda(), tile)
        ws = B.alloc_workspace(B.sdwino_workspace_bytes(*dims))
        y_dev = B.sdwino_conv3x3_f32(x.cuda(), wT, b.cuda(), layer.K, tile, workspace=ws).cpu()
        hws = B.alloc_workspace(B.sdwino_host_staging_bytes_f32(*dims) + B.sdwino_workspace_bytes(*dims))
        assert B.sdwino_host_staging_bytes_f32(*dims) >= 2 * B.sdwino_host_staging_bytes(*dims) - 8192
        y_host = torch.full((layer.N, layer.K, layer.H, layer.W), float("nan"), dtype=torch.float32).pin_memory()
        B.sdwino_conv3x3_host_f32(x, wT, b, y_host, tile, hws)                       # synchronous
        assert torch.equal(y_host, y_dev)
        y_host.fill_(float("nan"))
        for _ in range(3):                                                           # asynchronous, back to back
            B.sdwino_conv3x3_host_f32(x, wT, b, y_host, tile, hws, wait=False)
        B.sdwino_host_join()
        torch.cuda.synchronize()
        assert torch.equal(y_host, y_dev)
        ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
        assert _rel_err(y_host, ref) <= TOL
