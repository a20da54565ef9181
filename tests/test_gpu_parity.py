"""Parity of the CUDA path (through the C ABI) with the fp64 oracle on seeded synthetic inputs.

Bar: max|gpu - ref| <= 1e-2 * max|ref| per layer, ref = fp64 direct convolution of the fp16 inputs
(fp16 storage, fp32 accumulation).  The same bound is evaluated separately on the edge tiles.  A tighter
regression bound is asserted for F(2x2,3x3), whose error is dominated by the fp16 rounding of V and M
(about 7e-4 measured; 2.5e-3 leaves a 3x margin).
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


def _run(B, layer, tile, seed=0, with_bias=True, ws_bytes=None, x=None, w=None, b=None):
    if x is None:
        x, w, b = workloads.make_inputs(layer, seed=seed, with_bias=with_bias)
    wT = B.sdwino_filter_transform(w.cuda(), tile)
    if ws_bytes is None:
        ws_bytes = B.sdwino_workspace_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, tile)
    ws = B.alloc_workspace(ws_bytes)
    y = B.sdwino_conv3x3(x.cuda(), wT, None if b is None else b.cuda(), layer.K, tile, workspace=ws)
    assert B.sdwino_last_device_status() == B.OK
    return x, w, b, y.cpu()


def _rel_err(y, ref):
    return float(np.abs(y.double().numpy() - ref).max() / np.abs(ref).max())


def _edge_mask(H, W, m):
    """Pixels belonging to the first/last tile row or column."""
    TH, TW = -(-H // m), -(-W // m)
    mask = np.zeros((H, W), dtype=bool)
    mask[:m, :] = True
    mask[:, :m] = True
    mask[(TH - 1) * m:, :] = True
    mask[:, (TW - 1) * m:] = True
    return mask


SMALL = [
    # C, K, H, W, N   -- several GEMM tiles in every direction plus ragged tails
    (1, 1, 4, 4, 1), (3, 4, 5, 7, 2), (4, 7, 1, 1, 3), (7, 33, 2, 9, 1), (33, 3, 13, 1, 2),
    (64, 128, 16, 16, 1), (65, 129, 17, 19, 1), (96, 160, 18, 21, 2), (130, 257, 33, 35, 1),
    (16, 16, 40, 56, 3), (200, 64, 23, 46, 1),
]


@pytest.mark.parametrize("tile", [2, 4])
@pytest.mark.parametrize("shape", SMALL)
def test_small_shapes_elementwise(B, shape, tile):
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b, y = _run(B, layer, tile, seed=sum(shape))
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    err = _rel_err(y, ref)
    assert err <= (TOL_F2_REGRESSION if tile == 2 else TOL), err
    # the same bound on the edge tiles alone (padding and tile-index logic)
    mask = _edge_mask(H, W, tile)
    d = np.abs(y.double().numpy() - ref)[:, :, mask].max()
    assert d <= TOL * np.abs(ref).max()
    # and against the three-step fp64 Winograd route with the same interpolation points
    wino = oracle.winograd_conv3x3(x.numpy(), w.numpy(), b.numpy(), m=tile, points=None if tile == 2 else F4_POINTS)
    assert _rel_err(y, wino) <= TOL


@pytest.mark.parametrize("ctas,n_tile", [(1, 16), (1, 32), (1, 48), (1, 160), (1, 256), (2, 16), (2, 32), (2, 80),
                                          (2, 160), (2, 256)])
def test_forced_gemm_shapes(B, ctas, n_tile):
    # every GEMM launch shape (single CTA / CTA pair, channels per tile) must give the same convolution;
    # 1150 tiles = 9 blocks of 128 (an odd count, so the last CTA pair is half empty), K = 200 is ragged
    # for every n_tile, C = 72 leaves a partial channel block
    layer = ConvLayer(C=72, K=200, H=50, W=46, N=2)
    x, w, b = workloads.make_inputs(layer, seed=21)
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    B.sdwino_set_gemm_shape(ctas, n_tile)
    try:
        _, _, _, y = _run(B, layer, 2, x=x, w=w, b=b)
    finally:
        B.sdwino_set_gemm_shape(0, 0)
    assert _rel_err(y, ref) <= TOL_F2_REGRESSION


@pytest.mark.parametrize("tile", [2, 4])
@pytest.mark.parametrize("C,K", [(4, 40), (3, 17), (8, 8), (1, 5)])
def test_few_input_channels_fused_kernel_matches_gemm_path(B, C, K, tile):
    # layers with at most 8 (F2) / 4 (F4) input channels take the single fused kernel; forcing a GEMM shape
    # sends the same layer through the three-kernel path: both must agree with the oracle and with each other
    layer = ConvLayer(C=C, K=K, H=21, W=26, N=2)
    x, w, b = workloads.make_inputs(layer, seed=5 + C)
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    n0 = B.sdwino_launch_count()
    _, _, _, y_auto = _run(B, layer, tile, x=x, w=w, b=b)
    launches_auto = B.sdwino_launch_count() - n0
    B.sdwino_set_gemm_shape(1, 16)
    try:
        n1 = B.sdwino_launch_count()
        _, _, _, y_gemm = _run(B, layer, tile, x=x, w=w, b=b)
        launches_gemm = B.sdwino_launch_count() - n1
    finally:
        B.sdwino_set_gemm_shape(0, 0)
    assert _rel_err(y_auto, ref) <= TOL and _rel_err(y_gemm, ref) <= TOL
    assert _rel_err(y_auto, y_gemm.double().numpy()) <= TOL
    assert launches_gemm == 4                       # filter transform + three kernels of one pass
    fused_expected = C <= (8 if tile == 2 else 4)
    assert launches_auto == (2 if fused_expected else 4)


FEW_K = [
    # C, K, H, W, N: W % 8 == 0; ragged channel blocks (C % 16, C % 64), odd H, several images, more than
    # two 64-channel filter blocks (ring instead of resident filters), a last block of tiles that is partial
    (16, 4, 8, 8, 1), (70, 3, 10, 16, 2), (128, 3, 32, 32, 1), (130, 8, 17, 24, 2), (320, 4, 64, 64, 2),
    (200, 7, 33, 40, 1), (300, 5, 7, 8, 3), (129, 1, 9, 48, 1), (64, 2, 130, 136, 1),
]


@pytest.mark.parametrize("shape", FEW_K)
def test_few_output_channels_fused_kernel(B, shape):
    # F2 layers with at most 8 output channels: one kernel (input transform -> tcgen05 -> output transform on
    # chip) once the layer is large enough; the threshold is lowered so that small ragged shapes take it too
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=sum(shape))
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    B.sdwino_set_fused_min_tiles(1)
    try:
        n0 = B.sdwino_launch_count()
        _, _, _, y = _run(B, layer, 2, x=x, w=w, b=b)
        assert B.sdwino_launch_count() - n0 == 2          # filter transform + the fused kernel
        _, _, _, y2 = _run(B, layer, 2, x=x, w=w, b=b)
    finally:
        B.sdwino_set_fused_min_tiles(0)
    assert torch.equal(y, y2)                              # deterministic
    assert _rel_err(y, ref) <= TOL_F2_REGRESSION
    mask = _edge_mask(H, W, 2)
    assert np.abs(y.double().numpy() - ref)[:, :, mask].max() <= TOL * np.abs(ref).max()
    # the three-kernel path on the same inputs
    B.sdwino_set_gemm_shape(1, 16)
    try:
        _, _, _, y_gemm = _run(B, layer, 2, x=x, w=w, b=b)
    finally:
        B.sdwino_set_gemm_shape(0, 0)
    assert _rel_err(y, y_gemm.double().numpy()) <= TOL_F2_REGRESSION


def test_few_output_channels_default_threshold_and_no_bias(B):
    # 6272 tiles = 49 blocks: above the default threshold without touching the knob; no bias
    layer = ConvLayer(C=48, K=3, H=112, W=112, N=2)
    x, w, _ = workloads.make_inputs(layer, seed=11, with_bias=False)
    n0 = B.sdwino_launch_count()
    _, _, _, y = _run(B, layer, 2, x=x, w=w, b=None)
    assert B.sdwino_launch_count() - n0 == 2
    ks = [0, 2]
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), None, channels=ks)
    d = np.abs(y[:, ks].double().numpy() - ref).max()
    assert d <= TOL_F2_REGRESSION * np.abs(ref).max()
    with pytest.raises(B.SdwinoError):
        B.sdwino_set_fused_min_tiles(-1)


def test_set_gemm_shape_rejects_bad_values(B):
    for ctas, n in [(3, 0), (-1, 0), (0, 8), (0, 272), (1, 100)]:
        with pytest.raises(B.SdwinoError):
            B.sdwino_set_gemm_shape(ctas, n)
    B.sdwino_set_gemm_shape(0, 0)


@pytest.mark.parametrize("tile", [2, 4])
def test_no_bias_and_zero_input(B, tile):
    layer = ConvLayer(C=20, K=24, H=11, W=10, N=2)
    x, w, b, y = _run(B, layer, tile, with_bias=False)
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), None)
    assert _rel_err(y, ref) <= TOL
    # x = 0  =>  y = bias exactly (every transform of zero is zero)
    x0, w0, b0 = workloads.make_inputs(layer, seed=3)
    x0.zero_()
    _, _, _, y0 = _run(B, layer, tile, x=x0, w=w0, b=b0)
    assert torch.equal(y0, b0.view(1, -1, 1, 1).expand_as(y0))


@pytest.mark.parametrize("tile", [2, 4])
def test_delta_filter_copies_input(B, tile):
    # centre tap 1 on the diagonal: y = x.  F(2x2) reproduces it exactly (all transforms are sums of
    # fp16 values that stay representable for |x| <= 2); F(4x4) within tolerance.
    layer = ConvLayer(C=8, K=8, H=12, W=14, N=1)
    x, w, b = workloads.make_inputs(layer, seed=5, with_bias=False)
    x = (x * 8).round() / 8
    x.clamp_(-2, 2)
    w.zero_()
    for c in range(8):
        w[c, c, 1, 1] = 1
    _, _, _, y = _run(B, layer, tile, x=x, w=w, b=None)
    if tile == 2:
        assert torch.equal(y, x)
    else:
        assert (y.float() - x.float()).abs().max() <= TOL * x.float().abs().max()


@pytest.mark.parametrize("tile", [2, 4])
@pytest.mark.parametrize("KC", [(320, 320), (3, 128), (130, 7)])
def test_filter_transform_matches_oracle(B, KC, tile):
    K, C = KC
    a = tile + 2
    g = torch.Generator().manual_seed(K + C)
    w = (torch.randn(K, C, 3, 3, generator=g) / (9 * C) ** 0.5).half()
    wT = B.sdwino_filter_transform(w.cuda(), tile)
    Kb, Cb = -(-K // 16), -(-C // 64)
    # header, then U[a*a][Cb][Kb][16][64]  ->  [a*a][Kb*16][Cb*64]
    hdr = wT[:16].view(torch.int32).cpu().tolist()          # 1 KB header: magic 'SDWU', K, C, tile
    assert hdr == [0x55574453, K, C, tile]
    U = wT[1024:].view(torch.float16)[:a * a * Kb * Cb * 1024].view(a * a, Cb, Kb, 16, 64).permute(0, 2, 3, 1, 4)
    U = U.reshape(a * a, Kb * 16, Cb * 64).cpu()
    Uo = oracle.filter_transform(w.numpy(), tile, points=None if tile == 2 else F4_POINTS)
    Uo = torch.from_numpy(Uo.reshape(K, C, a * a).transpose(2, 0, 1).copy())
    got = U[:, :K, :C].double()
    # |U - fp16(U64)| <= 1 ulp(fp16): compare with the two fp16 neighbours of the exact value
    ref16 = Uo.half()
    ulp = torch.maximum((torch.nextafter(ref16, torch.full_like(ref16, float("inf"))) - ref16).double().abs(),
                        (ref16 - torch.nextafter(ref16, torch.full_like(ref16, -float("inf")))).double().abs())
    assert bool(((got - ref16.double()).abs() <= ulp).all())
    # padding rows and columns are zero
    assert float(U[:, :, C:].abs().max() if Cb * 64 > C else 0) == 0
    assert float(U[:, K:, :].abs().max() if Kb * 16 > K else 0) == 0


def test_single_layer_config_full(B):
    # the small single-layer configuration, every output element
    layer = workloads.single_layer()[0]
    x, w, b, y = _run(B, layer, 2)
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    assert _rel_err(y, ref) <= TOL_F2_REGRESSION


def _sampled_check(B, layer, tile, nch, seed=0):
    x, w, b, y = _run(B, layer, tile, seed=seed)
    rng = np.random.default_rng(seed + layer.K)
    ks = np.sort(rng.choice(layer.K, size=min(nch, layer.K), replace=False))
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy(), channels=ks.tolist())
    got = y[:, torch.from_numpy(ks)].double().numpy()
    scale = np.abs(ref).max()
    err = np.abs(got - ref).max() / scale
    mask = _edge_mask(layer.H, layer.W, tile)
    edge = np.abs(got - ref)[:, :, mask].max() / scale
    return err, edge


@pytest.mark.parametrize("idx", range(16))
def test_sd15_unet_layers_sampled_channels(B, idx):
    # the benchmarked workload at full size: 16 seeded output channels, all spatial positions
    layer = workloads.sd15_unet()[idx]
    err, edge = _sampled_check(B, layer, 2, 16)
    assert err <= TOL_F2_REGRESSION and edge <= TOL, (layer.name, err, edge)


@pytest.mark.parametrize("idx", [0, 1, 2, 5, 9])
def test_vae_layers_sampled_channels(B, idx):
    layer = workloads.sd_vae_decoder_512()[idx]
    nch = 16 if layer.direct_flops < 1e11 else 4
    err, edge = _sampled_check(B, layer, 2, nch)
    assert err <= TOL_F2_REGRESSION and edge <= TOL, (layer.name, err, edge)


@pytest.mark.parametrize("idx,N", [(1, 1), (3, 2), (6, 4), (7, 1), (15, 8)])
@pytest.mark.parametrize("tile", [2, 4])
def test_sd21_unet_layers_both_tiles(B, idx, N, tile):
    layer = workloads.sd21_unet(N)[idx]
    err, edge = _sampled_check(B, layer, tile, 8)
    assert err <= TOL and edge <= TOL, (layer.name, tile, err, edge)


def test_multi_pass_equals_single_pass_bitwise(B):
    layer = ConvLayer(C=48, K=72, H=50, W=46, N=2)      # 1150 tiles -> 9 GEMM tiles of 128
    x, w, b = workloads.make_inputs(layer, seed=9)
    _, _, _, y_full = _run(B, layer, 2, x=x, w=w, b=b)
    small = B.sdwino_workspace_min_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, 2)
    _, _, _, y_min = _run(B, layer, 2, x=x, w=w, b=b, ws_bytes=small)            # 128 tiles per pass
    _, _, _, y_mid = _run(B, layer, 2, x=x, w=w, b=b, ws_bytes=small * 3 + 5000)  # 384 tiles per pass
    assert torch.equal(y_full, y_min) and torch.equal(y_full, y_mid)


def test_run_to_run_determinism_and_canaries(B):
    layer = ConvLayer(C=40, K=36, H=21, W=27, N=2)
    x, w, b = workloads.make_inputs(layer, seed=11)
    wT = B.sdwino_filter_transform(w.cuda(), 2)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, 2))
    n = layer.N * layer.K * layer.H * layer.W
    pad = 4096
    canary = torch.full((n + 2 * pad,), 1234.0, dtype=torch.float16, device="cuda")
    y = canary[pad:pad + n].view(layer.N, layer.K, layer.H, layer.W)
    B.sdwino_conv3x3(x.cuda(), wT, b.cuda(), layer.K, 2, y=y, workspace=ws)
    first = y.clone()
    B.sdwino_conv3x3(x.cuda(), wT, b.cuda(), layer.K, 2, y=y, workspace=ws)
    assert B.sdwino_last_device_status() == B.OK
    assert torch.equal(first, y)
    assert bool((canary[:pad] == 1234.0).all()) and bool((canary[pad + n:] == 1234.0).all())


def test_registered_workspace_and_host_entry_match_device_entry(B):
    layer = ConvLayer(C=24, K=40, H=19, W=16, N=2)
    x, w, b = workloads.make_inputs(layer, seed=13)
    _, _, _, y_dev = _run(B, layer, 2, x=x, w=w, b=b)
    wT = B.sdwino_filter_transform(w.cuda(), 2)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, 2))
    B.sdwino_set_workspace(ws)
    try:
        y_reg = B.sdwino_conv3x3(x.cuda(), wT, b.cuda(), layer.K, 2)
        assert torch.equal(y_reg.cpu(), y_dev)
    finally:
        B.sdwino_set_workspace(None)
    with pytest.raises(B.SdwinoError) as e:
        B.sdwino_conv3x3(x.cuda(), wT, b.cuda(), layer.K, 2)
    assert e.value.status == B.ERR_WORKSPACE
    args = (layer.N, layer.C, layer.H, layer.W, layer.K, 2)
    hws = B.alloc_workspace(B.sdwino_host_staging_bytes(*args) + B.sdwino_workspace_bytes(*args))
    y_host = torch.empty(layer.N, layer.K, layer.H, layer.W, dtype=torch.float16).pin_memory()
    B.sdwino_conv3x3_host(x.pin_memory(), wT, b.pin_memory(), y_host, 2, hws)
    assert torch.equal(y_host, y_dev)


def test_non_default_stream_and_launch_counter(B):
    layer = ConvLayer(C=16, K=16, H=8, W=8, N=1)
    x, w, b = workloads.make_inputs(layer, seed=17)
    _, _, _, y_ref = _run(B, layer, 2, x=x, w=w, b=b)
    s = torch.cuda.Stream()
    before = B.sdwino_launch_count()
    with torch.cuda.stream(s):
        wT = B.sdwino_filter_transform(w.cuda(), 2)
        ws = B.alloc_workspace(B.sdwino_workspace_bytes(1, 16, 8, 8, 16, 2))
        y = B.sdwino_conv3x3(x.cuda(), wT, b.cuda(), 16, 2, workspace=ws)
    s.synchronize()
    assert B.sdwino_launch_count() - before == 4      # filter + input + GEMM + output
    assert torch.equal(y.cpu(), y_ref)


def test_bounded_wait_reports_timeout_and_context_stays_usable(B):
    # a wait that nothing satisfies gives up after its limit, the kernel returns normally, the host reads the
    # status once, and the next convolution is unaffected
    assert B.sdwino_last_device_status() == B.OK
    B.sdwino_selftest_wait_timeout(1_000_000)            # 1 ms
    assert B.sdwino_last_device_status() == B.ERR_TIMEOUT
    assert B.sdwino_last_device_status() == B.OK          # cleared by the read
    with pytest.raises(B.SdwinoError):
        B.sdwino_selftest_wait_timeout(0)
    with pytest.raises(B.SdwinoError):
        B.sdwino_selftest_wait_timeout(20_000_000)        # more than 10 ms is refused
    layer = ConvLayer(C=32, K=48, H=10, W=12, N=1)
    x, w, b, y = _run(B, layer, 2, seed=2)
    assert _rel_err(y, oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())) <= TOL_F2_REGRESSION


@pytest.mark.parametrize("idx,tile", [(5, 2), (6, 4), (8, 4), (15, 2), (16, 2), (25, 2)])
def test_sdxl_layers_sampled_channels(B, idx, tile):
    # SDXL at 1024x1024: weight-streaming UNet layers, a large F4 layer, the few-channel layers at full size
    layer = workloads.sdxl_1024()[idx]
    err, edge = _sampled_check(B, layer, tile, nch=3, seed=idx)
    assert err <= TOL and edge <= TOL, (layer.name, err, edge)


def _random_shapes(count, seed):
    rng = np.random.default_rng(seed)
    shapes = []
    for _ in range(count):
        C = int(rng.choice([1, 2, 5, 8, 9, 17, 40, 64, 70, 130, 200]))
        K = int(rng.choice([1, 3, 8, 9, 16, 31, 48, 100, 160, 260]))
        H = int(rng.integers(1, 41))
        W = int(rng.choice([int(rng.integers(1, 41)), 8 * int(rng.integers(1, 6))]))   # half of them W % 8 == 0
        N = int(rng.integers(1, 4))
        shapes.append((C, K, H, W, N))
    return shapes


@pytest.mark.parametrize("shape", _random_shapes(24, seed=2412))
def test_seeded_random_shapes_both_tiles(B, shape):
    # a seeded draw over channel counts (few / ragged / several blocks), odd and even sizes, scalar and vector
    # transform paths, small batches: every path of the dispatcher must agree with the oracle
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=sum(shape))
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    scale = np.abs(ref).max()
    for tile in (2, 4):
        _, _, _, y = _run(B, layer, tile, x=x, w=w, b=b)
        d = np.abs(y.double().numpy() - ref)
        assert d.max() <= (TOL_F2_REGRESSION if tile == 2 else TOL) * scale, (shape, tile, d.max() / scale)
        mask = _edge_mask(H, W, tile)
        assert d[:, :, mask].max() <= TOL * scale


def test_async_host_entry_pipelines_calls_and_matches_device_entry(B):
    # several layers enqueued back to back through the asynchronous host entry (uploads on the library's copy
    # stream, alternating input slots), one synchronisation at the end: every result equals the device entry
    shapes = [(24, 40, 20, 24, 2), (40, 16, 12, 16, 1), (8, 24, 16, 16, 2), (64, 64, 9, 11, 1), (24, 40, 20, 24, 2)]
    stream = torch.cuda.Stream()
    jobs = []
    ws_bytes = 0
    for i, (C, K, H, W, N) in enumerate(shapes):
        layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
        x, w, b = workloads.make_inputs(layer, seed=40 + i, pin=True)
        tile = 2 if i % 2 == 0 else 4
        wT = B.sdwino_filter_transform(w.cuda(), tile)
        y = torch.empty(N, K, H, W, dtype=torch.float16).pin_memory()
        args = (N, C, H, W, K, tile)
        ws_bytes = max(ws_bytes, B.sdwino_host_staging_bytes(*args) + B.sdwino_workspace_bytes(*args))
        jobs.append((layer, tile, x, w, b, wT, y))
    ws = B.alloc_workspace(ws_bytes)
    torch.cuda.synchronize()
    for rep in range(2):                       # the second round reuses both slots
        for layer, tile, x, w, b, wT, y in jobs:
            y.zero_()
            B.sdwino_conv3x3_host(x, wT, b, y, tile, ws, stream=stream, wait=False)
        B.sdwino_host_join(stream)
        stream.synchronize()
        assert B.sdwino_last_device_status(stream) == B.OK
        for layer, tile, x, w, b, wT, y in jobs:
            ws2 = B.alloc_workspace(B.sdwino_workspace_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, tile))
            y_dev = B.sdwino_conv3x3(x.cuda(), wT, b.cuda(), layer.K, tile, workspace=ws2)
            assert torch.equal(y, y_dev.cpu()), (layer.name, tile, rep)


@pytest.mark.parametrize("tile", [2, 4])
@pytest.mark.parametrize("scale", [2.0 ** -10, 64.0])
def test_relative_error_is_scale_invariant_within_fp16_range(B, tile, scale):
    # V and M are stored in fp16: powers of two well inside its range only shift exponents, so the relative
    # error must not change (overflow of V needs |x| of a few thousand, underflow |x| below about 1e-5)
    layer = ConvLayer(C=96, K=64, H=24, W=32, N=1)
    x, w, b = workloads.make_inputs(layer, seed=9)
    xs = (x.float() * scale).half()
    bs = (b.float() * scale).half()
    _, _, _, y = _run(B, layer, tile, x=x, w=w, b=b)
    _, _, _, ysc = _run(B, layer, tile, x=xs, w=w, b=bs)
    ref = oracle.direct_conv3x3(xs.numpy(), w.numpy(), bs.numpy())
    assert _rel_err(ysc, ref) <= (TOL_F2_REGRESSION if tile == 2 else TOL)
    if scale > 1:      # exact power-of-two scaling without subnormals: bit-identical up to the exponent shift
        assert torch.equal((y.float() * scale).half(), ysc)


@pytest.mark.parametrize("case", ["tile", "channels_gemm", "few_in", "few_out"])
def test_mismatched_filter_buffer_is_reported_and_never_read(B, case):
    # wT carries a header (tile, K, C); every kernel that reads U checks it first.  A buffer transformed for
    # another tile size or other channel counts -- possibly much smaller than the one the call expects -- must give
    # SDWINO_ERR_INVALID_ARG through the device status word, leave the context usable and not touch memory
    # behind the buffer.
    if case == "tile":
        made, used, tile_made, tile_used = (64, 64), (64, 64), 2, 4
    elif case == "channels_gemm":
        made, used, tile_made, tile_used = (16, 16), (320, 320), 2, 2          # 50x smaller than expected
    elif case == "few_in":
        made, used, tile_made, tile_used = (8, 4), (64, 4), 2, 2               # (K, C): fused few-input-channel kernel
    else:
        made, used, tile_made, tile_used = (3, 32), (3, 64), 2, 2              # fused few-output-channel kernel
    g = torch.Generator().manual_seed(3)
    w = (torch.randn(made[0], made[1], 3, 3, generator=g) * 0.1).half()
    wT = B.sdwino_filter_transform(w.cuda(), tile_made)
    K, C = used
    H = W = 112 if case == "few_out" else 16
    N = 2 if case == "few_out" else 1
    x = torch.randn(N, C, H, W, generator=g).half().cuda()
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(N, C, H, W, K, tile_used))
    y = torch.full((N, K, H, W), 7.0, dtype=torch.float16, device="cuda")
    B.sdwino_conv3x3(x, wT, None, K, tile_used, y=y, workspace=ws)
    assert B.sdwino_last_device_status() == B.ERR_INVALID_ARG
    assert B.sdwino_last_device_status() == B.OK
    assert bool((y == 7.0).all())                           # nothing was computed from the wrong filters
    # the context is fine: a correct call right after
    layer = ConvLayer(C=32, K=48, H=10, W=12, N=1)
    xx, ww, bb, yy = _run(B, layer, 2, seed=2)
    assert _rel_err(yy, oracle.direct_conv3x3(xx.numpy(), ww.numpy(), bb.numpy())) <= TOL_F2_REGRESSION


@pytest.mark.parametrize("force_gemm", [False, True])
def test_hand_worked_example_bit_exact(B, force_gemm):
    # tests/golden/hand_worked_4x4.txt: every value of the example is representable in fp16 and every partial sum
    # exact, so F(2x2) must reproduce the hand-computed y bit for bit -- through the few-channel kernel and
    # through the three-kernel path
    import os
    rows, on = [], False
    with open(os.path.join(os.path.dirname(__file__), "golden", "hand_worked_4x4.txt")) as f:
        for line in f:
            line = line.strip()
            if line.startswith("["):
                on = line == "[y]"
            elif on and line and not line.startswith("#"):
                rows.append([float(v) for v in line.split()])
    want = torch.tensor(rows, dtype=torch.float16)
    x = torch.arange(1, 17, dtype=torch.float16).reshape(1, 1, 4, 4)
    w = torch.arange(1, 10, dtype=torch.float16).reshape(1, 1, 3, 3)
    b = torch.tensor([0.5], dtype=torch.float16)
    layer = ConvLayer(C=1, K=1, H=4, W=4, N=1)
    if force_gemm:
        B.sdwino_set_gemm_shape(1, 16)
    try:
        _, _, _, y = _run(B, layer, 2, x=x, w=w, b=b)
    finally:
        B.sdwino_set_gemm_shape(0, 0)
    assert torch.equal(y[0, 0], want)


@pytest.mark.parametrize("shape", [(64, 48, 64, 64, 2), (40, 16, 32, 32, 1), (24, 32, 16, 16, 3), (16, 16, 8, 8, 2),
                                   (9, 16, 20, 40, 1), (130, 16, 37, 24, 1), (12, 16, 140, 136, 1), (10, 16, 5, 8, 5),
                                   (33, 16, 260, 8, 1), (20, 16, 3, 264, 1), (6, 16, 248, 248, 1), (70, 16, 96, 96, 2)])
def test_staged_activation_transform_matches_register_kernel_bitwise(B, shape):
    # F(4x4), one pass, W % 8 == 0: the activation transform stages its input tiles in shared memory by TMA.  It
    # must produce the bits of the register-only kernel (same arithmetic) for whole-image blocks, blocks that
    # hang over the right and bottom edges, several channel images per step, and ragged channel counts.
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    B.sdwino_set_input_staging(2)
    try:
        x, w, b, y_staged = _run(B, layer, 4, seed=7)
        B.sdwino_set_input_staging(0)
        _, _, _, y_regs = _run(B, layer, 4, x=x, w=w, b=b)
    finally:
        B.sdwino_set_input_staging(1)
    assert torch.equal(y_staged, y_regs)
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    assert _rel_err(y_staged, ref) <= TOL


@pytest.mark.parametrize("shape,passes", [((24, 32, 100, 64, 3), 2), ((16, 16, 96, 96, 2), 3), ((8, 16, 64, 256, 1), 4),
                                          ((20, 16, 40, 128, 2), 5)])
def test_staged_activation_transform_over_several_passes(B, shape, passes):
    # F(4x4) with a workspace for a fraction of the tiles: the passes are cut at whole tile rows, each runs the
    # TMA-staged transform on its rows (blocks that straddle a cut are visited by both passes), the last one
    # zero-fills the padding of its last block of 128 tiles.  Same bits as one pass and as the register kernel.
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=13)
    full = B.sdwino_workspace_bytes(N, C, H, W, K, 4)
    B.sdwino_set_input_staging(2)
    try:
        _, _, _, y_one = _run(B, layer, 4, x=x, w=w, b=b)
        _, _, _, y_cut = _run(B, layer, 4, x=x, w=w, b=b, ws_bytes=full // passes + 4096)
        B.sdwino_set_input_staging(0)
        _, _, _, y_regs = _run(B, layer, 4, x=x, w=w, b=b, ws_bytes=full // passes + 4096)
    finally:
        B.sdwino_set_input_staging(1)
    assert torch.equal(y_one, y_cut) and torch.equal(y_one, y_regs)
    assert _rel_err(y_one, oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())) <= TOL


@pytest.mark.parametrize("shared", [True, False])
def test_async_host_entry_with_layers_of_different_sizes(B, shared):
    # Layers of very different sizes enqueued back to back through the asynchronous host entry.  With one shared
    # workspace their staging layouts overlap, so the library must order each call after the copies and kernels of
    # the calls still in flight (a 60 MB upload would otherwise land in memory that the previous layer's kernels
    # are still reading); with a workspace per layer the copies are free to overlap.  Either way every result
    # equals the device entry.
    shapes = [(64, 32, 96, 96, 2), (1200, 16, 64, 64, 4), (16, 256, 32, 32, 1), (320, 320, 64, 64, 2), (8, 16, 256, 256, 2),
              (256, 64, 16, 16, 1), (64, 32, 96, 96, 2)]
    stream = torch.cuda.Stream()
    jobs = []
    for i, (C, K, H, W, N) in enumerate(shapes):
        layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
        x, w, b = workloads.make_inputs(layer, seed=70 + i, pin=True)
        tile = B.sdwino_choose_tile(N, C, H, W, K)
        wT = B.sdwino_filter_transform(w.cuda(), tile)
        y = torch.empty(N, K, H, W, dtype=torch.float16).pin_memory()
        nbytes = B.sdwino_host_staging_bytes(N, C, H, W, K, tile) + B.sdwino_workspace_bytes(N, C, H, W, K, tile)
        jobs.append([layer, tile, x, b, wT, y, nbytes])
    if shared:
        ws_all = B.alloc_workspace(max(j[6] for j in jobs))
        spaces = [ws_all] * len(jobs)
    else:
        spaces = [B.alloc_workspace(j[6]) for j in jobs]
    expect = []
    for (layer, tile, x, b, wT, y, _) in jobs:
        ws2 = B.alloc_workspace(B.sdwino_workspace_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, tile))
        expect.append(B.sdwino_conv3x3(x.cuda(), wT, b.cuda(), layer.K, tile, workspace=ws2).cpu())
    torch.cuda.synchronize()
    for rep in range(3):
        for (layer, tile, x, b, wT, y, _), wsl in zip(jobs, spaces):
            y.zero_()
            B.sdwino_conv3x3_host(x, wT, b, y, tile, wsl, stream=stream, wait=False)
        B.sdwino_host_join(stream)
        stream.synchronize()
        assert B.sdwino_last_device_status(stream) == B.OK
        for (layer, tile, x, b, wT, y, _), want in zip(jobs, expect):
            assert torch.equal(y, want), (layer.name, tile, rep, shared)


@pytest.mark.parametrize("act", ["none", "silu"])
@pytest.mark.parametrize("shape,tile", [((32, 48, 16, 16, 2), 2), ((32, 48, 16, 16, 2), 4), ((20, 24, 9, 11, 1), 2),
                                        ((20, 24, 9, 11, 1), 4), ((4, 40, 12, 16, 1), 2), ((40, 4, 12, 16, 2), 2),
                                        ((64, 64, 64, 64, 1), 4), ((17, 33, 13, 24, 3), 4)])
def test_fused_residual_and_activation(B, shape, tile, act):
    # y = act(conv + bias + residual) in the output transform: vector and scalar kernels, both tiles, layers that
    # would otherwise take a single-kernel path, the residual aliasing y
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=sum(shape) + tile)
    g = torch.Generator().manual_seed(99)
    res = torch.randn((N, K, H, W), generator=g).half()
    ref = oracle.epilogue(oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy()), res.numpy(),
                          "silu" if act == "silu" else None)
    wT = B.sdwino_filter_transform(w.cuda(), tile)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(N, C, H, W, K, tile))
    flag = B.ACT_SILU if act == "silu" else B.ACT_NONE
    y = B.sdwino_conv3x3_ex(x.cuda(), wT, b.cuda(), res.cuda(), K, tile, flag, ws)
    assert B.sdwino_last_device_status() == B.OK
    assert _rel_err(y.cpu(), ref) <= TOL
    # in place: the residual is y
    y2 = res.cuda().clone()
    B.sdwino_conv3x3_ex(x.cuda(), wT, b.cuda(), y2, K, tile, flag, ws, y=y2)
    assert torch.equal(y2, y)
    # no residual, no bias
    y3 = B.sdwino_conv3x3_ex(x.cuda(), wT, None, None, K, tile, flag, ws)
    ref3 = oracle.epilogue(oracle.direct_conv3x3(x.numpy(), w.numpy(), None), None, "silu" if act == "silu" else None)
    assert _rel_err(y3.cpu(), ref3) <= TOL
    if act == "none":
        # nothing to fuse: the plain entry point, bit for bit
        y4 = B.sdwino_conv3x3(x.cuda(), wT, None, K, tile, workspace=ws)
        assert torch.equal(y3, y4)


def test_fused_epilogue_rejects_unknown_activation(B):
    layer = ConvLayer(C=16, K=16, H=8, W=8, N=1)
    x, w, b = workloads.make_inputs(layer, seed=3)
    wT = B.sdwino_filter_transform(w.cuda(), 2)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(1, 16, 8, 8, 16, 2))
    with pytest.raises(B.SdwinoError) as e:
        B.sdwino_conv3x3_ex(x.cuda(), wT, b.cuda(), None, 16, 2, 7, ws)
    assert e.value.status == B.ERR_UNSUPPORTED


@pytest.mark.parametrize("tile", [2, 4])
def test_more_than_2_to_31_elements(B, tile):
    # x and y of 2.15e9 elements each (4.3 GB): element offsets no longer fit 32 bits, the layer takes about twenty
    # passes, and with F(4x4) the passes are cut at whole tile rows for the TMA-staged transform.  Checked on
    # patches that the oracle computes from crops of x: the two corners that see the zero padding and a patch
    # whose offsets lie beyond 2^31 and 2^32 bytes.
    C, K, H, W = 16, 16, 11600, 11584
    assert C * H * W > 2 ** 31
    free, _ = torch.cuda.mem_get_info()
    if free < (24 << 30):
        pytest.skip("needs 24 GB of free device memory")
    g = torch.Generator(device="cuda").manual_seed(5)
    x = torch.empty((1, C, H, W), dtype=torch.float16, device="cuda")
    for c in range(C):
        x[0, c] = torch.randn((H, W), generator=g, device="cuda", dtype=torch.float32).half()
    layer = ConvLayer(C=C, K=K, H=16, W=16, N=1)
    _, w, b = workloads.make_inputs(layer, seed=21)
    wT = B.sdwino_filter_transform(w.cuda(), tile)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(1, C, H, W, K, tile))
    y = B.sdwino_conv3x3(x, wT, b.cuda(), K, tile, workspace=ws)
    assert B.sdwino_last_device_status() == B.OK
    S = 40
    for (i0, j0) in [(0, 0), (H - S, W - S), (H // 2 + 3, W // 2 - 5), (H - 2 * S, 8)]:
        # crop with one extra row / column where the image continues; the oracle pads the crop with zeros, so its
        # outermost rows and columns are only right where they coincide with the image border
        r0, r1, c0, c1 = max(i0 - 1, 0), min(i0 + S + 1, H), max(j0 - 1, 0), min(j0 + S + 1, W)
        crop = x[:, :, r0:r1, c0:c1].cpu().numpy()
        ref = oracle.direct_conv3x3(crop, w.numpy(), b.numpy())[:, :, i0 - r0:i0 - r0 + S, j0 - c0:j0 - c0 + S]
        got = y[:, :, i0:i0 + S, j0:j0 + S].cpu().double().numpy()
        assert np.abs(got - ref).max() <= TOL * np.abs(ref).max(), (tile, i0, j0)


@pytest.mark.parametrize("shape,tile", [((128, 128, 128, 128, 3), 4), ((256, 256, 128, 128, 2), 4), ((256, 256, 96, 96, 1), 2),
                                        ((320, 320, 128, 128, 1), 4), ((192, 200, 100, 104, 2), 4), ((64, 96, 160, 160, 2), 4),
                                        ((256, 128, 256, 256, 1), 4)])
def test_filter_resident_gemm_matches_streaming_gemm_bitwise(B, shape, tile):
    _check_resident_against_forced_shapes(B, shape, tile, [(1, None), (1, 128), (1, 64)])


@pytest.mark.parametrize("shape,tile", [((512, 512, 256, 256, 1), 4), ((512, 512, 128, 128, 1), 2), ((576, 500, 192, 192, 2), 4)])
def test_automatic_gemm_shape_on_large_layers_matches_forced_shapes_bitwise(B, shape, tile):
    # 512-channel layers with thousands of tiles (the automatic choice is CTA pairs): same bits as either shape forced
    _check_resident_against_forced_shapes(B, shape, tile, [(2, 256), (1, 256)])


@pytest.mark.parametrize("shape,tile", [((960, 320, 64, 64, 2), 4), ((640, 640, 48, 48, 1), 4), ((320, 320, 96, 96, 1), 4),
                                        ((200, 150, 40, 48, 3), 2), ((640, 320, 40, 40, 1), 4)])
def test_two_blocks_of_tiles_per_cta_match_forced_shapes_bitwise(B, shape, tile):
    # layers of 2 to 15 blocks of 128 tiles: a CTA tile covers two blocks (two accumulators, one filter box per
    # stage); an odd number of blocks leaves the last tile half empty.  Forcing a shape switches that off.
    _check_resident_against_forced_shapes(B, shape, tile, [(1, None), (1, 64)])


def _check_resident_against_forced_shapes(B, shape, tile, forced):
    # Layers with few channels and thousands of tiles keep the filter block of a (position, k-tile) in shared memory
    # and give every CTA a contiguous run of tiles; forcing the same GEMM shape by hand switches that off.  Same MMAs
    # in the same order: same bits.  Ragged K and C, runs that end inside a CTA's range, both tiles.
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b, y_res = _run(B, layer, tile, seed=31)
    n_auto = min(256, -(-K // 16) * 16)
    outs = []
    for ctas, n_tile in forced:
        B.sdwino_set_gemm_shape(ctas, n_auto if n_tile is None else n_tile)
        try:
            outs.append(_run(B, layer, tile, x=x, w=w, b=b)[3])
        finally:
            B.sdwino_set_gemm_shape(0, 0)
    for y_str in outs:
        assert torch.equal(y_res, y_str)
    nch = 8
    ks = sorted(np.random.default_rng(3).choice(K, nch, replace=False).tolist())
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy(), channels=ks)
    assert np.abs(y_res[:, ks].double().numpy() - ref).max() <= TOL * np.abs(ref).max()


def _random_large_shapes(count, seed):
    rng = np.random.default_rng(seed)
    shapes = []
    while len(shapes) < count:
        W = int(rng.choice([8, 16, 24, 32, 40, 48, 64, 64, 96, 128, 128, 192, 256, 320, 512]))
        H = int(rng.choice([W, max(1, W // 2), W + int(rng.integers(0, 9)), int(rng.integers(1, 70))]))
        C = int(rng.choice([9, 16, 40, 64, 96, 128, 192, 200, 256, 256, 320, 384, 512, 640]))
        K = int(rng.choice([9, 16, 48, 64, 100, 128, 160, 200, 256, 256, 320, 512, 640]))
        N = int(rng.choice([1, 1, 2, 3]))
        tile = int(rng.choice([2, 4, 4]))
        if N * C * H * W > 1.5e8 or N * K * H * W > 1.5e8 or 2.0 * N * K * C * H * W * 9 > 1.5e12:
            continue
        shapes.append((C, K, H, W, N, tile))
    return shapes


@pytest.mark.parametrize("shape", _random_large_shapes(40, seed=5781))
def test_seeded_random_layers_against_plain_kernels_and_oracle(B, shape):
    # A seeded draw over layer sizes up to a few hundred MB: whatever the dispatcher picks (staged transforms, CTA
    # pairs, two blocks of tiles per CTA tile, resident filters, one pass) must give the bits of the plain kernels
    # (register-only transforms, single-CTA streaming GEMM of a forced shape), also when the layer is cut into
    # about three passes with staging forced on, and must agree with the oracle on sampled channels.
    C, K, H, W, N, tile = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    rng = np.random.default_rng(sum(shape))
    x, w, b = workloads.make_inputs(layer, seed=sum(shape))
    xd, bd = x.cuda(), b.cuda()
    wT = B.sdwino_filter_transform(w.cuda(), tile)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(N, C, H, W, K, tile))
    y_auto = B.sdwino_conv3x3(xd, wT, bd, K, tile, workspace=ws)
    assert B.sdwino_last_device_status() == B.OK
    n_auto = min(256, -(-K // 16) * 16)
    B.sdwino_set_input_staging(0)
    B.sdwino_set_gemm_shape(1, int(rng.choice([n_auto, 64, 16])))
    try:
        y_plain = B.sdwino_conv3x3(xd, wT, bd, K, tile, workspace=ws)
    finally:
        B.sdwino_set_gemm_shape(0, 0)
        B.sdwino_set_input_staging(1)
    B.sdwino_set_input_staging(2)
    try:
        small = max(B.sdwino_workspace_min_bytes(N, C, H, W, K, tile) * 3, B.sdwino_workspace_bytes(N, C, H, W, K, tile) // 3)
        y_cut = B.sdwino_conv3x3(xd, wT, bd, K, tile, workspace=B.alloc_workspace(small))
    finally:
        B.sdwino_set_input_staging(1)
    assert torch.equal(y_auto, y_plain) and torch.equal(y_auto, y_cut)
    ks = sorted(rng.choice(K, min(K, 4), replace=False).tolist())
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy(), channels=ks)
    assert np.abs(y_auto[:, ks].cpu().double().numpy() - ref).max() <= TOL * np.abs(ref).max()


def test_concurrent_host_threads_on_their_own_streams(B):
    # compute calls with an explicit workspace may come from several host threads at once (ctypes releases the
    # interpreter lock during a call): each thread has its own stream, workspace and layer; the results are the bits
    # of the same calls made one after the other
    import threading
    shapes = [((72, 200, 50, 46, 2), 2), ((64, 48, 64, 64, 2), 4), ((4, 40, 16, 16, 2), 2), ((130, 257, 33, 35, 1), 4),
              ((48, 3, 64, 64, 2), 2), ((320, 320, 32, 32, 1), 2)]
    jobs = []
    for i, (shape, tile) in enumerate(shapes):
        C, K, H, W, N = shape
        layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
        x, w, b = workloads.make_inputs(layer, seed=40 + i)
        wT = B.sdwino_filter_transform(w.cuda(), tile)
        ws = B.alloc_workspace(B.sdwino_workspace_bytes(N, C, H, W, K, tile))
        jobs.append((layer, tile, x.cuda(), wT, b.cuda(), ws))
    torch.cuda.synchronize()
    serial = [B.sdwino_conv3x3(xd, wT, bd, layer.K, tile, workspace=ws).clone() for layer, tile, xd, wT, bd, ws in jobs]
    torch.cuda.synchronize()
    results = [None] * len(jobs)
    errors = []
    start = threading.Barrier(len(jobs))

    def work(i):
        try:
            layer, tile, xd, wT, bd, ws = jobs[i]
            st = torch.cuda.Stream()
            y = torch.empty_like(serial[i])
            start.wait()
            for _ in range(25):
                B.sdwino_conv3x3(xd, wT, bd, layer.K, tile, y=y, workspace=ws, stream=st)
            st.synchronize()
            results[i] = y
        except Exception as e:   # noqa: BLE001
            errors.append((i, repr(e)))

    threads = [threading.Thread(target=work, args=(i,)) for i in range(len(jobs))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    assert B.sdwino_last_device_status() == B.OK
    for i in range(len(jobs)):
        assert torch.equal(results[i], serial[i]), shapes[i]


@pytest.mark.parametrize("shape,tile", [((64, 48, 64, 64, 2), 4), ((72, 200, 50, 46, 2), 2), ((4, 40, 16, 16, 2), 2),
                                        ((48, 3, 64, 64, 8), 2)])
def test_first_call_inside_a_stream_capture_and_graph_replay(B, shape, tile):
    # the calls of a layer captured into a CUDA graph as the very first calls on their buffers (tensor maps not yet
    # cached: they are encoded during the capture, which must not disturb it), then replayed on new inputs
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=77)
    wT = B.sdwino_filter_transform(w.cuda(), tile)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(N, C, H, W, K, tile) + 4096)[4096 - 1024:]   # an address no test used
    xd, bd = torch.zeros_like(x, device="cuda"), b.cuda()
    y = torch.empty(N, K, H, W, dtype=torch.float16, device="cuda")
    torch.cuda.synchronize()
    st = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        B.sdwino_conv3x3(xd, wT, bd, K, tile, y=y, workspace=ws, stream=torch.cuda.current_stream())
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    for rep in range(2):
        y.zero_()
        xd.copy_(x.cuda() if rep == 0 else (2 * x).cuda())
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        assert B.sdwino_last_device_status() == B.OK
        want = ref if rep == 0 else 2 * (ref - b.double().numpy()[None, :, None, None]) + b.double().numpy()[None, :, None, None]
        assert _rel_err(y.cpu(), want) <= (TOL_F2_REGRESSION if tile == 2 else TOL)


@pytest.mark.parametrize("shape", [(1, 70000, 3, 3, 1), (70000, 1, 3, 3, 1), (16, 70000, 8, 8, 1), (70000, 16, 8, 8, 1),
                                   (3, 5, 2, 2, 70000), (9, 9, 3, 70000, 1), (4, 70000, 5, 5, 1)])
@pytest.mark.parametrize("tile", [2, 4])
def test_more_than_65535_channels_images_or_columns(B, shape, tile):
    # one dimension past the 65535 limit of grid.y / grid.z: the kernels that spend a row of blocks per channel
    # continue along grid.z; 8 sampled output channels against the oracle
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=9)
    _, _, _, y = _run(B, layer, tile, x=x, w=w, b=b)
    ks = sorted(np.random.default_rng(1).choice(K, min(K, 8), replace=False).tolist())
    if K > 8:
        ks[-1] = K - 1                       # the last channel sits in the last row of blocks
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy()[ks], b.numpy()[ks])
    assert _rel_err(y[:, ks], ref) <= (TOL_F2_REGRESSION if tile == 2 else TOL)
