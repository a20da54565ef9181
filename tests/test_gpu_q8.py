"""8-bit transformed filters: sdwino_filter_quantize / sdwino_conv3x3_q8 against the fp64 oracle that applies the
same quantisation rule (integers in [-127, 127] with one fp32 scale per transform position and output channel).

Bar: max|gpu - ref| <= 1e-2 * max|ref| per layer, ref = the fp64 Winograd evaluation with the quantised filter.  The
integers themselves are compared too: the library forms U in fp32 and the oracle in fp64 before both round to fp16, so
an element can fall on the other side of an fp16 rounding boundary now and then; the test allows such elements to
differ by one and requires all but a small fraction to be equal.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_05781_b200 import workloads
from paper_2412_05781_b200.workloads import ConvLayer

pytestmark = pytest.mark.gpu

TOL = 1e-2
F4_POINTS = (0, 0.75, -0.75, 1.5, -1.5)


@pytest.fixture(scope="module")
def B():
    from paper_2412_05781_b200 import build_library
    build_library()
    from paper_2412_05781_b200 import binding
    assert torch.cuda.is_available()
    return binding


def _points(tile):
    return None if tile == 2 else F4_POINTS


@pytest.mark.parametrize("tile", [2, 4])
@pytest.mark.parametrize("KC", [(48, 72), (5, 130), (320, 320), (17, 3)])
def test_quantised_filter_matches_oracle(B, KC, tile):
    K, C = KC
    g = torch.Generator().manual_seed(K * 1000 + C)
    w = (torch.randn(K, C, 3, 3, generator=g) / (9 * C) ** 0.5).half()
    wT = B.sdwino_filter_transform(w.cuda(), tile)
    wTq = B.sdwino_filter_quantize(wT, K, C, tile)
    assert B.sdwino_last_device_status() == B.OK
    a2 = (tile + 2) ** 2
    Kb, Cb = -(-K // 16), -(-C // 64)
    raw = wTq.cpu().numpy()
    hdr = raw[:16].view(np.uint32)
    assert hdr[1] == K and hdr[2] == C and hdr[3] == (tile | 0x100)
    nb = a2 * Kb * Cb * 1024
    q_gpu = raw[1024:1024 + nb].reshape(a2, Cb, Kb, 16, 64).astype(np.int32) - 128
    s_off = 1024 + -(-nb // 1024) * 1024
    s_gpu = raw[s_off:s_off + a2 * Kb * 16 * 4].view(np.float32).reshape(a2, Kb * 16)
    q_ref, s_ref = oracle.quantize_filter_int8(oracle.filter_transform(w.numpy(), tile, _points(tile)))   # [K, C, a, a]
    # bring the library's blocked layout [pos][Cb][Kb][16][64] to [K, C, pos]
    q_lin = q_gpu.transpose(2, 3, 1, 4, 0).reshape(Kb * 16, Cb * 64, a2)
    assert not q_lin[K:].any() and not q_lin[:, C:].any()                      # padding rows and columns are zero
    q_lin = q_lin[:K, :C]
    q_ref = q_ref.reshape(K, C, a2)
    diff = np.abs(q_lin - q_ref)
    assert diff.max() <= 1 and (diff != 0).mean() <= 5e-3, (diff.max(), (diff != 0).mean())
    s_lin = s_gpu[:, :K].T                                                      # [K, pos]
    assert np.allclose(s_lin, s_ref.reshape(K, a2), rtol=1.5e-3, atol=0)
    assert np.all(s_gpu[:, K:] == 1.0)                                          # padding rows: all zeros, scale 1


SHAPES = [
    # C, K, H, W, N
    (64, 96, 16, 16, 1), (72, 200, 18, 22, 2), (130, 257, 9, 11, 1), (16, 24, 40, 56, 2),   # ragged, scalar and vector kernels
    (1280, 1280, 16, 16, 2), (2560, 1280, 8, 8, 2),                                          # weight streaming: one tile per CTA
    (320, 320, 64, 64, 2),                                                                   # several tiles per CTA
    (4, 40, 12, 12, 1), (40, 4, 24, 32, 1),                                                  # few channels: the GEMM path all the same
]


@pytest.mark.parametrize("tile", [2, 4])
@pytest.mark.parametrize("shape", SHAPES)
def test_q8_convolution_matches_oracle(B, shape, tile):
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=sum(shape))
    wTq = B.sdwino_filter_quantize(B.sdwino_filter_transform(w.cuda(), tile), K, C, tile)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(N, C, H, W, K, tile))
    y = B.sdwino_conv3x3_q8(x.cuda(), wTq, b.cuda(), K, tile, ws)
    assert B.sdwino_last_device_status() == B.OK
    full = layer.direct_flops < 3e9
    if full:
        ref = oracle.winograd_conv3x3_q8(x.numpy(), w.numpy(), b.numpy(), tile, _points(tile))
        got = y.cpu().double().numpy()
    else:   # large layers: four output channels (the Winograd oracle is slow), always the first and the last
        ks = sorted({0, K - 1, K // 2, K // 3})
        ref = oracle.winograd_conv3x3_q8(x.numpy(), w.numpy()[ks], b.numpy()[ks], tile, _points(tile))
        got = y[:, torch.tensor(ks, device=y.device)].cpu().double().numpy()
    err = np.abs(got - ref).max() / np.abs(ref).max()
    assert err <= TOL, err
    # and it is the quantised operator, not the plain one: close to the exact convolution, but measurably off
    exact = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy(), channels=None if full else ks)
    off = np.abs(got - exact).max() / np.abs(exact).max()
    assert off <= (4e-2 if tile == 2 else 1.2e-1), off


def test_q8_and_fp16_filters_are_not_interchangeable(B):
    layer = ConvLayer(C=64, K=48, H=16, W=16, N=1)
    x, w, b = workloads.make_inputs(layer, seed=1)
    wT = B.sdwino_filter_transform(w.cuda(), 2)
    wTq = B.sdwino_filter_quantize(wT, layer.K, layer.C, 2)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(1, 64, 16, 16, 48, 2))
    y = torch.full((1, 48, 16, 16), 7.0, dtype=torch.float16, device="cuda")
    B.sdwino_conv3x3_q8(x.cuda(), wT, b.cuda(), layer.K, 2, ws, y=y)             # an fp16 filter where 8 bits are expected
    assert B.sdwino_last_device_status() == B.ERR_INVALID_ARG
    assert bool((y == 7.0).all())
    B.sdwino_conv3x3(x.cuda(), wTq[:wT.numel()] if wTq.numel() >= wT.numel() else wTq, b.cuda(), layer.K, 2, y=y, workspace=ws)
    assert B.sdwino_last_device_status() == B.ERR_INVALID_ARG
    assert bool((y == 7.0).all())
    # a filter quantised for another layer shape is refused by the quantiser itself
    wT_other = B.sdwino_filter_transform(w[:, :32].contiguous().cuda(), 2)
    B.sdwino_filter_quantize(wT_other, layer.K, layer.C, 2)
    assert B.sdwino_last_device_status() == B.ERR_INVALID_ARG
    assert B.sdwino_filter_q8_bytes(48, 64, 3) == 0 and B.lib.sdwino_filter_q8_bytes(0, 64, 2) == 0


def test_q8_weight_streaming_layer_in_a_graph_is_deterministic(B):
    layer = ConvLayer(C=1280, K=1280, H=8, W=8, N=2)
    x, w, b = workloads.make_inputs(layer, seed=9)
    wTq = B.sdwino_filter_quantize(B.sdwino_filter_transform(w.cuda(), 2), layer.K, layer.C, 2)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(2, 1280, 8, 8, 1280, 2))
    xd, bd = x.cuda(), b.cuda()
    y0 = B.sdwino_conv3x3_q8(xd, wTq, bd, layer.K, 2, ws).clone()
    stream = torch.cuda.Stream()
    y = torch.zeros_like(y0)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        B.sdwino_conv3x3_q8(xd, wTq, bd, layer.K, 2, ws, y=y, stream=stream)
    for _ in range(3):
        y.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(y, y0)
    assert B.sdwino_last_device_status() == B.OK
