"""The pipelined single-launch path of F(4x4,3x3): one persistent launch whose CTAs transform, multiply and
inverse-transform successive blocks of tiles through rings of V and M that stay in L2.

It runs the arithmetic of the three-kernel path (same transform code, same MMAs in the same order), so its output
must be the same bits; both are also held against the fp64 oracle.  The hook sdwino_set_pipeline(2, ring, lead)
sends small layers through it, with rings far shorter than the layer so that every reuse dependency is exercised.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_05781_b200 import workloads
from paper_2412_05781_b200.workloads import ConvLayer

pytestmark = pytest.mark.gpu

TOL = 1e-2


@pytest.fixture(scope="module")
def B():
    from paper_2412_05781_b200 import build_library
    build_library()
    from paper_2412_05781_b200 import binding
    assert torch.cuda.is_available()
    return binding


def _conv(B, layer, x, w, b, mode, ring=0, lead=0):
    wT = B.sdwino_filter_transform(w.cuda(), 4)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, 4))
    B.sdwino_set_pipeline(mode, ring, lead)
    try:
        n0 = B.sdwino_launch_count()
        y = B.sdwino_conv3x3(x.cuda(), wT, None if b is None else b.cuda(), layer.K, 4, workspace=ws)
        status = B.sdwino_last_device_status()
        launches = B.sdwino_launch_count() - n0
    finally:
        B.sdwino_set_pipeline(1, 0, 0)
    assert status == B.OK, B.status_string(status)
    return y.cpu(), launches


SHAPES = [
    # C, K, H, W, N, ring, lead
    (64, 48, 64, 64, 2, 0, 0),        # 4 blocks of tiles, filters resident, ring = whole layer
    (64, 48, 64, 64, 2, 2, 1),        # the same through a ring of two blocks
    (32, 256, 96, 96, 1, 3, 1),       # 5 blocks (576 tiles: a ragged last block), n_tile 256 resident, groups of 4 CTAs
    (72, 200, 56, 72, 2, 3, 2),       # ragged C and K
    (40, 24, 50, 64, 1, 1, 1),        # H not a multiple of the tile, a ring of ONE block
    (512, 512, 64, 64, 1, 2, 1),      # 144 (position, k-tile) pairs: one CTA each, n_tile 128 resident
    (640, 320, 32, 32, 2, 2, 1),      # three k-tiles of 112 channels, filters resident
    (640, 640, 32, 32, 2, 1, 1),      # filters too large to stay resident: streaming GEMM in block order, ring of one
    (640, 640, 48, 64, 1, 2, 1),      # the same with a ragged last block
    (16, 16, 128, 256, 1, 4, 2),      # 16 blocks, tiny channel counts
]


@pytest.mark.parametrize("shape", SHAPES)
def test_pipelined_launch_matches_three_kernels_bitwise_and_oracle(B, shape):
    C, K, H, W, N, ring, lead = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=C + K + H)
    y_three, launches_three = _conv(B, layer, x, w, b, mode=0)
    y_pipe, launches_pipe = _conv(B, layer, x, w, b, mode=2, ring=ring, lead=lead)
    assert launches_three == 3 and launches_pipe == 1
    assert torch.equal(y_pipe, y_three)
    ks = sorted({0, K - 1, K // 2, K // 3})
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy(), channels=ks)
    got = y_pipe[:, torch.tensor(ks)].double().numpy()
    assert np.abs(got - ref).max() <= TOL * np.abs(ref).max()


def test_pipelined_launch_on_a_long_layer_with_the_library_s_ring_and_repeats_bitwise(B):
    # 256 -> 256 at 256x256: 4096 tiles = 32 blocks, ring and lead chosen by the library (shorter than the layer)
    layer = ConvLayer(C=256, K=256, H=256, W=256, N=1)
    x, w, b = workloads.make_inputs(layer, seed=11)
    y_three, launches_default = _conv(B, layer, x, w, b, mode=1)
    assert launches_default == 3        # the library does not take the pipelined launch by itself (it measured slower)
    y_pipe, launches = _conv(B, layer, x, w, b, mode=2)
    assert launches == 1
    assert torch.equal(y_pipe, y_three)
    # the counters are reset by every call: a second and third call give the same bits
    for _ in range(2):
        y_again, _ = _conv(B, layer, x, w, b, mode=2)
        assert torch.equal(y_again, y_three)
    ks = [0, 100, 255]
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy(), channels=ks)
    assert np.abs(y_pipe[:, torch.tensor(ks)].double().numpy() - ref).max() <= TOL * np.abs(ref).max()


def test_pipelined_launch_without_bias_and_inside_a_graph(B):
    layer = ConvLayer(C=96, K=160, H=64, W=128, N=1)
    x, w, _ = workloads.make_inputs(layer, seed=3, with_bias=False)
    y_three, _ = _conv(B, layer, x, w, None, mode=0)
    wT = B.sdwino_filter_transform(w.cuda(), 4)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, 4))
    xd = x.cuda()
    y = torch.zeros(layer.N, layer.K, layer.H, layer.W, dtype=torch.float16, device="cuda")
    B.sdwino_set_pipeline(2, 2, 1)
    try:
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            B.sdwino_conv3x3(xd, wT, None, layer.K, 4, y=y, workspace=ws, stream=stream)    # warm: kernel attributes
        stream.synchronize()
        y.zero_()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            B.sdwino_conv3x3(xd, wT, None, layer.K, 4, y=y, workspace=ws, stream=stream)
        for _ in range(3):
            y.zero_()
            graph.replay()
            torch.cuda.synchronize()
            assert B.sdwino_last_device_status() == B.OK
            assert torch.equal(y.cpu(), y_three)
    finally:
        B.sdwino_set_pipeline(1, 0, 0)


def test_set_pipeline_rejects_bad_values(B):
    for args in [(-1, 0, 0), (3, 0, 0), (1, -1, 0), (1, 0, -2)]:
        with pytest.raises(B.SdwinoError):
            B.sdwino_set_pipeline(*args)
    B.sdwino_set_pipeline(1, 0, 0)
