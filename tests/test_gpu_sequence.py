"""sdwino_conv3x3_sequence: several layers in one call, with or without the L2 prefetch of the next layer's filters.

A sequence must give, layer by layer, the bits of the single-layer calls (it launches the same kernels); every layer is
also held against the fp64 oracle on its own seeded input.  A chained case (each layer reads the output of the one
before) checks the ordering on the stream, again against single-layer calls fed the same way.
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


LAYERS = [
    ConvLayer(C=4, K=64, H=32, W=32, N=2),        # few input channels: the single-kernel path inside a sequence
    ConvLayer(C=64, K=96, H=32, W=32, N=2),
    ConvLayer(C=96, K=640, H=16, W=16, N=2),      # 2 MB of filters with tile 2: prefetched
    ConvLayer(C=640, K=640, H=8, W=8, N=2),       # direct form (tile 1), 7 MB of filters
    ConvLayer(C=640, K=320, H=19, W=23, N=1),     # ragged image, tile 4 filters of 14 MB
    ConvLayer(C=320, K=4, H=32, W=32, N=2),       # few output channels
]
TILES = [2, 4, 2, 1, 4, 4]


def _make(B, seeds_from=0):
    data, host = [], []
    for i, (L, tile) in enumerate(zip(LAYERS, TILES)):
        x, w, b = workloads.make_inputs(L, seed=seeds_from + i)
        wT = B.sdwino_filter_transform(w.cuda(), tile)
        y = torch.full((L.N, L.K, L.H, L.W), float("nan"), dtype=torch.float16, device="cuda")
        data.append((x.cuda(), wT, b.cuda(), y, L.K, tile))
        host.append((x, w, b))
    return data, host


@pytest.mark.parametrize("prefetch_mb", [0, 4, 64])
def test_sequence_matches_single_layer_calls_bitwise_and_the_oracle(B, prefetch_mb):
    data, host = _make(B)
    seq = B.make_sequence(data)
    need = B.sdwino_workspace_bytes_sequence(seq)
    assert need == max(B.sdwino_workspace_bytes(L.N, L.C, L.H, L.W, L.K, t) for L, t in zip(LAYERS, TILES))
    ws = B.alloc_workspace(need)
    torch.cuda.synchronize()
    n0 = B.sdwino_launch_count()
    B.sdwino_conv3x3_sequence(seq, ws, prefetch_mb << 20)
    assert B.sdwino_last_device_status() == B.OK
    launches = B.sdwino_launch_count() - n0
    singles = 0
    for (x, wT, b, y, K, tile), (xh, wh, bh), L in zip(data, host, LAYERS):
        n1 = B.sdwino_launch_count()
        y_single = B.sdwino_conv3x3(x, wT, b, K, tile, workspace=ws)
        singles += B.sdwino_launch_count() - n1
        assert torch.equal(y, y_single), L.name
        ref = oracle.direct_conv3x3(xh.numpy(), wh.numpy(), bh.numpy())
        err = np.abs(y.cpu().double().numpy() - ref).max() / np.abs(ref).max()
        assert err <= TOL, (L.name, tile, err)
    # prefetch launches: one for every layer after the first whose share of filters reaches 1 MB
    if prefetch_mb == 0:
        assert launches == singles
    else:
        assert singles < launches <= singles + len(LAYERS) - 1


def test_sequence_runs_a_chain_in_stream_order_and_inside_a_graph(B):
    # four layers, each reading the output of the one before it
    chain = [ConvLayer(C=32, K=48, H=40, W=24, N=1), ConvLayer(C=48, K=640, H=40, W=24, N=1),
             ConvLayer(C=640, K=64, H=40, W=24, N=1), ConvLayer(C=64, K=16, H=40, W=24, N=1)]
    tiles = [4, 2, 4, 2]
    x0, _, _ = workloads.make_inputs(chain[0], seed=7)
    bufs = [x0.cuda()] + [torch.zeros(L.N, L.K, L.H, L.W, dtype=torch.float16, device="cuda") for L in chain]
    data = []
    for i, (L, t) in enumerate(zip(chain, tiles)):
        _, w, b = workloads.make_inputs(L, seed=20 + i)      # variance-preserving filters: the chain stays near unit scale
        data.append((bufs[i], B.sdwino_filter_transform(w.cuda(), t), b.cuda(), bufs[i + 1], L.K, t))
    seq = B.make_sequence(data)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes_sequence(seq))
    # reference: the same chain through single-layer calls
    expect = []
    for (x, wT, b, y, K, t) in data:
        B.sdwino_conv3x3(x, wT, b, K, t, y=y, workspace=ws)
        expect.append(y.clone())
    assert B.sdwino_last_device_status() == B.OK
    assert all(torch.isfinite(e).all() for e in expect) and float(expect[-1].abs().max()) > 0
    for prefetch in (0, 8 << 20):
        for y in bufs[1:]:
            y.zero_()
        stream = torch.cuda.Stream()
        stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(stream):
            B.sdwino_conv3x3_sequence(seq, ws, prefetch, stream=stream)      # warm: kernel attributes, side stream
        stream.synchronize()
        assert all(torch.equal(y, e) for y, e in zip(bufs[1:], expect))
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            B.sdwino_conv3x3_sequence(seq, ws, prefetch, stream=stream)
        for _ in range(3):
            for y in bufs[1:]:
                y.zero_()
            graph.replay()
            torch.cuda.synchronize()
            assert B.sdwino_last_device_status() == B.OK
            assert all(torch.equal(y, e) for y, e in zip(bufs[1:], expect))


def test_sequence_with_a_bad_layer_launches_nothing(B):
    data, _ = _make(B, seeds_from=50)
    seq = B.make_sequence(data)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes_sequence(seq))
    seq[len(seq) - 1].tile = 3
    torch.cuda.synchronize()
    n0 = B.sdwino_launch_count()
    with pytest.raises(B.SdwinoError) as e:
        B.sdwino_conv3x3_sequence(seq, ws, 8 << 20)
    assert e.value.status == B.ERR_UNSUPPORTED
    seq[len(seq) - 1].tile = 4
    small = B.alloc_workspace(1 << 16)
    with pytest.raises(B.SdwinoError) as e:
        B.sdwino_conv3x3_sequence(seq, small, 0)
    assert e.value.status == B.ERR_WORKSPACE
    assert B.sdwino_launch_count() == n0
    torch.cuda.synchronize()
    assert all(torch.isnan(d[3]).all() for d in data)      # no y was touched
