"""The allocation-free entry point, sdwino_conv3x3_static, against the ordinary one.

Some users of the library cannot allocate device memory where they call it (inside a stream capture, in
a plug-in that is handed fixed buffers, in a process with a frozen memory budget).  For them the
library carries its scratch as a built-in device array.  This file is named so that pytest collects it
last: if it fails, a run that stops at the first failure has already run every other test.  It passes
alone in a fresh process and after the other tests (the built-in array is shared and keeps old contents,
which must not matter).
"""
import gc

import numpy as np
import pytest
import torch

import oracle
from paper_2412_05781_b200 import workloads
from paper_2412_05781_b200.workloads import ConvLayer

pytestmark = pytest.mark.gpu

TOL = 1e-2   # the tolerance of the parity tests: max|a - b| <= TOL * max|b|


@pytest.fixture(scope="module")
def B():
    from paper_2412_05781_b200 import build_library
    build_library()
    from paper_2412_05781_b200 import binding
    assert torch.cuda.is_available()
    return binding


def _both(B, layer, tile, seed, with_oracle=False):
    x, w, b = workloads.make_inputs(layer, seed=seed)
    xd, bd = x.cuda(), b.cuda()
    wT = B.sdwino_filter_transform(w.cuda(), tile)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, tile))
    y_ref = B.sdwino_conv3x3(xd, wT, bd, layer.K, tile, workspace=ws)
    y = torch.full_like(y_ref, float("nan"))                  # caller-provided output buffer
    gc.collect()                                              # tensors of earlier tests must not be freed in between
    torch.cuda.synchronize()
    # nothing may be allocated on this path: neither through torch's allocator nor behind its back
    torch_before = torch.cuda.memory_allocated()
    free_before, _ = torch.cuda.mem_get_info()
    B.sdwino_conv3x3_static(xd, wT, bd, layer.K, tile, y)     # scratch = the library's built-in array
    assert B.sdwino_last_device_status() == B.OK             # synchronises the stream
    free_after, _ = torch.cuda.mem_get_info()
    assert torch.cuda.memory_allocated() <= torch_before      # (a collection in between may only lower it)
    assert free_after == free_before, (free_before, free_after)
    if with_oracle:
        # the fp64 definition of the operator, on its own: the static entry does not lean on the other entry
        ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
        err = float(np.abs(y.cpu().double().numpy() - ref).max() / np.abs(ref).max())
        assert err <= TOL, (layer.name, tile, err)
    return y.cpu().float(), y_ref.cpu().float()


@pytest.mark.parametrize("tile", [2, 4])
def test_static_scratch_matches_workspace_entry_point_twice_in_a_row(B, tile):
    # two calls in a row with different layers: the second finds the first one's V and M in the array
    for seed, layer in enumerate([ConvLayer(C=96, K=160, H=40, W=36, N=2), ConvLayer(C=40, K=24, H=19, W=23, N=1)]):
        y, y_ref = _both(B, layer, tile, seed, with_oracle=True)
        assert not torch.isnan(y).any()
        err = float((y - y_ref).abs().max() / y_ref.abs().max())
        assert err <= TOL, (layer.name, tile, err)
        # same kernels, same arithmetic: the pass length is the only thing that may differ
        assert torch.equal(y, y_ref)


def test_static_scratch_takes_several_passes_on_a_large_layer(B):
    # 2 * 64 * 64 tiles * 16 positions * (320 + 320) channels = 84 MB of V and M: three passes through 32 MiB
    layer = ConvLayer(C=320, K=320, H=128, W=128, N=2)
    y, y_ref = _both(B, layer, 2, seed=5)
    assert float((y - y_ref).abs().max() / y_ref.abs().max()) <= TOL
    assert torch.equal(y, y_ref)


def test_static_scratch_rejects_layers_beyond_its_size(B):
    # 128 tiles * 36 positions * (2560 + 1280) channels * 2 bytes = 35 MB > 32 MiB: refused, nothing launched
    layer = ConvLayer(C=2560, K=1280, H=8, W=8, N=1)
    x = torch.zeros(layer.N, layer.C, layer.H, layer.W, dtype=torch.float16, device="cuda")
    y = torch.zeros(layer.N, layer.K, layer.H, layer.W, dtype=torch.float16, device="cuda")
    wT = B.alloc_workspace(B.sdwino_filter_bytes(layer.K, layer.C, 4))
    before = B.sdwino_launch_count()
    with pytest.raises(B.SdwinoError) as e:
        B.sdwino_conv3x3_static(x, wT, None, layer.K, 4, y)
    assert e.value.status == B.ERR_WORKSPACE
    assert B.sdwino_launch_count() == before
    with pytest.raises(B.SdwinoError) as e:
        B.sdwino_conv3x3_static(x, wT, None, layer.K, 3, y)
    assert e.value.status == B.ERR_UNSUPPORTED


@pytest.mark.parametrize("tile,limit", [(2, 8191), (4, 3640)])
def test_static_scratch_size_boundary(B, tile, limit):
    # 128 tiles * (tile+2)^2 positions * (C + K) channels * 2 bytes + 2 KiB must fit the 32 MiB array:
    # C + K = limit is the last layer accepted, limit + 1 the first one refused
    K = 16
    for total, accepted in [(limit, True), (limit + 1, False)]:
        C = total - K
        x = torch.zeros(1, C, 4, 4, dtype=torch.float16, device="cuda")
        y = torch.full((1, K, 4, 4), float("nan"), dtype=torch.float16, device="cuda")
        w = torch.zeros(K, C, 3, 3, dtype=torch.float16, device="cuda")
        wT = B.sdwino_filter_transform(w, tile)
        if accepted:
            B.sdwino_conv3x3_static(x, wT, None, K, tile, y)
            assert B.sdwino_last_device_status() == B.OK
            assert float(y.abs().max()) == 0.0            # zero input, zero filter, no bias
        else:
            with pytest.raises(B.SdwinoError) as e:
                B.sdwino_conv3x3_static(x, wT, None, K, tile, y)
            assert e.value.status == B.ERR_WORKSPACE
