"""The direct convolution entry (tile 1: nine per-tap GEMMs on the tensor cores), stride 1 and 2, against the fp64
definition.  Bar: max|gpu - ref| <= 1e-2 * max|ref| per layer; measured about 5e-4 (the nine partial sums are rounded
to fp16 once each), so a regression bound of 2.5e-3 is asserted as for F(2x2)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_05781_b200 import workloads
from paper_2412_05781_b200.workloads import ConvLayer

pytestmark = pytest.mark.gpu

TOL = 1e-2
TOL_REGRESSION = 2.5e-3


@pytest.fixture(scope="module")
def B():
    from paper_2412_05781_b200 import build_library
    build_library()
    from paper_2412_05781_b200 import binding
    assert torch.cuda.is_available()
    return binding


def _direct(B, layer, stride, x, w, b, ws_bytes=None):
    wT = B.sdwino_filter_transform(w.cuda(), 1)
    if ws_bytes is None:
        ws_bytes = B.sdwino_workspace_bytes_direct(layer.N, layer.C, layer.H, layer.W, layer.K, stride)
    ws = B.alloc_workspace(ws_bytes)
    y = B.sdwino_conv3x3_direct(x.cuda(), wT, None if b is None else b.cuda(), layer.K, stride, ws)
    assert B.sdwino_last_device_status() == B.OK
    return y.cpu()


SHAPES = [
    # C, K, H, W, N
    (1, 1, 4, 4, 1), (3, 4, 5, 7, 2), (7, 33, 2, 9, 1), (33, 3, 13, 1, 2), (64, 128, 16, 16, 1), (65, 129, 17, 19, 1),
    (96, 160, 18, 21, 2), (130, 257, 33, 35, 1), (16, 16, 40, 56, 3), (4, 40, 12, 12, 1), (40, 4, 24, 32, 1),
]


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("shape", SHAPES)
def test_direct_convolution_elementwise(B, shape, stride):
    C, K, H, W, N = shape
    layer = ConvLayer(C=C, K=K, H=H, W=W, N=N)
    x, w, b = workloads.make_inputs(layer, seed=sum(shape) + stride)
    y = _direct(B, layer, stride, x, w, b)
    ref = oracle.direct_conv3x3_strided(x.numpy(), w.numpy(), b.numpy(), stride)
    assert tuple(y.shape) == ref.shape
    err = np.abs(y.double().numpy() - ref).max() / np.abs(ref).max()
    assert err <= TOL_REGRESSION, err
    # border pixels alone (padding and window origins)
    d = np.abs(y.double().numpy() - ref)
    edge = max(d[:, :, 0].max(), d[:, :, -1].max(), d[:, :, :, 0].max(), d[:, :, :, -1].max())
    assert edge <= TOL * np.abs(ref).max()


@pytest.mark.parametrize("CKH", [(320, 320, 64), (640, 640, 32), (1280, 1280, 16)])
def test_unet_downsampling_convolutions_full_size(B, CKH):
    # the three stride-2 convolutions of the SD v1.x UNet encoder (latent 64 -> 32 -> 16 -> 8), batch 2
    C, K, H = CKH
    layer = ConvLayer(C=C, K=K, H=H, W=H, N=2)
    x, w, b = workloads.make_inputs(layer, seed=C)
    y = _direct(B, layer, 2, x, w, b)
    ref = oracle.direct_conv3x3_strided(x.numpy(), w.numpy(), b.numpy(), 2)
    assert np.abs(y.double().numpy() - ref).max() <= TOL_REGRESSION * np.abs(ref).max()


def test_direct_stride_1_agrees_with_winograd_and_passes_and_errors(B):
    layer = ConvLayer(C=72, K=200, H=30, W=26, N=2)
    x, w, b = workloads.make_inputs(layer, seed=4)
    y = _direct(B, layer, 1, x, w, b)
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy())
    assert np.abs(y.double().numpy() - ref).max() <= TOL_REGRESSION * np.abs(ref).max()
    # several passes through a small workspace give the same bits
    small = 3 * 128 * 9 * (72 + 200) * 2 + 1024
    y_small = _direct(B, layer, 1, x, w, b, ws_bytes=small)
    assert torch.equal(y, y_small)
    # no bias; zero input gives the bias exactly
    y0 = _direct(B, layer, 2, torch.zeros_like(x), w, b)
    assert torch.equal(y0, b.view(1, -1, 1, 1).expand_as(y0).contiguous())
    # errors: stride 3 is not offered, a Winograd filter buffer is refused by the header check
    wT1 = B.sdwino_filter_transform(w.cuda(), 1)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes_direct(2, 72, 30, 26, 200, 1))
    with pytest.raises(B.SdwinoError) as e:
        B.sdwino_conv3x3_direct(x.cuda(), wT1, b.cuda(), 200, 3, ws, y=torch.empty(2, 200, 10, 9, dtype=torch.float16, device="cuda"))
    assert e.value.status == B.ERR_UNSUPPORTED
    wT2 = B.sdwino_filter_transform(w.cuda(), 2)
    yk = torch.full((2, 200, 30, 26), 3.0, dtype=torch.float16, device="cuda")
    B.sdwino_conv3x3_direct(x.cuda(), wT2, b.cuda(), 200, 1, ws, y=yk)
    assert B.sdwino_last_device_status() == B.ERR_INVALID_ARG and bool((yk == 3.0).all())
    assert B.sdwino_workspace_bytes_direct(2, 72, 30, 26, 200, 0) == 0
