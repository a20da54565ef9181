"""Every 3x3 convolution of every benchmark workload, at full size, with the algorithm the library ships for it.

One case per layer of the five workloads (single layer; SD v1.5 UNet, batch 2; SD VAE decoder to 512x512;
SD v2.1 UNet at 768x768; SDXL at 1024x1024 with its VAE decoder): the layer runs through the C ABI with the tile
that sdwino_choose_algorithm names -- which is what the benchmark times -- and seeded output channels (always the
first and the last one) are compared over all spatial positions with the fp64 direct convolution.  Bar:
max|gpu - ref| <= 1e-2 * max|ref| over the sampled channels, and the same bound on the edge tiles alone.
The SD v2.1 sweep is run at batch 1 and 8 with BOTH algorithms on every layer (the workload compares them), and at
batch 2 and 4 with the chosen one on a subset.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_05781_b200 import workloads

pytestmark = pytest.mark.gpu

TOL = 1e-2
TOL_F2_REGRESSION = 2.5e-3


@pytest.fixture(scope="module")
def B():
    from paper_2412_05781_b200 import build_library
    build_library()
    from paper_2412_05781_b200 import binding
    assert torch.cuda.is_available()
    return binding


def _channels(K, nch, seed):
    """nch distinct output channels, always including 0 and K - 1."""
    ks = {0, K - 1}
    rng = np.random.default_rng(seed)
    while len(ks) < min(nch, K):
        ks.add(int(rng.integers(0, K)))
    return sorted(ks)


def _check_layer(B, layer, tile, seed, nch=4):
    x, w, b = workloads.make_inputs(layer, seed=seed)
    wT = B.sdwino_filter_transform(w.cuda(), tile)
    ws = B.alloc_workspace(B.sdwino_workspace_bytes(layer.N, layer.C, layer.H, layer.W, layer.K, tile))
    y = B.sdwino_conv3x3(x.cuda(), wT, b.cuda(), layer.K, tile, workspace=ws)
    assert B.sdwino_last_device_status() == B.OK
    ks = _channels(layer.K, nch, seed + layer.K)
    got = y[:, torch.tensor(ks, device=y.device)].cpu().double().numpy()
    del y, ws, wT
    ref = oracle.direct_conv3x3(x.numpy(), w.numpy(), b.numpy(), channels=ks)
    scale = np.abs(ref).max()
    diff = np.abs(got - ref)
    err = diff.max() / scale
    m = tile
    TH, TW = -(-layer.H // m), -(-layer.W // m)
    edge = max(diff[:, :, :m, :].max(), diff[:, :, (TH - 1) * m:, :].max(), diff[:, :, :, :m].max(),
               diff[:, :, :, (TW - 1) * m:].max()) / scale
    bound = TOL if tile == 4 else TOL_F2_REGRESSION
    assert err <= bound and edge <= bound, (layer.name, tile, err, edge)


def _cases():
    out = []
    for name in ("single", "sd15_unet", "sd_vae_512", "sdxl_1024"):
        for idx, layer in enumerate(workloads.WORKLOADS[name]()):
            out.append(pytest.param(name, idx, id=f"{name}-{idx}-{layer.name}"))
    return out


@pytest.mark.parametrize("name,idx", _cases())
def test_every_layer_with_the_shipped_tile(B, name, idx):
    layer = workloads.WORKLOADS[name]()[idx]
    tile = B.sdwino_choose_algorithm(layer.N, layer.C, layer.H, layer.W, layer.K)
    assert tile in (1, 2, 4)
    _check_layer(B, layer, tile, seed=idx)


@pytest.mark.parametrize("tile", [2, 4])
@pytest.mark.parametrize("N", [1, 8])
@pytest.mark.parametrize("idx", range(16))
def test_sd21_unet_every_layer_both_tiles(B, idx, N, tile):
    layer = workloads.sd21_unet(N)[idx]
    _check_layer(B, layer, tile, seed=100 + idx)


@pytest.mark.parametrize("idx,N", [(1, 2), (4, 2), (8, 2), (13, 2), (3, 4), (7, 4), (10, 4), (15, 4)])
def test_sd21_unet_batches_2_and_4_with_the_shipped_tile(B, idx, N):
    layer = workloads.sd21_unet(N)[idx]
    tile = B.sdwino_choose_algorithm(layer.N, layer.C, layer.H, layer.W, layer.K)
    _check_layer(B, layer, tile, seed=200 + idx)
