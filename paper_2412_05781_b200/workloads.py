"""Seeded synthetic inputs and layer lists shaped like Stable Diffusion's 3x3 convolutions.

This module holds no arithmetic of the method: it only names layer shapes and draws
random tensors.  Both the CUDA path's callers (tests, benchmark) and the CPU oracle's
callers take their inputs from here.

Recipe (every layer): x ~ N(0, 1), w ~ N(0, 1/sqrt(9*C)) (standard deviation),
bias ~ N(0, 0.02), drawn in fp32 from ``torch.Generator().manual_seed(seed)`` on the
CPU in the order x, w, bias, then rounded to fp16; NCHW / KCRS contiguous.  The
shapes stand in for the SD v1.5 / v2.1 / SDXL UNet and VAE-decoder 3x3 convolutions
(stride 1, pad 1); trained weights and real activations are not used.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import torch


@dataclass(frozen=True)
class ConvLayer:
    """One stride-1 pad-1 3x3 convolution: x[N,C,H,W] * w[K,C,3,3] -> y[N,K,H,W]."""
    C: int
    K: int
    H: int
    W: int
    N: int = 1

    @property
    def name(self) -> str:
        return f"{self.C}->{self.K}@{self.H}x{self.W}n{self.N}"

    @property
    def direct_flops(self) -> int:
        """2*N*K*C*H*W*9, the direct-convolution-equivalent flop count."""
        return 2 * self.N * self.K * self.C * self.H * self.W * 9

    def tiles(self, m: int) -> int:
        return self.N * (-(-self.H // m)) * (-(-self.W // m))


def _mk(pairs, N):
    return [ConvLayer(C=c, K=k, H=h, W=h, N=N) for (c, k, h) in pairs]


_UNET_V15 = [(4, 320, 64), (320, 320, 64), (320, 640, 32), (640, 640, 32), (640, 1280, 16),
             (1280, 1280, 16), (1280, 1280, 8), (2560, 1280, 8), (2560, 1280, 16),
             (1920, 1280, 16), (1920, 640, 32), (1280, 640, 32), (960, 640, 32),
             (960, 320, 64), (640, 320, 64), (320, 4, 64)]

_VAE_512 = [(4, 512, 64), (512, 512, 64), (512, 512, 128), (512, 512, 256), (512, 256, 256),
            (256, 256, 256), (256, 256, 512), (256, 128, 512), (128, 128, 512), (128, 3, 512)]

_UNET_SDXL = [(4, 320, 128), (320, 320, 128), (320, 640, 64), (640, 640, 64), (640, 1280, 32),
              (1280, 1280, 32), (2560, 1280, 32), (1920, 1280, 32), (1280, 1280, 64),
              (1920, 640, 64), (1280, 640, 64), (960, 640, 64), (640, 640, 128),
              (960, 320, 128), (640, 320, 128), (320, 4, 128)]

_VAE_1024 = [(4, 512, 128), (512, 512, 128), (512, 512, 256), (512, 512, 512), (512, 256, 512),
             (256, 256, 512), (256, 256, 1024), (256, 128, 1024), (128, 128, 1024),
             (128, 3, 1024)]


def single_layer() -> List[ConvLayer]:
    """The small single-layer case: 320->320 at 32x32, batch 1."""
    return [ConvLayer(C=320, K=320, H=32, W=32, N=1)]


def sd15_unet(N: int = 2) -> List[ConvLayer]:
    """SD v1.5 UNet 3x3 convolutions at 512x512 (latent 64x64), batch 2 (CFG)."""
    return _mk(_UNET_V15, N)


def sd_vae_decoder_512() -> List[ConvLayer]:
    """SD VAE-decoder 3x3 convolutions for a 512x512 image, batch 1."""
    return _mk(_VAE_512, 1)


def sd21_unet(N: int = 1) -> List[ConvLayer]:
    """SD v2.1 UNet at 768x768 (latent 96x96): the v1.5 list with 64/32/16/8 -> 96/48/24/12."""
    scale = {64: 96, 32: 48, 16: 24, 8: 12}
    return _mk([(c, k, scale[h]) for (c, k, h) in _UNET_V15], N)


def sdxl_1024() -> List[ConvLayer]:
    """SDXL at 1024x1024: UNet (latent 128, batch 2) followed by the VAE decoder (batch 1)."""
    return _mk(_UNET_SDXL, 2) + _mk(_VAE_1024, 1)


WORKLOADS = {
    "single": single_layer,
    "sd15_unet": sd15_unet,
    "sd_vae_512": sd_vae_decoder_512,
    "sd21_unet": sd21_unet,
    "sdxl_1024": sdxl_1024,
}


def make_inputs(layer: ConvLayer, seed: int = 0, with_bias: bool = True,
                pin: bool = False, dtype: torch.dtype = torch.float16):
    """Return (x, w, bias) as CPU tensors drawn by the recipe in the module docstring: fp16 by default,
    the same draws left in fp32 with dtype=torch.float32 (inputs of the fp32 interface)."""
    assert dtype in (torch.float16, torch.float32)
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(layer.N, layer.C, layer.H, layer.W, generator=g, dtype=torch.float32)
    w = torch.randn(layer.K, layer.C, 3, 3, generator=g, dtype=torch.float32)
    w.mul_(1.0 / (9.0 * layer.C) ** 0.5)
    b: Optional[torch.Tensor] = None
    if with_bias:
        b = torch.randn(layer.K, generator=g, dtype=torch.float32).mul_(0.02).to(dtype)
    x, w = x.to(dtype), w.to(dtype)
    if pin:
        x, w = x.pin_memory(), w.pin_memory()
        b = b.pin_memory() if b is not None else None
    return x, w, b
