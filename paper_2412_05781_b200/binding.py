"""ctypes binding of the sdwino C ABI (include/sdwino.h).

Argument marshalling only: every step of the convolution runs in the CUDA kernels of
libsdwino.so.  torch is used for device memory and streams.  There is no fallback: if the
shared library is missing the import of this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from .build import LIB_PATH

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_MISALIGNED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(7)

EXPORTS = [
    "sdwino_version", "sdwino_status_string", "sdwino_filter_bytes", "sdwino_filter_transform",
    "sdwino_workspace_bytes", "sdwino_workspace_min_bytes", "sdwino_set_workspace", "sdwino_conv3x3",
    "sdwino_conv3x3_ws", "sdwino_host_staging_bytes", "sdwino_conv3x3_host",
    "sdwino_last_device_status", "sdwino_launch_count", "sdwino_profile_enable", "sdwino_profile_collect",
    "sdwino_profile_records", "sdwino_set_gemm_shape", "sdwino_conv3x3_static", "sdwino_set_fused_min_tiles", "sdwino_choose_tile",
    "sdwino_selftest_wait_timeout", "sdwino_conv3x3_host_async", "sdwino_host_join", "sdwino_set_input_staging", "sdwino_conv3x3_ex",
    "sdwino_filter_transform_f32", "sdwino_conv3x3_f32", "sdwino_conv3x3_f32_ex",
    "sdwino_host_staging_bytes_f32", "sdwino_conv3x3_host_f32", "sdwino_conv3x3_host_f32_async", "sdwino_set_pipeline",
    "sdwino_conv3x3_f32_scaled", "sdwino_filter_q8_bytes", "sdwino_filter_quantize", "sdwino_conv3x3_q8",
    "sdwino_workspace_bytes_direct", "sdwino_conv3x3_direct", "sdwino_choose_algorithm",
    "sdwino_workspace_bytes_sequence", "sdwino_conv3x3_sequence",
]

class SdwinoLayer(ctypes.Structure):
    """struct sdwino_layer of the C ABI."""
    _fields_ = [("x", ctypes.c_void_p), ("wT", ctypes.c_void_p), ("bias", ctypes.c_void_p), ("y", ctypes.c_void_p),
                ("N", ctypes.c_int), ("C", ctypes.c_int), ("H", ctypes.c_int), ("W", ctypes.c_int), ("K", ctypes.c_int),
                ("tile", ctypes.c_int)]

KERNEL_KINDS = ("filter_transform", "input_transform", "wino_gemm", "output_transform", "fused", "layer")


class SdwinoError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2412_05781_b200.build` "
            "(there is no non-CUDA fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.sdwino_version.restype = i
    lib.sdwino_status_string.restype = ctypes.c_char_p
    lib.sdwino_status_string.argtypes = [i]
    lib.sdwino_filter_bytes.restype = sz
    lib.sdwino_filter_bytes.argtypes = [i, i, i]
    lib.sdwino_filter_transform.restype = i
    lib.sdwino_filter_transform.argtypes = [vp, vp, i, i, i, vp]
    for name in ("sdwino_workspace_bytes", "sdwino_workspace_min_bytes", "sdwino_host_staging_bytes",
                 "sdwino_host_staging_bytes_f32"):
        getattr(lib, name).restype = sz
        getattr(lib, name).argtypes = [i] * 6
    lib.sdwino_set_workspace.restype = i
    lib.sdwino_set_workspace.argtypes = [vp, sz]
    lib.sdwino_conv3x3.restype = i
    lib.sdwino_conv3x3.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp]
    lib.sdwino_conv3x3_static.restype = i
    lib.sdwino_conv3x3_static.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp]
    lib.sdwino_conv3x3_ws.restype = i
    lib.sdwino_conv3x3_ws.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp, sz, vp]
    lib.sdwino_conv3x3_ex.restype = i
    lib.sdwino_conv3x3_ex.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, i, vp, sz, vp]
    lib.sdwino_filter_transform_f32.restype = i
    lib.sdwino_filter_transform_f32.argtypes = [vp, vp, i, i, i, vp]
    lib.sdwino_conv3x3_f32.restype = i
    lib.sdwino_conv3x3_f32.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp, sz, vp]
    lib.sdwino_conv3x3_f32_scaled.restype = i
    lib.sdwino_conv3x3_f32_scaled.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp, sz, vp]
    lib.sdwino_conv3x3_f32_ex.restype = i
    lib.sdwino_conv3x3_f32_ex.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, i, vp, sz, vp]
    lib.sdwino_conv3x3_host.restype = i
    lib.sdwino_conv3x3_host.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp, sz, vp]
    lib.sdwino_host_join.restype = i
    lib.sdwino_host_join.argtypes = [vp]
    lib.sdwino_conv3x3_host_async.restype = i
    lib.sdwino_conv3x3_host_async.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp, sz, vp]
    for name in ("sdwino_conv3x3_host_f32", "sdwino_conv3x3_host_f32_async"):
        getattr(lib, name).restype = i
        getattr(lib, name).argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp, sz, vp]
    lib.sdwino_last_device_status.restype = i
    lib.sdwino_last_device_status.argtypes = [vp]
    lib.sdwino_launch_count.restype = ctypes.c_ulonglong
    lib.sdwino_profile_records.restype = i
    lib.sdwino_profile_records.argtypes = [ctypes.POINTER(i), ctypes.POINTER(ctypes.c_float), i, i]
    lib.sdwino_set_gemm_shape.restype = i
    lib.sdwino_set_gemm_shape.argtypes = [i, i]
    lib.sdwino_set_input_staging.restype = i
    lib.sdwino_set_input_staging.argtypes = [i]
    lib.sdwino_selftest_wait_timeout.restype = i
    lib.sdwino_selftest_wait_timeout.argtypes = [ctypes.c_ulonglong, vp]
    lib.sdwino_choose_tile.restype = i
    lib.sdwino_choose_tile.argtypes = [i, i, i, i, i]
    lib.sdwino_choose_algorithm.restype = i
    lib.sdwino_choose_algorithm.argtypes = [i, i, i, i, i]
    lib.sdwino_set_fused_min_tiles.restype = i
    lib.sdwino_set_fused_min_tiles.argtypes = [ctypes.c_longlong]
    lib.sdwino_filter_q8_bytes.restype = sz
    lib.sdwino_filter_q8_bytes.argtypes = [i, i, i]
    lib.sdwino_filter_quantize.restype = i
    lib.sdwino_filter_quantize.argtypes = [vp, vp, i, i, i, vp]
    lib.sdwino_conv3x3_q8.restype = i
    lib.sdwino_conv3x3_q8.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp, sz, vp]
    lib.sdwino_workspace_bytes_direct.restype = sz
    lib.sdwino_workspace_bytes_direct.argtypes = [i] * 6
    lib.sdwino_conv3x3_direct.restype = i
    lib.sdwino_conv3x3_direct.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp, sz, vp]
    lib.sdwino_set_pipeline.restype = i
    lib.sdwino_set_pipeline.argtypes = [i, i, i]
    lib.sdwino_profile_enable.restype = i
    lib.sdwino_profile_enable.argtypes = [i]
    lib.sdwino_profile_collect.restype = i
    lib.sdwino_profile_collect.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_ulonglong)]
    lib.sdwino_workspace_bytes_sequence.restype = sz
    lib.sdwino_workspace_bytes_sequence.argtypes = [ctypes.POINTER(SdwinoLayer), i]
    lib.sdwino_conv3x3_sequence.restype = i
    lib.sdwino_conv3x3_sequence.argtypes = [ctypes.POINTER(SdwinoLayer), i, vp, sz, sz, vp]
    return lib


lib = _load()


def status_string(status: int) -> str:
    return lib.sdwino_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise SdwinoError(status, where)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def sdwino_version() -> int:
    return int(lib.sdwino_version())


def sdwino_filter_bytes(K: int, C: int, tile: int) -> int:
    return int(lib.sdwino_filter_bytes(K, C, tile))


def sdwino_workspace_bytes(N: int, C: int, H: int, W: int, K: int, tile: int) -> int:
    return int(lib.sdwino_workspace_bytes(N, C, H, W, K, tile))


def sdwino_workspace_min_bytes(N: int, C: int, H: int, W: int, K: int, tile: int) -> int:
    return int(lib.sdwino_workspace_min_bytes(N, C, H, W, K, tile))


def sdwino_host_staging_bytes(N: int, C: int, H: int, W: int, K: int, tile: int) -> int:
    return int(lib.sdwino_host_staging_bytes(N, C, H, W, K, tile))


def sdwino_launch_count() -> int:
    return int(lib.sdwino_launch_count())


def sdwino_last_device_status(stream: Optional[torch.cuda.Stream] = None) -> int:
    return int(lib.sdwino_last_device_status(_stream_ptr(stream)))


def sdwino_selftest_wait_timeout(limit_ns: int, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Launch the bounded-wait self-test; sdwino_last_device_status() reports ERR_TIMEOUT afterwards."""
    _check(lib.sdwino_selftest_wait_timeout(limit_ns, _stream_ptr(stream)), "sdwino_selftest_wait_timeout")


def sdwino_set_gemm_shape(ctas: int = 0, n_tile: int = 0) -> None:
    """Force single-CTA (1) or CTA-pair (2) GEMM tiles and/or the channels per tile; 0 = automatic."""
    _check(lib.sdwino_set_gemm_shape(ctas, n_tile), "sdwino_set_gemm_shape")


def sdwino_set_input_staging(mode: int = 1) -> None:
    """Test hook for the F(4x4) activation transform: 0 register-only kernel, 1 automatic, 2 TMA-staged kernel
    wherever it applies."""
    _check(lib.sdwino_set_input_staging(int(mode)), "sdwino_set_input_staging")


def sdwino_choose_tile(N: int, C: int, H: int, W: int, K: int) -> int:
    """2 or 4: the output tile size (F(2x2) / F(4x4)) expected to be faster for this layer."""
    t = int(lib.sdwino_choose_tile(N, C, H, W, K))
    if t not in (2, 4):
        raise SdwinoError(ERR_INVALID_ARG, "sdwino_choose_tile")
    return t


def sdwino_choose_algorithm(N: int, C: int, H: int, W: int, K: int) -> int:
    """1, 2 or 4: direct convolution, F(2x2) or F(4x4), whichever is expected to be fastest for this layer."""
    t = int(lib.sdwino_choose_algorithm(N, C, H, W, K))
    if t not in (1, 2, 4):
        raise SdwinoError(ERR_INVALID_ARG, "sdwino_choose_algorithm")
    return t


def sdwino_set_fused_min_tiles(p_tiles: int = 0) -> None:
    """Blocks of 128 tiles from which few-output-channel layers take the single fused kernel; 0 = default."""
    _check(lib.sdwino_set_fused_min_tiles(p_tiles), "sdwino_set_fused_min_tiles")


def sdwino_set_pipeline(mode: int = 1, ring: int = 0, lead: int = 0) -> None:
    """Tuning / test hook: 0 never take the pipelined single-launch path, 1 where it is faster, 2 wherever possible;
    ring / lead in blocks of 128 tiles (0 = chosen by the library)."""
    _check(lib.sdwino_set_pipeline(mode, ring, lead), "sdwino_set_pipeline")


def sdwino_profile_enable(mode) -> None:
    """0 / False: off; 1 / True: CUDA events around every kernel launch; 2: around every convolution call as a whole
    (kind "layer")."""
    _check(lib.sdwino_profile_enable(int(mode)), "sdwino_profile_enable")


def sdwino_profile_collect():
    """-> {kernel kind: (total milliseconds, launches)} since the last collect."""
    ms = (ctypes.c_double * len(KERNEL_KINDS))()
    n = (ctypes.c_ulonglong * len(KERNEL_KINDS))()
    _check(lib.sdwino_profile_collect(ms, n), "sdwino_profile_collect")
    return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(KERNEL_KINDS)}


def sdwino_profile_records(capacity: int = 1 << 16, keep: bool = False):
    """-> [(kernel kind, milliseconds)] in launch order since the last collect; keep=True leaves the
    records in place (launches captured in a CUDA graph, read again after every replay)."""
    kinds = (ctypes.c_int * capacity)()
    ms = (ctypes.c_float * capacity)()
    n = int(lib.sdwino_profile_records(kinds, ms, capacity, 1 if keep else 0))
    if n > capacity:
        raise RuntimeError(f"{n} profile records, capacity {capacity}")
    return [(KERNEL_KINDS[kinds[i]], float(ms[i])) for i in range(n)]


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """Device scratch of `nbytes` bytes (torch allocations are at least 512-byte aligned;
    the returned view starts on a 1024-byte boundary)."""
    buf = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 1024
    return buf[off:off + nbytes]


def sdwino_filter_transform(w: torch.Tensor, tile: int, stream=None) -> torch.Tensor:
    """w: fp16 CUDA [K, C, 3, 3] contiguous -> wT (opaque uint8 CUDA tensor, tile-specific)."""
    assert w.is_cuda and w.dtype == torch.float16 and w.is_contiguous() and w.dim() == 4
    K, C = int(w.shape[0]), int(w.shape[1])
    assert tuple(w.shape[2:]) == (3, 3)
    nbytes = sdwino_filter_bytes(K, C, tile)
    if nbytes == 0:
        raise SdwinoError(ERR_UNSUPPORTED if tile not in (1, 2, 4) else ERR_INVALID_ARG, "sdwino_filter_bytes")
    wT = alloc_workspace(nbytes, w.device)
    _check(lib.sdwino_filter_transform(w.data_ptr(), wT.data_ptr(), K, C, tile, _stream_ptr(stream)),
           "sdwino_filter_transform")
    return wT


def sdwino_set_workspace(workspace: Optional[torch.Tensor]) -> None:
    if workspace is None:
        _check(lib.sdwino_set_workspace(None, 0), "sdwino_set_workspace")
    else:
        _check(lib.sdwino_set_workspace(workspace.data_ptr(), workspace.numel() * workspace.element_size()),
               "sdwino_set_workspace")


def sdwino_conv3x3(x: torch.Tensor, wT: torch.Tensor, bias: Optional[torch.Tensor], K: int, tile: int,
                   y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                   stream=None) -> torch.Tensor:
    """x: fp16 CUDA [N, C, H, W]; returns y fp16 [N, K, H, W].  With `workspace=None` the scratch
    registered by sdwino_set_workspace is used."""
    assert x.is_cuda and x.dtype == torch.float16 and x.is_contiguous() and x.dim() == 4
    N, C, H, W = (int(v) for v in x.shape)
    if y is None:
        y = torch.empty((N, K, H, W), dtype=torch.float16, device=x.device)
    assert y.is_contiguous() and y.dtype == torch.float16 and tuple(y.shape) == (N, K, H, W)
    if bias is not None:
        assert bias.is_cuda and bias.dtype == torch.float16 and bias.numel() == K and bias.is_contiguous()
    if workspace is None:
        rc = lib.sdwino_conv3x3(x.data_ptr(), wT.data_ptr(), _ptr(bias), y.data_ptr(), N, C, H, W, K, tile,
                                _stream_ptr(stream))
    else:
        rc = lib.sdwino_conv3x3_ws(x.data_ptr(), wT.data_ptr(), _ptr(bias), y.data_ptr(), N, C, H, W, K, tile,
                                   workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                   _stream_ptr(stream))
    _check(rc, "sdwino_conv3x3")
    return y


ACT_NONE, ACT_SILU = 0, 1


def sdwino_conv3x3_ex(x: torch.Tensor, wT: torch.Tensor, bias: Optional[torch.Tensor], residual: Optional[torch.Tensor],
                      K: int, tile: int, activation: int, workspace: torch.Tensor, y: Optional[torch.Tensor] = None,
                      stream=None) -> torch.Tensor:
    """y = act(conv3x3(x) + bias + residual): residual fp16 CUDA [N, K, H, W] or None (may be y itself),
    activation ACT_NONE or ACT_SILU."""
    assert x.is_cuda and x.dtype == torch.float16 and x.is_contiguous() and x.dim() == 4
    N, C, H, W = (int(v) for v in x.shape)
    if y is None:
        y = torch.empty((N, K, H, W), dtype=torch.float16, device=x.device)
    assert y.is_contiguous() and y.dtype == torch.float16 and tuple(y.shape) == (N, K, H, W)
    if bias is not None:
        assert bias.is_cuda and bias.dtype == torch.float16 and bias.numel() == K and bias.is_contiguous()
    if residual is not None:
        assert residual.is_cuda and residual.dtype == torch.float16 and residual.is_contiguous()
        assert tuple(residual.shape) == (N, K, H, W)
    rc = lib.sdwino_conv3x3_ex(x.data_ptr(), wT.data_ptr(), _ptr(bias), _ptr(residual), y.data_ptr(), N, C, H, W, K,
                               tile, int(activation), workspace.data_ptr(),
                               workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(rc, "sdwino_conv3x3_ex")
    return y


def sdwino_filter_transform_f32(w: torch.Tensor, tile: int, stream=None) -> torch.Tensor:
    """w: fp32 CUDA [K, C, 3, 3] contiguous -> wT (the same opaque buffer sdwino_filter_transform makes)."""
    assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous() and w.dim() == 4
    K, C = int(w.shape[0]), int(w.shape[1])
    assert tuple(w.shape[2:]) == (3, 3)
    nbytes = sdwino_filter_bytes(K, C, tile)
    if nbytes == 0:
        raise SdwinoError(ERR_UNSUPPORTED if tile not in (1, 2, 4) else ERR_INVALID_ARG, "sdwino_filter_bytes")
    wT = alloc_workspace(nbytes, w.device)
    _check(lib.sdwino_filter_transform_f32(w.data_ptr(), wT.data_ptr(), K, C, tile, _stream_ptr(stream)),
           "sdwino_filter_transform_f32")
    return wT


def sdwino_conv3x3_f32(x: torch.Tensor, wT: torch.Tensor, bias: Optional[torch.Tensor], K: int, tile: int,
                       workspace: torch.Tensor, y: Optional[torch.Tensor] = None, stream=None,
                       scaled: bool = False) -> torch.Tensor:
    """The convolution with fp32 x [N, C, H, W], bias [K] (or None) and y [N, K, H, W].  scaled=True calls
    sdwino_conv3x3_f32_scaled: activations of any fp32 magnitude."""
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous() and x.dim() == 4
    N, C, H, W = (int(v) for v in x.shape)
    if y is None:
        y = torch.empty((N, K, H, W), dtype=torch.float32, device=x.device)
    assert y.is_cuda and y.is_contiguous() and y.dtype == torch.float32 and tuple(y.shape) == (N, K, H, W)
    if bias is not None:
        assert bias.is_cuda and bias.dtype == torch.float32 and bias.numel() == K and bias.is_contiguous()
    fn = lib.sdwino_conv3x3_f32_scaled if scaled else lib.sdwino_conv3x3_f32
    rc = fn(x.data_ptr(), wT.data_ptr(), _ptr(bias), y.data_ptr(), N, C, H, W, K, tile,
            workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(rc, "sdwino_conv3x3_f32_scaled" if scaled else "sdwino_conv3x3_f32")
    return y


def sdwino_conv3x3_f32_ex(x: torch.Tensor, wT: torch.Tensor, bias: Optional[torch.Tensor], residual: Optional[torch.Tensor],
                          K: int, tile: int, activation: int, workspace: torch.Tensor, y: Optional[torch.Tensor] = None,
                          stream=None) -> torch.Tensor:
    """y = act(conv3x3(x) + bias + residual) with fp32 tensors (residual may be y itself)."""
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous() and x.dim() == 4
    N, C, H, W = (int(v) for v in x.shape)
    if y is None:
        y = torch.empty((N, K, H, W), dtype=torch.float32, device=x.device)
    assert y.is_cuda and y.is_contiguous() and y.dtype == torch.float32 and tuple(y.shape) == (N, K, H, W)
    if bias is not None:
        assert bias.is_cuda and bias.dtype == torch.float32 and bias.numel() == K and bias.is_contiguous()
    if residual is not None:
        assert residual.is_cuda and residual.dtype == torch.float32 and residual.is_contiguous()
        assert tuple(residual.shape) == (N, K, H, W)
    rc = lib.sdwino_conv3x3_f32_ex(x.data_ptr(), wT.data_ptr(), _ptr(bias), _ptr(residual), y.data_ptr(), N, C, H, W, K,
                                   tile, int(activation), workspace.data_ptr(),
                                   workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(rc, "sdwino_conv3x3_f32_ex")
    return y


STATIC_SCRATCH_BYTES = 32 << 20


def sdwino_conv3x3_static(x: torch.Tensor, wT: torch.Tensor, bias: Optional[torch.Tensor], K: int, tile: int,
                          y: torch.Tensor, stream=None) -> torch.Tensor:
    """The convolution with the library's built-in scratch array: for callers that may not allocate
    device memory.  x, wT, bias and the output y are all supplied by the caller; this wrapper allocates
    nothing either.  Layers whose smallest pass does not fit the STATIC_SCRATCH_BYTES array raise
    SdwinoError(ERR_WORKSPACE).  Calls share the array, so do not let two of them overlap on the GPU."""
    assert x.is_cuda and x.dtype == torch.float16 and x.is_contiguous() and x.dim() == 4
    N, C, H, W = (int(v) for v in x.shape)
    assert y.is_cuda and y.is_contiguous() and y.dtype == torch.float16 and tuple(y.shape) == (N, K, H, W)
    rc = lib.sdwino_conv3x3_static(x.data_ptr(), wT.data_ptr(), _ptr(bias), y.data_ptr(), N, C, H, W, K, tile,
                                   _stream_ptr(stream))
    _check(rc, "sdwino_conv3x3_static")
    return y


def sdwino_host_staging_bytes_f32(N: int, C: int, H: int, W: int, K: int, tile: int) -> int:
    return int(lib.sdwino_host_staging_bytes_f32(N, C, H, W, K, tile))


def sdwino_host_join(stream: Optional[torch.cuda.Stream] = None) -> None:
    """Make `stream` wait for the downloads of all earlier sdwino_conv3x3_host(..., wait=False) calls."""
    _check(lib.sdwino_host_join(_stream_ptr(stream)), "sdwino_host_join")


def sdwino_conv3x3_host(x: torch.Tensor, wT: torch.Tensor, bias: Optional[torch.Tensor], y: torch.Tensor,
                        tile: int, workspace: torch.Tensor, stream=None, wait: bool = True) -> torch.Tensor:
    """x, bias, y: fp16 CPU tensors (ideally pinned); wT and workspace on the device.  wait=True returns y
    after the stream has been synchronised; wait=False (sdwino_conv3x3_host_async) returns once the work is
    enqueued: y is complete after sdwino_host_join(stream) and a synchronisation of the stream."""
    assert not x.is_cuda and not y.is_cuda and x.dtype == torch.float16 and y.dtype == torch.float16
    assert x.is_contiguous() and y.is_contiguous()
    N, C, H, W = (int(v) for v in x.shape)
    K = int(y.shape[1])
    fn = lib.sdwino_conv3x3_host if wait else lib.sdwino_conv3x3_host_async
    rc = fn(x.data_ptr(), wT.data_ptr(), _ptr(bias), y.data_ptr(), N, C, H, W, K, tile,
            workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(rc, "sdwino_conv3x3_host" if wait else "sdwino_conv3x3_host_async")
    return y


def sdwino_conv3x3_host_f32(x: torch.Tensor, wT: torch.Tensor, bias: Optional[torch.Tensor], y: torch.Tensor,
                            tile: int, workspace: torch.Tensor, stream=None, wait: bool = True) -> torch.Tensor:
    """sdwino_conv3x3_host for the fp32 interface: x, bias, y are fp32 CPU tensors; the workspace holds
    sdwino_host_staging_bytes_f32(...) in front of the scratch."""
    assert not x.is_cuda and not y.is_cuda and x.dtype == torch.float32 and y.dtype == torch.float32
    assert x.is_contiguous() and y.is_contiguous() and (bias is None or bias.dtype == torch.float32)
    N, C, H, W = (int(v) for v in x.shape)
    K = int(y.shape[1])
    fn = lib.sdwino_conv3x3_host_f32 if wait else lib.sdwino_conv3x3_host_f32_async
    rc = fn(x.data_ptr(), wT.data_ptr(), _ptr(bias), y.data_ptr(), N, C, H, W, K, tile,
            workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(rc, "sdwino_conv3x3_host_f32" if wait else "sdwino_conv3x3_host_f32_async")
    return y


def sdwino_filter_q8_bytes(K: int, C: int, tile: int) -> int:
    return int(lib.sdwino_filter_q8_bytes(K, C, tile))


def sdwino_filter_quantize(wT: torch.Tensor, K: int, C: int, tile: int, stream=None) -> torch.Tensor:
    """wT (fp16 transformed filter of a [K, C, 3, 3] weight) -> the 8-bit transformed filter (opaque uint8 tensor)."""
    nbytes = int(lib.sdwino_filter_q8_bytes(K, C, tile))
    if nbytes == 0:
        raise SdwinoError(ERR_UNSUPPORTED if tile not in (2, 4) else ERR_INVALID_ARG, "sdwino_filter_q8_bytes")
    wTq = alloc_workspace(nbytes, wT.device)
    _check(lib.sdwino_filter_quantize(wT.data_ptr(), wTq.data_ptr(), K, C, tile, _stream_ptr(stream)),
           "sdwino_filter_quantize")
    return wTq


def sdwino_conv3x3_q8(x: torch.Tensor, wTq: torch.Tensor, bias: Optional[torch.Tensor], K: int, tile: int,
                      workspace: torch.Tensor, y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """The convolution with an 8-bit transformed filter (fp16 x, bias, y)."""
    assert x.is_cuda and x.dtype == torch.float16 and x.is_contiguous() and x.dim() == 4
    N, C, H, W = (int(v) for v in x.shape)
    if y is None:
        y = torch.empty((N, K, H, W), dtype=torch.float16, device=x.device)
    assert y.is_cuda and y.is_contiguous() and y.dtype == torch.float16 and tuple(y.shape) == (N, K, H, W)
    rc = lib.sdwino_conv3x3_q8(x.data_ptr(), wTq.data_ptr(), _ptr(bias), y.data_ptr(), N, C, H, W, K, tile,
                               workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(rc, "sdwino_conv3x3_q8")
    return y


def sdwino_workspace_bytes_direct(N: int, C: int, H: int, W: int, K: int, stride: int) -> int:
    return int(lib.sdwino_workspace_bytes_direct(N, C, H, W, K, stride))


def sdwino_conv3x3_direct(x: torch.Tensor, wT: torch.Tensor, bias: Optional[torch.Tensor], K: int, stride: int,
                          workspace: torch.Tensor, y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """The direct 3x3 convolution (pad 1) with stride 1 or 2: wT from sdwino_filter_transform(w, 1)."""
    assert x.is_cuda and x.dtype == torch.float16 and x.is_contiguous() and x.dim() == 4
    N, C, H, W = (int(v) for v in x.shape)
    Ho, Wo = (H - 1) // max(stride, 1) + 1, (W - 1) // max(stride, 1) + 1
    if y is None:
        y = torch.empty((N, K, Ho, Wo), dtype=torch.float16, device=x.device)
    assert y.is_cuda and y.is_contiguous() and y.dtype == torch.float16 and tuple(y.shape) == (N, K, Ho, Wo)
    rc = lib.sdwino_conv3x3_direct(x.data_ptr(), wT.data_ptr(), _ptr(bias), y.data_ptr(), N, C, H, W, K, stride,
                                   workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(rc, "sdwino_conv3x3_direct")
    return y


def make_sequence(layers) -> "ctypes.Array":
    """An array of struct sdwino_layer from (x, wT, bias or None, y, K, tile) tuples of CUDA tensors.  The tensors must
    stay alive while the array is used; nothing is copied."""
    arr = (SdwinoLayer * len(layers))()
    for d, (x, wT, bias, y, K, tile) in zip(arr, layers):
        assert x.is_cuda and x.dtype == torch.float16 and x.is_contiguous() and x.dim() == 4
        N, C, H, W = (int(v) for v in x.shape)
        assert y.is_cuda and y.dtype == torch.float16 and y.is_contiguous() and tuple(y.shape) == (N, K, H, W)
        d.x, d.wT, d.bias, d.y = x.data_ptr(), wT.data_ptr(), _ptr(bias), y.data_ptr()
        d.N, d.C, d.H, d.W, d.K, d.tile = N, C, H, W, K, tile
    return arr


def sdwino_workspace_bytes_sequence(seq) -> int:
    return int(lib.sdwino_workspace_bytes_sequence(seq, len(seq)))


def sdwino_conv3x3_sequence(seq, workspace: torch.Tensor, prefetch_bytes: int = 0, stream=None) -> None:
    """Runs the layers of `seq` (see make_sequence) in order on `stream`; prefetch_bytes > 0 also sends that much of each
    layer's filters towards L2 while the layer before it computes."""
    rc = lib.sdwino_conv3x3_sequence(seq, len(seq), workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                     prefetch_bytes, _stream_ptr(stream))
    _check(rc, "sdwino_conv3x3_sequence")
