"""Host-only checks of the C-ABI boundary: the library builds, loads and exports every symbol the
header declares, and argument validation answers without a GPU."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2412_05781_b200 import build_library
    build_library()
    from paper_2412_05781_b200 import binding as b
    return b


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "sdwino.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sdwino_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(binding):
    names = _declared_symbols()
    assert "sdwino_conv3x3" in names and "sdwino_filter_transform" in names
    for n in names:
        assert hasattr(binding.lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_version_and_status_strings(binding):
    assert binding.sdwino_version() >= 100
    seen = {binding.status_string(s) for s in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert binding.status_string(99) == "unknown status"


def test_size_queries(binding):
    # wT = a*a planes of ceil(K/16) x ceil(C/64) blocks of 16 x 64 fp16
    # 1 KB header + blocks of 16 x 64 fp16
    assert binding.sdwino_filter_bytes(320, 320, 2) == 1024 + 16 * 20 * 5 * 1024 * 2
    assert binding.sdwino_filter_bytes(3, 4, 4) == 1024 + 36 * 1 * 1 * 1024 * 2
    assert binding.sdwino_filter_bytes(0, 4, 2) == 0
    assert binding.sdwino_filter_bytes(4, 4, 3) == 0
    full = binding.sdwino_workspace_bytes(2, 320, 64, 64, 320, 2)
    small = binding.sdwino_workspace_min_bytes(2, 320, 64, 64, 320, 2)
    # P = 2*32*32 = 2048 tiles, (C + K) = 640 fp16 per position and tile
    assert full == 2048 * 16 * 640 * 2 + 1024
    assert small == 128 * 16 * 640 * 2 + 1024
    assert binding.sdwino_workspace_bytes(1, 1, 1, 1, 1, 5) == 0
    assert binding.sdwino_workspace_bytes(1, 0, 1, 1, 1, 2) == 0
    # two slots of x, bias and y, each rounded up to 1 KB
    assert binding.sdwino_host_staging_bytes(1, 4, 8, 8, 4, 2) == 1024 * 6
    assert binding.sdwino_host_staging_bytes_f32(1, 4, 8, 8, 4, 2) == 1024 * 2 * (1 + 1 + 1)
    assert binding.sdwino_host_staging_bytes_f32(1, 64, 8, 8, 64, 2) == 2 * (16384 + 1024 + 16384)
    # the direct form: tile 1 = nine taps as positions; a tile is an output pixel, so stride 2 quarters the workspace
    assert binding.sdwino_filter_bytes(320, 320, 1) == 1024 + 9 * 20 * 5 * 1024 * 2
    assert binding.sdwino_workspace_bytes(2, 320, 64, 64, 320, 1) == 2 * 64 * 64 * 9 * 640 * 2 + 1024
    assert binding.sdwino_workspace_bytes_direct(2, 320, 64, 64, 320, 1) == 2 * 64 * 64 * 9 * 640 * 2 + 1024
    assert binding.sdwino_workspace_bytes_direct(2, 320, 64, 64, 320, 2) == 2 * 32 * 32 * 9 * 640 * 2 + 1024
    assert binding.sdwino_workspace_bytes_direct(1, 4, 7, 9, 4, 2) == 128 * 9 * 8 * 2 + 1024      # 4 x 5 pixels -> one block
    assert binding.sdwino_workspace_bytes_direct(1, 4, 8, 8, 4, 3) == 0
    # 8-bit filters: header, one byte per element of the blocked layout, one fp32 scale per (position, padded k)
    assert binding.sdwino_filter_q8_bytes(320, 320, 2) == 1024 + 16 * 20 * 5 * 1024 + 16 * 320 * 4
    assert binding.sdwino_filter_q8_bytes(3, 4, 4) == 1024 + 36 * 1024 + 3072      # 36 * 16 * 4 = 2304 -> 3 KB
    assert binding.sdwino_filter_q8_bytes(3, 4, 1) == 0
    # the algorithm choice with the direct form among the candidates
    assert binding.sdwino_choose_algorithm(2, 1280, 8, 8, 1280) == 1          # 128 output pixels: one block
    assert binding.sdwino_choose_algorithm(2, 2560, 16, 16, 1280) == 2
    assert binding.sdwino_choose_algorithm(2, 4, 8, 8, 320) == 2              # few input channels: the fused F(2x2) kernel
    assert binding.sdwino_choose_algorithm(1, 512, 256, 256, 512) == 4


def test_argument_validation_without_gpu(binding):
    lib = binding.lib
    buf = ctypes.create_string_buffer(4096)
    p = (ctypes.addressof(buf) + 1023) // 1024 * 1024
    assert lib.sdwino_filter_transform(None, p, 4, 4, 2, None) == binding.ERR_INVALID_ARG
    assert lib.sdwino_filter_transform(p, p, 4, 4, 3, None) == binding.ERR_UNSUPPORTED
    assert lib.sdwino_filter_transform(p + 1, p, 4, 4, 2, None) == binding.ERR_MISALIGNED
    assert lib.sdwino_filter_transform(p, p + 16, 4, 4, 2, None) == binding.ERR_MISALIGNED
    assert lib.sdwino_conv3x3_ws(None, p, None, p, 1, 4, 8, 8, 4, 2, p, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert lib.sdwino_conv3x3_ws(p, p, None, p, 1, 4, 8, 0, 4, 2, p, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert lib.sdwino_conv3x3_ws(p, p, None, p, 1, 4, 8, 8, 4, 6, p, 1 << 20, None) == binding.ERR_UNSUPPORTED
    assert lib.sdwino_conv3x3_ws(p, p, None, p + 1, 1, 4, 8, 8, 4, 2, p, 1 << 20, None) == binding.ERR_MISALIGNED
    assert lib.sdwino_conv3x3_ws(p, p, None, p, 1, 4, 8, 8, 4, 2, None, 0, None) == binding.ERR_WORKSPACE
    assert lib.sdwino_conv3x3_ws(p, p, None, p, 1, 4, 8, 8, 4, 2, p, 4096, None) == binding.ERR_WORKSPACE
    assert lib.sdwino_conv3x3_ws(p, p, None, p, 1, 4, 8, 8, 4, 2, p + 8, 1 << 20, None) == binding.ERR_MISALIGNED
    # no workspace registered
    assert lib.sdwino_set_workspace(None, 0) == binding.OK
    assert lib.sdwino_conv3x3(p, p, None, p, 1, 4, 8, 8, 4, 2, None) == binding.ERR_WORKSPACE
    assert lib.sdwino_set_workspace(p, 0) == binding.ERR_INVALID_ARG
    assert lib.sdwino_set_workspace(p + 4, 64) == binding.ERR_MISALIGNED
    assert lib.sdwino_conv3x3_host(None, p, None, p, 1, 4, 8, 8, 4, 2, p, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert lib.sdwino_conv3x3_host(p, p, None, p, 1, 4, 8, 8, 4, 2, p, 1024, None) == binding.ERR_WORKSPACE
    # fused epilogue: unknown activation, odd residual pointer, then the checks of the plain call
    assert lib.sdwino_conv3x3_ex(p, p, None, None, p, 1, 4, 8, 8, 4, 2, 7, p, 1 << 20, None) == binding.ERR_UNSUPPORTED
    assert lib.sdwino_conv3x3_ex(p, p, None, p + 1, p, 1, 4, 8, 8, 4, 2, 1, p, 1 << 20, None) == binding.ERR_MISALIGNED
    assert lib.sdwino_conv3x3_ex(None, p, None, None, p, 1, 4, 8, 8, 4, 2, 1, p, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert lib.sdwino_conv3x3_ex(p, p, None, None, p, 1, 4, 8, 8, 4, 2, 0, None, 0, None) == binding.ERR_WORKSPACE
    # fp32 interface: the checks come before any CUDA call
    assert lib.sdwino_filter_transform_f32(None, p, 4, 4, 2, None) == binding.ERR_INVALID_ARG
    assert lib.sdwino_filter_transform_f32(p, p, 4, 4, 3, None) == binding.ERR_UNSUPPORTED
    assert lib.sdwino_filter_transform_f32(p + 2, p, 4, 4, 2, None) == binding.ERR_MISALIGNED
    assert lib.sdwino_conv3x3_f32(None, p, None, p, 1, 4, 8, 8, 4, 2, p, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert lib.sdwino_conv3x3_f32(p, p, None, p, 1, 4, 8, 8, 4, 5, p, 1 << 20, None) == binding.ERR_UNSUPPORTED
    assert lib.sdwino_conv3x3_f32(p + 2, p, None, p, 1, 4, 8, 8, 4, 2, p, 1 << 20, None) == binding.ERR_MISALIGNED
    assert lib.sdwino_conv3x3_f32(p, p, p + 2, p, 1, 4, 8, 8, 4, 2, p, 1 << 20, None) == binding.ERR_MISALIGNED
    assert lib.sdwino_conv3x3_f32(p, p, None, p, 1, 4, 8, 8, 4, 2, None, 0, None) == binding.ERR_WORKSPACE
    assert lib.sdwino_conv3x3_f32_ex(p, p, None, None, p, 1, 4, 8, 8, 4, 2, 7, p, 1 << 20, None) == binding.ERR_UNSUPPORTED
    assert lib.sdwino_conv3x3_f32_ex(p, p, None, p + 2, p, 1, 4, 8, 8, 4, 2, 1, p, 1 << 20, None) == binding.ERR_MISALIGNED
    assert lib.sdwino_conv3x3_f32_ex(None, p, None, None, p, 1, 4, 8, 8, 4, 2, 1, p, 1 << 20, None) == binding.ERR_INVALID_ARG
    # the later entry points: range-safe fp32, fp32 host buffers, 8-bit filters, the direct form, the pipeline hook
    assert lib.sdwino_conv3x3_f32_scaled(None, p, None, p, 1, 4, 8, 8, 4, 2, p, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert lib.sdwino_conv3x3_f32_scaled(p, p, None, p, 1, 4, 8, 8, 4, 5, p, 1 << 20, None) == binding.ERR_UNSUPPORTED
    assert lib.sdwino_conv3x3_f32_scaled(p, p, None, p, 1, 4, 8, 8, 4, 2, None, 0, None) == binding.ERR_WORKSPACE
    assert lib.sdwino_conv3x3_host_f32(None, p, None, p, 1, 4, 8, 8, 4, 2, p, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert lib.sdwino_conv3x3_host_f32(p, p, None, p, 1, 4, 8, 8, 4, 1, p, 1 << 20, None) == binding.ERR_UNSUPPORTED
    assert lib.sdwino_conv3x3_host_f32(p, p, None, p, 1, 4, 8, 8, 4, 2, p, 1024, None) == binding.ERR_WORKSPACE
    assert lib.sdwino_filter_quantize(None, p, 4, 4, 2, None) == binding.ERR_INVALID_ARG
    assert lib.sdwino_filter_quantize(p, p, 4, 4, 3, None) == binding.ERR_UNSUPPORTED
    assert lib.sdwino_filter_quantize(p, p + 16, 4, 4, 2, None) == binding.ERR_MISALIGNED
    assert lib.sdwino_conv3x3_q8(None, p, None, p, 1, 4, 8, 8, 4, 2, p, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert lib.sdwino_conv3x3_q8(p, p, None, p, 1, 4, 8, 8, 4, 1, p, 1 << 20, None) == binding.ERR_UNSUPPORTED   # no direct form in 8 bits
    assert lib.sdwino_conv3x3_q8(p, p, None, p, 1, 4, 8, 8, 4, 2, None, 0, None) == binding.ERR_WORKSPACE
    assert lib.sdwino_conv3x3_direct(None, p, None, p, 1, 4, 8, 8, 4, 1, p, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert lib.sdwino_conv3x3_direct(p, p, None, p, 1, 4, 8, 8, 4, 0, p, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert lib.sdwino_conv3x3_direct(p, p, None, p, 1, 4, 8, 8, 4, 3, p, 1 << 20, None) == binding.ERR_UNSUPPORTED
    assert lib.sdwino_conv3x3_direct(p, p, None, p, 1, 4, 8, 8, 4, 2, None, 0, None) == binding.ERR_WORKSPACE
    assert lib.sdwino_conv3x3_f32(p, p, None, p, 1, 4, 8, 8, 4, 1, p, 1 << 20, None) == binding.ERR_UNSUPPORTED      # tile 1: fp16 entries only
    assert lib.sdwino_set_pipeline(3, 0, 0) == binding.ERR_INVALID_ARG
    assert lib.sdwino_set_pipeline(1, -1, 0) == binding.ERR_INVALID_ARG
    assert lib.sdwino_set_pipeline(1, 0, 0) == binding.OK
    assert lib.sdwino_profile_enable(3) == binding.ERR_INVALID_ARG and lib.sdwino_profile_enable(0) == binding.OK
    # test hooks reject values outside their range and accept the defaults
    assert lib.sdwino_set_input_staging(3) == binding.ERR_INVALID_ARG
    assert lib.sdwino_set_input_staging(-1) == binding.ERR_INVALID_ARG
    assert lib.sdwino_set_input_staging(1) == binding.OK
    assert lib.sdwino_set_gemm_shape(0, 0) == binding.OK


def test_sequence_entry_validates_every_layer_before_anything_runs(binding):
    lib, Layer = binding.lib, binding.SdwinoLayer
    buf = ctypes.create_string_buffer(4096)
    p = (ctypes.addressof(buf) + 1023) // 1024 * 1024

    def seq(*specs):
        arr = (Layer * len(specs))()
        for d, (x, wT, bias, y, N, C, H, W, K, tile) in zip(arr, specs):
            d.x, d.wT, d.bias, d.y, d.N, d.C, d.H, d.W, d.K, d.tile = x, wT, bias, y, N, C, H, W, K, tile
        return arr

    good = (p, p, None, p, 1, 4, 8, 8, 4, 2)
    big = (p, p, None, p, 2, 320, 64, 64, 320, 4)
    # workspace of a list = the largest single-pass workspace among its layers; an invalid member makes it 0
    assert lib.sdwino_workspace_bytes_sequence(seq(good, big), 2) == binding.sdwino_workspace_bytes(2, 320, 64, 64, 320, 4)
    assert lib.sdwino_workspace_bytes_sequence(seq(good), 1) == binding.sdwino_workspace_bytes(1, 4, 8, 8, 4, 2)
    assert lib.sdwino_workspace_bytes_sequence(seq(good, (p, p, None, p, 1, 4, 8, 8, 4, 3)), 2) == 0
    assert lib.sdwino_workspace_bytes_sequence(None, 1) == 0
    assert lib.sdwino_workspace_bytes_sequence(seq(good), 0) == 0
    call = lib.sdwino_conv3x3_sequence
    assert call(None, 1, p, 1 << 20, 0, None) == binding.ERR_INVALID_ARG
    assert call(seq(good), 0, p, 1 << 20, 0, None) == binding.ERR_INVALID_ARG
    # a fault in the LAST layer is found before the first one is launched (no GPU here: a launch would be ERR_CUDA)
    assert call(seq(good, (None, p, None, p, 1, 4, 8, 8, 4, 2)), 2, p, 1 << 20, 0, None) == binding.ERR_INVALID_ARG
    assert call(seq(good, (p, p, None, p, 1, 4, 8, 0, 4, 2)), 2, p, 1 << 20, 0, None) == binding.ERR_INVALID_ARG
    assert call(seq(good, (p, p, None, p, 1, 4, 8, 8, 4, 3)), 2, p, 1 << 20, 0, None) == binding.ERR_UNSUPPORTED
    assert call(seq(good, (p, p, None, p + 1, 1, 4, 8, 8, 4, 2)), 2, p, 1 << 20, 0, None) == binding.ERR_MISALIGNED
    assert call(seq(good, (p, p + 16, None, p, 1, 4, 8, 8, 4, 2)), 2, p, 1 << 20, 0, None) == binding.ERR_MISALIGNED
    assert call(seq(good, good), 2, None, 0, 0, None) == binding.ERR_WORKSPACE
    assert call(seq(good, good), 2, p, 4096, 0, None) == binding.ERR_WORKSPACE
    assert call(seq(good, good), 2, p + 8, 1 << 20, 0, None) == binding.ERR_MISALIGNED
    # the struct of the binding has the layout of the header: four pointers, six ints
    assert ctypes.sizeof(Layer) == 4 * ctypes.sizeof(ctypes.c_void_p) + 6 * ctypes.sizeof(ctypes.c_int)


def test_missing_library_fails_loudly(monkeypatch, binding):
    import importlib
    from paper_2412_05781_b200 import build as bmod
    monkeypatch.setattr(bmod, "LIB_PATH", "/nonexistent/libsdwino.so")
    import paper_2412_05781_b200.binding as bind
    monkeypatch.setattr(bind, "LIB_PATH", "/nonexistent/libsdwino.so")
    with pytest.raises(ImportError):
        bind._load()


def test_product_package_does_not_import_oracle():
    pkg = os.path.join(ROOT, "paper_2412_05781_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src and "conv_oracle" not in src, f


def test_choose_tile_is_host_arithmetic(binding):
    # few-channel layers -> F(2x2); weight-heavy layers -> F(2x2); activation-heavy layers -> F(4x4)
    assert binding.sdwino_choose_tile(2, 4, 64, 64, 320) == 2
    assert binding.sdwino_choose_tile(2, 320, 64, 64, 4) == 4      # few output channels, 2048 tiles
    assert binding.sdwino_choose_tile(1, 128, 512, 512, 3) == 2    # few output channels, 65536 tiles
    assert binding.sdwino_choose_tile(2, 1280, 8, 8, 1280) == 2
    assert binding.sdwino_choose_tile(2, 2560, 16, 16, 1280) == 2
    assert binding.sdwino_choose_tile(2, 320, 64, 64, 320) == 4
    assert binding.sdwino_choose_tile(1, 512, 256, 256, 512) == 4
    # threshold: 2 * tiles * (C + K) >= K * C with tiles = N * ceil(H/2) * ceil(W/2)
    assert binding.sdwino_choose_tile(1, 64, 7, 7, 64) == 4       # 2*16*128 = 4096 >= 4096
    assert binding.sdwino_choose_tile(1, 64, 6, 7, 64) == 2       # 2*12*128 = 3072 <  4096
    # between 0.65 and 1 of the threshold: F(4x4) only with at least 256 tiles
    assert binding.sdwino_choose_tile(2, 2560, 24, 24, 1280) == 4  # 288 tiles, ratio 0.68
    assert binding.sdwino_choose_tile(1, 640, 24, 24, 1280) == 2   # 144 tiles, ratio 0.68
    assert binding.sdwino_choose_tile(2, 640, 16, 16, 1280) == 2   # 128 tiles, ratio 0.60
    with pytest.raises(binding.SdwinoError):
        binding.sdwino_choose_tile(0, 1, 1, 1, 1)
