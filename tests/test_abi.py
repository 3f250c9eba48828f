"""Host-side checks that need no GPU: the shared library builds, loads, exports every symbol the
header declares, its pure host functions agree with the layout the oracle states, and argument
errors are reported as status codes before anything touches a device."""
import ctypes
import os
import re

import numpy as np

import oracle as O
from paper_2605_19561_b200 import torq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "torq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(torq_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = torq.lib()
    names = _declared_symbols()
    assert {"torq_rotate_quantize", "torq_mxfp4_gemm", "torq_rotated_linear", "torq_quantize_mxfp4"} <= set(names)
    for n in names:
        assert hasattr(L, n), n


def test_scale_layout_functions_match_the_oracle_statement():
    for rows, k in [(1, 32), (64, 256), (129, 4096), (2048, 14336), (200, 96)]:
        assert torq.torq_scales_bytes(rows, k) == O.scale_layout_bytes(rows, k)
    g = np.random.default_rng(0)
    for _ in range(2000):
        k = int(g.integers(1, 500)) * 32
        r = int(g.integers(0, 5000))
        c = int(g.integers(0, k // 32))
        assert torq.torq_scale_offset(r, c, k) == int(O.scale_layout_offset(r, c, k))


def test_workspace_holds_codes_and_scales():
    M, d, N = 130, 256, 64
    need = torq.torq_workspace_bytes(M, d, N)
    assert need >= M * d // 2 + torq.torq_scales_bytes(M, d)
    assert need % 256 == 0


def test_argument_errors_are_status_codes():
    L = torq.lib()
    one = ctypes.c_void_p(16)      # non-null, 16-byte aligned, never dereferenced on these paths
    odd = ctypes.c_void_p(24)
    assert L.torq_rotate_quantize(None, None, None, 4, 64, one, one, None) == 1
    assert L.torq_rotate_quantize(one, None, None, 4, 48, one, one, None) == 2      # d % 32 != 0
    assert L.torq_rotate_quantize(one, None, None, 0, 64, one, one, None) == 2      # M < 1
    assert L.torq_rotate_quantize(odd, None, None, 4, 64, one, one, None) == 3
    assert L.torq_mxfp4_gemm(one, one, one, None, 4, 8, 128, one, 0, None) == 1
    assert L.torq_mxfp4_gemm(one, one, one, one, 4, 8, 96, one, 0, None) == 2       # K % 128 != 0
    assert L.torq_mxfp4_gemm(one, one, one, one, 4, 12, 128, one, 0, None) == 2     # N % 8 != 0
    assert L.torq_mxfp4_gemm(one, one, one, one, 4, 8, 128, one, 5, None) == 2      # bad dtype
    assert L.torq_quantize_mxfp4(one, 0, 4, 64, None, one, None) == 1
    assert L.torq_quantize_mxfp4(one, 0, 4, 33, one, one, None) == 2
    assert L.torq_rotated_linear(one, one, one, one, one, 4, 128, 8, one, 0, None, 0, None, None, None) == 7
    assert L.torq_rotated_linear(one, one, one, one, one, 4, 128, 8, one, 0, one, 16, None, None, None) == 7
    assert L.torq_rotated_linear(one, one, one, one, one, 4, 96, 8, one, 0, one, 1 << 20, None, None, None) == 2
    assert L.torq_probe_fp4_peak(100, None, None) == 1
    import ctypes as _c
    assert L.torq_probe_fp4_peak(0, _c.byref(_c.c_double()), None) == 2
    assert L.torq_status_string(0) == b"ok" and L.torq_status_string(6)


def test_nvfp4_and_calibration_argument_errors_and_sizes():
    L = torq.lib()
    one = ctypes.c_void_p(16)
    odd = ctypes.c_void_p(24)
    # sizes: 16-element blocks -> twice the scale bytes of the 32-element layout for the same K
    for rows, k in [(1, 64), (64, 256), (129, 4096), (200, 96)]:
        assert torq.torq_nvfp4_scales_bytes(rows, k) == O.nv_scale_layout_bytes(rows, k)
    assert torq.torq_nvfp4_scales_bytes(128, 4096) == 2 * torq.torq_scales_bytes(128, 4096)
    assert torq.torq_nvfp4_workspace_bytes(2048, 4096, 6144) >= 2048 * 2048 + torq.torq_nvfp4_scales_bytes(2048, 4096)
    # few tokens: room for the fp32 partials of the split rotation as well
    assert torq.torq_nvfp4_workspace_bytes(16, 4096, 6144) > 16 * 2048 + torq.torq_nvfp4_scales_bytes(16, 4096) + 4 * 128 * 4096
    assert L.torq_quantize_nvfp4(one, 0, 4, 64, 1.0, None, one, None) == 1
    assert L.torq_quantize_nvfp4(one, 0, 4, 24, 1.0, one, one, None) == 2            # d % 16 != 0
    assert L.torq_quantize_nvfp4(one, 0, 4, 64, 0.0, one, one, None) == 2            # tensor scale must be > 0
    assert L.torq_quantize_nvfp4(one, 0, 4, 64, float("inf"), one, one, None) == 2
    assert L.torq_quantize_nvfp4(odd, 0, 4, 64, 1.0, one, one, None) == 3
    assert L.torq_rotate_quantize_nvfp4(one, None, None, 4, 64, 1.0, one, one, None) == 1    # R_inter is required
    assert L.torq_rotate_quantize_nvfp4(one, one, None, 4, 64, -1.0, one, one, None) == 2
    assert L.torq_nvfp4_gemm(one, one, 1.0, one, one, 1.0, 4, 8, 96, one, 0, None) == 2     # K % 128 != 0
    assert L.torq_nvfp4_gemm(one, one, 0.0, one, one, 1.0, 4, 8, 128, one, 0, None) == 2
    assert L.torq_nvfp4_gemm(one, None, 1.0, one, one, 1.0, 4, 8, 128, one, 0, None) == 1
    assert L.torq_rotated_linear_nvfp4(one, one, one, 1.0, one, one, 1.0, 4, 128, 8, one, 0, one, 16, None, None,
                                       None) == 7
    assert L.torq_expand_intra16(None, 64, one, None) == 1
    assert L.torq_expand_intra16(one, 48, one, None) == 2
    assert L.torq_block_covariance(one, 4, 48, one, None) == 2
    assert L.torq_block_covariance(None, 4, 64, one, None) == 1
    assert L.torq_givens_equalize(one, 0, 1e-9, one, None, None, None) == 2
    assert L.torq_givens_equalize(one, 8, -1.0, one, None, None, None) == 2
    assert L.torq_givens_equalize(None, 8, 1e-9, one, None, None, None) == 1


def test_mxint4_argument_errors_and_sizes():
    L = torq.lib()
    one = ctypes.c_void_p(16)
    odd = ctypes.c_void_p(24)
    # operand form: one byte per element, plus the 32-block scale tiles
    assert torq.torq_mxint4_workspace_bytes(2048, 4096, 6144) == 2048 * 4096 + torq.torq_scales_bytes(2048, 4096)
    assert torq.torq_mxint4_workspace_bytes(0, 4096, 8) == 0
    assert L.torq_quantize_mxint4(one, 0, 4, 64, 0, None, one, None) == 1
    assert L.torq_quantize_mxint4(one, 0, 4, 48, 1, one, one, None) == 2              # d % 32 != 0
    assert L.torq_quantize_mxint4(odd, 0, 4, 64, 1, one, one, None) == 3
    assert L.torq_mxint4_expand(None, 4, 64, one, None) == 1
    assert L.torq_mxint4_expand(one, 4, 40, one, None) == 2
    assert L.torq_rotate_quantize_mxint4(one, None, None, 4, 64, one, one, None) == 1         # R_inter is required
    assert L.torq_rotate_quantize_mxint4(one, one, None, 4, 48, one, one, None) == 2
    assert L.torq_mxint4_gemm(one, one, one, one, 4, 8, 96, one, 0, None) == 2               # K % 128 != 0
    assert L.torq_rotate_quantize_structured_mxint4(one, None, None, 4, 256, one, one, None) == 1
    assert L.torq_rotate_quantize_structured_mxint4(one, one, None, 4, 96, one, one, None) == 2   # d % 256 != 0
    assert L.torq_mxint4_gemm(one, None, one, one, 4, 8, 128, one, 0, None) == 1
    assert L.torq_mxint4_gemm(one, one, odd, one, 4, 8, 128, one, 0, None) == 3
    assert L.torq_rotated_linear_mxint4(one, one, one, one, one, 4, 128, 8, one, 0, one, 16, None, None, None) == 7
    assert L.torq_rotated_linear_mxint4(one, None, one, one, one, 4, 128, 8, one, 0, one, 1 << 20, None, None,
                                        None) == 1


def test_probe_argument_errors():
    L = torq.lib()
    one = ctypes.c_void_p(16)
    d = ctypes.c_double(0.0)
    assert L.torq_probe_fp4_peak(100, None, None) == 1
    assert L.torq_probe_fp4_peak(0, ctypes.byref(d), None) == 2


def test_pair_tile_list_covers_every_output_exactly_once():
    """Host logic of the CTA-pair kernels' tile list: whatever the planner trades, the tiles partition the
    [row tiles x cols] output, narrow tiles start on a multiple of 64 columns (two 32-blocks: the scale bytes
    of a block pair never straddle two tiles), and the longest pair never gets longer than with 256-column
    tiles alone."""
    import numpy as np
    shapes = [(2048, 4096), (2048, 6144), (2048, 14336), (1024, 5120), (16384, 5120), (8192, 51200), (300, 256),
              (129, 4096), (4864, 1024), (3840, 1280), (2560, 2048), (2500, 2048), (2048, 4000), (640, 768),
              (19 * 256, 1024), (75 * 256, 256), (74 * 256 + 1, 512)]
    for pairs in (74, 66, 8):
        for rows, cols in shapes:
            tl = torq.torq_pair_tile_list(rows, cols, pairs)
            rt = (rows + 255) // 256
            cover = np.zeros((rt, (cols + 31) // 32), np.int32)
            for mp, c0, w in tl:
                assert 0 <= mp < rt and w in (192, 256) and c0 % 64 == 0 and c0 < cols
                assert w == 256 or (cols % 256 == 0 and c0 + w <= cols)
                cover[mp, c0 // 32:min(cols, c0 + w + 31) // 32 if c0 + w < cols else cover.shape[1]] += 1
            assert (cover == 1).all(), (pairs, rows, cols)
            # wide tiles are dealt before narrow ones
            widths = [w for _, _, w in tl]
            assert widths == sorted(widths, reverse=True)
            load = np.zeros(pairs)
            for i, w in enumerate(widths):
                load[i % pairs] += w / 256.0
            wide_only = -(-(rt * ((cols + 255) // 256)) // pairs)
            assert load.max() <= wide_only + 1e-9
    # the LLaMA3-8B QKV rotation on 74 pairs: one wave of 74 wide tiles, then 72 narrow ones
    tl = torq.torq_pair_tile_list(2048, 4096, 74)
    assert [w for _, _, w in tl].count(256) == 74 and [w for _, _, w in tl].count(192) == 72
    assert torq.lib().torq_pair_tile_list(0, 4096, 74, None, 0) == -1
