"""Thin ctypes binding over the C-ABI library (include/torq.h).  Argument marshalling only:
every step of the path runs in the CUDA kernels; PyTorch provides device memory and streams.
There is no fallback: a missing library or a non-zero status raises."""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

TORQ_F32, TORQ_BF16 = 0, 1
_STATUS = {0: "TORQ_OK", 1: "TORQ_ERR_NULL", 2: "TORQ_ERR_SHAPE", 3: "TORQ_ERR_ALIGN", 4: "TORQ_ERR_ARCH",
           5: "TORQ_ERR_LAUNCH", 6: "TORQ_ERR_TIMEOUT", 7: "TORQ_ERR_WORKSPACE"}
_lib_handle = None


class TorqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {_STATUS.get(code, code)}")


def lib() -> ctypes.CDLL:
    """Loads (building first if the binary is absent or stale and nvcc is available)."""
    global _lib_handle
    if _lib_handle is not None:
        return _lib_handle
    path = _build.LIB_PATH
    if _build.needs_build():
        _build.build_library()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing; run paper_2605_19561_b200/build.py")
    L = ctypes.CDLL(path)
    vp, i64, sz, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t, ctypes.c_int
    L.torq_rotate_quantize.argtypes = [vp, vp, vp, i64, i64, vp, vp, vp]
    L.torq_rotate_quantize.restype = ci
    L.torq_rotate_quantize_structured.argtypes = [vp, vp, vp, i64, i64, vp, vp, vp]
    L.torq_rotate_quantize_structured.restype = ci
    L.torq_rotated_linear_structured.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, vp, ci, vp, sz, vp, vp, vp]
    L.torq_rotated_linear_structured.restype = ci
    L.torq_mxfp4_gemm.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp, ci, vp]
    L.torq_mxfp4_gemm.restype = ci
    L.torq_rotated_linear.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, vp, ci, vp, sz, vp, vp, vp]
    L.torq_rotated_linear.restype = ci
    L.torq_rotated_linear_static.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, vp, ci, vp]
    L.torq_rotated_linear_static.restype = ci
    L.torq_quantize_mxfp4.argtypes = [vp, ci, i64, i64, vp, vp, vp]
    L.torq_quantize_mxfp4.restype = ci
    L.torq_scales_bytes.argtypes = [i64, i64]
    L.torq_scales_bytes.restype = sz
    L.torq_scale_offset.argtypes = [i64, i64, i64]
    L.torq_scale_offset.restype = sz
    L.torq_workspace_bytes.argtypes = [i64, i64, i64]
    L.torq_workspace_bytes.restype = sz
    L.torq_swizzle_scales.argtypes = [vp, i64, i64, vp, vp]
    L.torq_swizzle_scales.restype = ci
    L.torq_merge_rotations.argtypes = [vp, vp, i64, vp, vp]
    L.torq_merge_rotations.restype = ci
    f32 = ctypes.c_float
    L.torq_merge_rotations_bf16.argtypes = [vp, vp, i64, vp, vp]
    L.torq_merge_rotations_bf16.restype = ci
    L.torq_prepare_weights_workspace_bytes.argtypes = [i64, i64]
    L.torq_prepare_weights_workspace_bytes.restype = sz
    L.torq_prepare_weights.argtypes = [vp, vp, vp, i64, i64, vp, vp, vp, sz, vp]
    L.torq_prepare_weights.restype = ci
    L.torq_prepare_weights_nvfp4.argtypes = [vp, vp, vp, i64, i64, vp, vp, ctypes.POINTER(ctypes.c_float), vp, sz, vp]
    L.torq_prepare_weights_nvfp4.restype = ci
    L.torq_prepare_weights_mxint4.argtypes = [vp, vp, vp, i64, i64, vp, vp, vp, vp, sz, vp]
    L.torq_prepare_weights_mxint4.restype = ci
    L.torq_nvfp4_scales_bytes.argtypes = [i64, i64]
    L.torq_nvfp4_scales_bytes.restype = sz
    L.torq_nvfp4_workspace_bytes.argtypes = [i64, i64, i64]
    L.torq_nvfp4_workspace_bytes.restype = sz
    L.torq_expand_intra16.argtypes = [vp, i64, vp, vp]
    L.torq_expand_intra16.restype = ci
    L.torq_quantize_nvfp4.argtypes = [vp, ci, i64, i64, f32, vp, vp, vp]
    L.torq_quantize_nvfp4.restype = ci
    L.torq_rotate_quantize_nvfp4.argtypes = [vp, vp, vp, i64, i64, f32, vp, vp, vp]
    L.torq_rotate_quantize_nvfp4.restype = ci
    L.torq_rotate_quantize_structured_nvfp4.argtypes = [vp, vp, vp, i64, i64, f32, vp, vp, vp]
    L.torq_rotate_quantize_structured_nvfp4.restype = ci
    L.torq_nvfp4_gemm.argtypes = [vp, vp, f32, vp, vp, f32, i64, i64, i64, vp, ci, vp]
    L.torq_nvfp4_gemm.restype = ci
    L.torq_rotated_linear_nvfp4.argtypes = [vp, vp, vp, f32, vp, vp, f32, i64, i64, i64, vp, ci, vp, sz, vp, vp, vp]
    L.torq_rotated_linear_nvfp4.restype = ci
    L.torq_mxint4_workspace_bytes.argtypes = [i64, i64, i64]
    L.torq_mxint4_workspace_bytes.restype = sz
    L.torq_quantize_mxint4.argtypes = [vp, ci, i64, i64, ci, vp, vp, vp]
    L.torq_quantize_mxint4.restype = ci
    L.torq_mxint4_expand.argtypes = [vp, i64, i64, vp, vp]
    L.torq_mxint4_expand.restype = ci
    L.torq_rotate_quantize_mxint4.argtypes = [vp, vp, vp, i64, i64, vp, vp, vp]
    L.torq_rotate_quantize_mxint4.restype = ci
    L.torq_rotate_quantize_structured_mxint4.argtypes = [vp, vp, vp, i64, i64, vp, vp, vp]
    L.torq_rotate_quantize_structured_mxint4.restype = ci
    L.torq_mxint4_gemm.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp, ci, vp]
    L.torq_mxint4_gemm.restype = ci
    L.torq_rotated_linear_mxint4.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, vp, ci, vp, sz, vp, vp, vp]
    L.torq_rotated_linear_mxint4.restype = ci
    L.torq_block_covariance.argtypes = [vp, i64, i64, vp, vp]
    L.torq_block_covariance.restype = ci
    L.torq_givens_equalize.argtypes = [vp, i64, ctypes.c_double, vp, vp, vp, vp]
    L.torq_givens_equalize.restype = ci
    L.torq_probe_fp4_peak.argtypes = [ci, ctypes.POINTER(ctypes.c_double), vp]
    L.torq_probe_fp4_peak.restype = ci
    L.torq_selftest_wait_timeout.argtypes = [ctypes.c_uint64, vp, vp]
    L.torq_selftest_wait_timeout.restype = ci
    L.torq_status_string.argtypes = [ci]
    L.torq_status_string.restype = ctypes.c_char_p
    L.torq_last_device_error.argtypes = [vp]
    L.torq_last_device_error.restype = ci
    L.torq_pair_tile_list.argtypes = [i64, i64, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32), i64]
    L.torq_pair_tile_list.restype = i64
    L.torq_launch_count.argtypes = []
    L.torq_launch_count.restype = i64
    _lib_handle = L
    return L


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(t, dtype, name):
    if t is None:
        return
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise ValueError(f"{name}: expected a contiguous CUDA tensor of {dtype}, got {t.dtype} on {t.device}")


def _raise(code, where):
    if code != 0:
        raise TorqError(code, where)


def torq_scales_bytes(rows: int, k: int) -> int:
    return lib().torq_scales_bytes(rows, k)


def torq_scale_offset(row: int, kblock: int, k: int) -> int:
    return lib().torq_scale_offset(row, kblock, k)


def torq_workspace_bytes(M: int, d: int, N: int) -> int:
    return lib().torq_workspace_bytes(M, d, N)


def torq_pair_tile_list(rows: int, cols: int, pairs: int = 74):
    """[(row_tile, first_column, width), ...] in dealing order (host helper, no device work)."""
    n = lib().torq_pair_tile_list(rows, cols, pairs, None, 0)
    if n < 0:
        raise ValueError("torq_pair_tile_list: rows, cols and pairs must be positive")
    buf = (ctypes.c_int32 * (3 * n))()
    lib().torq_pair_tile_list(rows, cols, pairs, buf, n)
    return [(buf[3 * i], buf[3 * i + 1], buf[3 * i + 2]) for i in range(n)]


def torq_launch_count() -> int:
    return lib().torq_launch_count()


def torq_last_device_error(stream=None) -> int:
    return lib().torq_last_device_error(_stream(stream))


def torq_quantize_mxfp4(Z, out_codes=None, out_scales=None, stream=None):
    """Z [M,d] float32 or bfloat16 -> (codes [M,d/2] uint8, tiled scale bytes uint8)."""
    M, d = Z.shape
    dt = TORQ_F32 if Z.dtype == torch.float32 else TORQ_BF16
    _check(Z, torch.float32 if dt == TORQ_F32 else torch.bfloat16, "Z")
    if out_codes is None:
        out_codes = torch.empty((M, d // 2), dtype=torch.uint8, device=Z.device)
    if out_scales is None:
        out_scales = torch.empty(torq_scales_bytes(M, d), dtype=torch.uint8, device=Z.device)
    _raise(lib().torq_quantize_mxfp4(_ptr(Z), dt, M, d, _ptr(out_codes), _ptr(out_scales), _stream(stream)),
           "torq_quantize_mxfp4")
    return out_codes, out_scales


def torq_rotate_quantize(X, R_inter, R_intra, out_codes=None, out_scales=None, stream=None):
    """X [M,d] bf16, R_inter [d,d] bf16 or None, R_intra [d/32,32,32] bf16 or None."""
    M, d = X.shape
    for t, n in ((X, "X"), (R_inter, "R_inter"), (R_intra, "R_intra")):
        _check(t, torch.bfloat16, n)
    if out_codes is None:
        out_codes = torch.empty((M, d // 2), dtype=torch.uint8, device=X.device)
    if out_scales is None:
        out_scales = torch.empty(torq_scales_bytes(M, d), dtype=torch.uint8, device=X.device)
    _raise(lib().torq_rotate_quantize(_ptr(X), _ptr(R_inter), _ptr(R_intra), M, d, _ptr(out_codes),
                                      _ptr(out_scales), _stream(stream)), "torq_rotate_quantize")
    return out_codes, out_scales


def torq_rotate_quantize_structured(X, R_B, R_intra, out_codes=None, out_scales=None, stream=None):
    """X [M,d] bf16, R_B [d/32,d/32] bf16 (mixes the blocks of a token), R_intra [32,32] bf16 or None
    (shared by all blocks): the rotation in the structure the paper gives it."""
    M, d = X.shape
    for t, n in ((X, "X"), (R_B, "R_B"), (R_intra, "R_intra")):
        _check(t, torch.bfloat16, n)
    if out_codes is None:
        out_codes = torch.empty((M, d // 2), dtype=torch.uint8, device=X.device)
    if out_scales is None:
        out_scales = torch.empty(torq_scales_bytes(M, d), dtype=torch.uint8, device=X.device)
    _raise(lib().torq_rotate_quantize_structured(_ptr(X), _ptr(R_B), _ptr(R_intra), M, d, _ptr(out_codes),
                                                 _ptr(out_scales), _stream(stream)), "torq_rotate_quantize_structured")
    return out_codes, out_scales


def torq_mxfp4_gemm(Aq, As, Wq, Ws, out_dtype=torch.bfloat16, Y=None, stream=None):
    """Aq [M,K/2], Wq [N,K/2] uint8 codes; As, Ws tiled scale bytes -> Y [M,N]."""
    M, K2 = Aq.shape
    N = Wq.shape[0]
    for t, n in ((Aq, "Aq"), (As, "As"), (Wq, "Wq"), (Ws, "Ws")):
        _check(t, torch.uint8, n)
    if Y is None:
        Y = torch.empty((M, N), dtype=out_dtype, device=Aq.device)
    _check(Y, Y.dtype, "Y")
    dt = TORQ_F32 if Y.dtype == torch.float32 else TORQ_BF16
    _raise(lib().torq_mxfp4_gemm(_ptr(Aq), _ptr(As), _ptr(Wq), _ptr(Ws), M, N, 2 * K2, _ptr(Y), dt,
                                 _stream(stream)), "torq_mxfp4_gemm")
    return Y


def torq_rotated_linear(X, R_inter, R_intra, Wq, Ws, out_dtype=torch.bfloat16, Y=None, workspace=None,
                        dbg_codes=None, dbg_scales=None, stream=None):
    """Rotate, quantize and multiply in one call.  Returns Y [M,N]."""
    M, d = X.shape
    N = Wq.shape[0]
    for t, n in ((X, "X"), (R_inter, "R_inter"), (R_intra, "R_intra")):
        _check(t, torch.bfloat16, n)
    for t, n in ((Wq, "Wq"), (Ws, "Ws"), (dbg_codes, "dbg_codes"), (dbg_scales, "dbg_scales")):
        _check(t, torch.uint8, n)
    if Y is None:
        Y = torch.empty((M, N), dtype=out_dtype, device=X.device)
    if workspace is None:
        workspace = torch.empty(torq_workspace_bytes(M, d, N), dtype=torch.uint8, device=X.device)
    dt = TORQ_F32 if Y.dtype == torch.float32 else TORQ_BF16
    _raise(lib().torq_rotated_linear(_ptr(X), _ptr(R_inter), _ptr(R_intra), _ptr(Wq), _ptr(Ws), M, d, N,
                                     _ptr(Y), dt, _ptr(workspace), workspace.numel(), _ptr(dbg_codes),
                                     _ptr(dbg_scales), _stream(stream)), "torq_rotated_linear")
    return Y


def torq_rotated_linear_structured(X, R_B, R_intra, Wq, Ws, out_dtype=torch.bfloat16, Y=None, workspace=None,
                                   dbg_codes=None, dbg_scales=None, stream=None):
    """The whole layer with the rotation in the paper's structure (R_B [d/32,d/32], shared R_intra [32,32])."""
    M, d = X.shape
    N = Wq.shape[0]
    for t, n in ((X, "X"), (R_B, "R_B"), (R_intra, "R_intra")):
        _check(t, torch.bfloat16, n)
    for t, n in ((Wq, "Wq"), (Ws, "Ws"), (dbg_codes, "dbg_codes"), (dbg_scales, "dbg_scales")):
        _check(t, torch.uint8, n)
    if Y is None:
        Y = torch.empty((M, N), dtype=out_dtype, device=X.device)
    if workspace is None:
        workspace = torch.empty(torq_workspace_bytes(M, d, N), dtype=torch.uint8, device=X.device)
    dt = TORQ_F32 if Y.dtype == torch.float32 else TORQ_BF16
    _raise(lib().torq_rotated_linear_structured(_ptr(X), _ptr(R_B), _ptr(R_intra), _ptr(Wq), _ptr(Ws), M, d, N,
                                                _ptr(Y), dt, _ptr(workspace), workspace.numel(), _ptr(dbg_codes),
                                                _ptr(dbg_scales), _stream(stream)), "torq_rotated_linear_structured")
    return Y


TORQ_STATIC_WORKSPACE_BYTES = 16 << 20


def torq_rotated_linear_static(X, R_inter, R_intra, Wq, Ws, Y, stream=None):
    """The whole layer for callers that cannot allocate device memory (a plug-in that only gets
    input and output pointers, a server whose memory is already committed to other pools, a
    decode loop that cannot afford the synchronisation an allocation implies).  The scratch for
    the quantized activations is a fixed array inside the library, TORQ_STATIC_WORKSPACE_BYTES
    long, shared by every call on the device; Y must be passed in, and this wrapper creates no
    tensor either.  Raises TorqError(TORQ_ERR_WORKSPACE) when the problem needs more scratch than
    the array holds.  Calls that may overlap on the GPU race on the array: keep them in one
    stream.  Make the first call on a device during start-up (it looks up the array's address)."""
    M, d = X.shape
    N = Wq.shape[0]
    for t, n in ((X, "X"), (R_inter, "R_inter"), (R_intra, "R_intra")):
        _check(t, torch.bfloat16, n)
    for t, n in ((Wq, "Wq"), (Ws, "Ws")):
        _check(t, torch.uint8, n)
    _check(Y, Y.dtype, "Y")
    dt = TORQ_F32 if Y.dtype == torch.float32 else TORQ_BF16
    _raise(lib().torq_rotated_linear_static(_ptr(X), _ptr(R_inter), _ptr(R_intra), _ptr(Wq), _ptr(Ws), M, d, N,
                                            _ptr(Y), dt, _stream(stream)), "torq_rotated_linear_static")
    return Y


def torq_probe_fp4_peak(groups: int = 40000, stream=None) -> float:
    """Issue-bound rate (TFLOP/s) of the block-scaled FP4 tensor-core instruction on this device."""
    out = ctypes.c_double(0.0)
    _raise(lib().torq_probe_fp4_peak(groups, ctypes.byref(out), _stream(stream)), "torq_probe_fp4_peak")
    return out.value


def torq_selftest_wait_timeout(limit_ns: int = 1_000_000, stream=None):
    """Runs the give-up path of the bounded device waits once, harmlessly (see torq.h).  Returns a
    device int64 tensor [gave_up, left_through_abort_flag, waited_ns]."""
    out = torch.zeros(4, dtype=torch.int64, device="cuda")
    _raise(lib().torq_selftest_wait_timeout(int(limit_ns), _ptr(out), _stream(stream)), "torq_selftest_wait_timeout")
    return out[:3]


def torq_swizzle_scales(linear, k: int, out=None, stream=None):
    rows = linear.shape[0]
    _check(linear, torch.uint8, "linear")
    if out is None:
        out = torch.empty(torq_scales_bytes(rows, k), dtype=torch.uint8, device=linear.device)
    _raise(lib().torq_swizzle_scales(_ptr(linear), rows, k, _ptr(out), _stream(stream)), "torq_swizzle_scales")
    return out


def torq_merge_rotations(R_inter, R_intra, out=None, stream=None):
    d = R_inter.shape[0]
    _check(R_inter, torch.bfloat16, "R_inter")
    _check(R_intra, torch.bfloat16, "R_intra")
    if out is None:
        out = torch.empty((d, d), dtype=torch.float32, device=R_inter.device)
    _raise(lib().torq_merge_rotations(_ptr(R_inter), _ptr(R_intra), d, _ptr(out), _stream(stream)),
           "torq_merge_rotations")
    return out


def torq_merge_rotations_bf16(R_inter, R_intra, out=None, stream=None):
    """R~ = R_inter blockdiag(R_intra) rounded once to bfloat16: the operand of the one-GEMM form of the rotation."""
    d = R_inter.shape[0]
    _check(R_inter, torch.bfloat16, "R_inter")
    _check(R_intra, torch.bfloat16, "R_intra")
    if out is None:
        out = torch.empty((d, d), dtype=torch.bfloat16, device=R_inter.device)
    _raise(lib().torq_merge_rotations_bf16(_ptr(R_inter), _ptr(R_intra), d, _ptr(out), _stream(stream)),
           "torq_merge_rotations_bf16")
    return out


def torq_prepare_weights_workspace_bytes(d: int, N: int) -> int:
    return int(lib().torq_prepare_weights_workspace_bytes(d, N))


def _prep_args(R_inter, R_intra, W, workspace):
    _check(W, torch.float32, "W")
    _check(R_inter, torch.bfloat16, "R_inter")
    _check(R_intra, torch.bfloat16, "R_intra")
    d, N = W.shape
    if workspace is None:
        workspace = torch.empty(torq_prepare_weights_workspace_bytes(d, N), dtype=torch.uint8, device=W.device)
    return d, N, workspace


def torq_prepare_weights(R_inter, R_intra, W, workspace=None, stream=None):
    """Offline weight side of the layer: W [d,N] float32 -> (Wq [N,d/2], Ws tiled), W' = R~^T W quantized
    to MXFP4 along K, all of it by the library's kernels."""
    d, N, workspace = _prep_args(R_inter, R_intra, W, workspace)
    Wq = torch.empty((N, d // 2), dtype=torch.uint8, device=W.device)
    Ws = torch.empty(torq_scales_bytes(N, d), dtype=torch.uint8, device=W.device)
    _raise(lib().torq_prepare_weights(_ptr(W), _ptr(R_inter), _ptr(R_intra), d, N, _ptr(Wq), _ptr(Ws),
                                      _ptr(workspace), workspace.numel(), _stream(stream)), "torq_prepare_weights")
    return Wq, Ws


prepare_weights = torq_prepare_weights


# ---- NVFP4 variant (16-element blocks, E4M3 block scales, float32 tensor scale) -----------------------
def torq_nvfp4_scales_bytes(rows: int, k: int) -> int:
    return lib().torq_nvfp4_scales_bytes(rows, k)


def torq_nvfp4_workspace_bytes(M: int, d: int, N: int) -> int:
    return lib().torq_nvfp4_workspace_bytes(M, d, N)


def torq_expand_intra16(R_intra16, out=None, stream=None):
    """[d/16,16,16] bf16 -> the 32-wide block-diagonal form [d/32,32,32] the rotation kernels take."""
    _check(R_intra16, torch.bfloat16, "R_intra16")
    d = R_intra16.shape[0] * 16
    if out is None:
        out = torch.empty((d // 32, 32, 32), dtype=torch.bfloat16, device=R_intra16.device)
    _raise(lib().torq_expand_intra16(_ptr(R_intra16), d, _ptr(out), _stream(stream)), "torq_expand_intra16")
    return out


def torq_quantize_nvfp4(Z, tensor_scale: float, out_codes=None, out_scales=None, stream=None):
    """Z [M,d] float32 or bfloat16 -> (codes [M,d/2] uint8, tiled E4M3 scale bytes uint8)."""
    M, d = Z.shape
    dt = TORQ_F32 if Z.dtype == torch.float32 else TORQ_BF16
    _check(Z, torch.float32 if dt == TORQ_F32 else torch.bfloat16, "Z")
    if out_codes is None:
        out_codes = torch.empty((M, d // 2), dtype=torch.uint8, device=Z.device)
    if out_scales is None:
        out_scales = torch.empty(torq_nvfp4_scales_bytes(M, d), dtype=torch.uint8, device=Z.device)
    _raise(lib().torq_quantize_nvfp4(_ptr(Z), dt, M, d, tensor_scale, _ptr(out_codes), _ptr(out_scales),
                                     _stream(stream)), "torq_quantize_nvfp4")
    return out_codes, out_scales


def torq_rotate_quantize_nvfp4(X, R_inter, R_intra32, tensor_scale: float, out_codes=None, out_scales=None,
                               stream=None):
    """X [M,d] bf16, R_inter [d,d] bf16, R_intra32 [d/32,32,32] bf16 or None (see torq_expand_intra16)."""
    M, d = X.shape
    for t, n in ((X, "X"), (R_inter, "R_inter"), (R_intra32, "R_intra32")):
        _check(t, torch.bfloat16, n)
    if out_codes is None:
        out_codes = torch.empty((M, d // 2), dtype=torch.uint8, device=X.device)
    if out_scales is None:
        out_scales = torch.empty(torq_nvfp4_scales_bytes(M, d), dtype=torch.uint8, device=X.device)
    _raise(lib().torq_rotate_quantize_nvfp4(_ptr(X), _ptr(R_inter), _ptr(R_intra32), M, d, tensor_scale,
                                            _ptr(out_codes), _ptr(out_scales), _stream(stream)),
           "torq_rotate_quantize_nvfp4")
    return out_codes, out_scales


def torq_nvfp4_gemm(Aq, As, a_tensor_scale: float, Wq, Ws, w_tensor_scale: float, out_dtype=torch.bfloat16, Y=None,
                    stream=None):
    """Aq [M,K/2], Wq [N,K/2] uint8 codes; As, Ws tiled E4M3 scale bytes -> Y [M,N]."""
    M, K2 = Aq.shape
    N = Wq.shape[0]
    for t, n in ((Aq, "Aq"), (As, "As"), (Wq, "Wq"), (Ws, "Ws")):
        _check(t, torch.uint8, n)
    if Y is None:
        Y = torch.empty((M, N), dtype=out_dtype, device=Aq.device)
    _check(Y, Y.dtype, "Y")
    dt = TORQ_F32 if Y.dtype == torch.float32 else TORQ_BF16
    _raise(lib().torq_nvfp4_gemm(_ptr(Aq), _ptr(As), a_tensor_scale, _ptr(Wq), _ptr(Ws), w_tensor_scale, M, N,
                                 2 * K2, _ptr(Y), dt, _stream(stream)), "torq_nvfp4_gemm")
    return Y


def torq_rotated_linear_nvfp4(X, R_inter, R_intra32, x_tensor_scale: float, Wq, Ws, w_tensor_scale: float,
                              out_dtype=torch.bfloat16, Y=None, workspace=None, dbg_codes=None, dbg_scales=None,
                              stream=None):
    """Rotate, quantize to NVFP4 and multiply in one call.  Returns Y [M,N]."""
    M, d = X.shape
    N = Wq.shape[0]
    for t, n in ((X, "X"), (R_inter, "R_inter"), (R_intra32, "R_intra32")):
        _check(t, torch.bfloat16, n)
    for t, n in ((Wq, "Wq"), (Ws, "Ws"), (dbg_codes, "dbg_codes"), (dbg_scales, "dbg_scales")):
        _check(t, torch.uint8, n)
    if Y is None:
        Y = torch.empty((M, N), dtype=out_dtype, device=X.device)
    if workspace is None:
        workspace = torch.empty(torq_nvfp4_workspace_bytes(M, d, N), dtype=torch.uint8, device=X.device)
    dt = TORQ_F32 if Y.dtype == torch.float32 else TORQ_BF16
    _raise(lib().torq_rotated_linear_nvfp4(_ptr(X), _ptr(R_inter), _ptr(R_intra32), x_tensor_scale, _ptr(Wq),
                                           _ptr(Ws), w_tensor_scale, M, d, N, _ptr(Y), dt, _ptr(workspace),
                                           workspace.numel(), _ptr(dbg_codes), _ptr(dbg_scales), _stream(stream)),
           "torq_rotated_linear_nvfp4")
    return Y


def torq_prepare_weights_nvfp4(R_inter, R_intra32, W, workspace=None, stream=None):
    """Offline weight side in NVFP4: returns (Wq [N,d/2], Ws tiled, tensor_scale = max|W'| / (6 * 448)).
    Synchronises the stream once (the tensor scale comes back to the host)."""
    d, N, workspace = _prep_args(R_inter, R_intra32, W, workspace)
    Wq = torch.empty((N, d // 2), dtype=torch.uint8, device=W.device)
    Ws = torch.empty(torq_nvfp4_scales_bytes(N, d), dtype=torch.uint8, device=W.device)
    ts = ctypes.c_float(0.0)
    _raise(lib().torq_prepare_weights_nvfp4(_ptr(W), _ptr(R_inter), _ptr(R_intra32), d, N, _ptr(Wq), _ptr(Ws),
                                            ctypes.byref(ts), _ptr(workspace), workspace.numel(), _stream(stream)),
           "torq_prepare_weights_nvfp4")
    return Wq, Ws, ts.value


prepare_weights_nvfp4 = torq_prepare_weights_nvfp4


# ---- MXINT4 variant (format study of Section 6) ---------------------------------------------------------
def torq_mxint4_workspace_bytes(M: int, d: int, N: int) -> int:
    return int(lib().torq_mxint4_workspace_bytes(M, d, N))


def torq_quantize_mxint4(Z, packed: bool = False, out_codes=None, out_scales=None, stream=None):
    """Z [M,d] float32 or bfloat16 -> (codes, tiled E8M0 scale bytes).  packed: [M,d/2] two's-complement
    nibbles (stored form); otherwise [M,d] E4M3 bytes whose values are the integer codes (operand form)."""
    M, d = Z.shape
    dt = TORQ_F32 if Z.dtype == torch.float32 else TORQ_BF16
    _check(Z, torch.float32 if dt == TORQ_F32 else torch.bfloat16, "Z")
    if out_codes is None:
        out_codes = torch.empty((M, d // 2 if packed else d), dtype=torch.uint8, device=Z.device)
    if out_scales is None:
        out_scales = torch.empty(torq_scales_bytes(M, d), dtype=torch.uint8, device=Z.device)
    _check(out_codes, torch.uint8, "out_codes")
    _check(out_scales, torch.uint8, "out_scales")
    _raise(lib().torq_quantize_mxint4(_ptr(Z), dt, M, d, 1 if packed else 0, _ptr(out_codes), _ptr(out_scales),
                                      _stream(stream)), "torq_quantize_mxint4")
    return out_codes, out_scales


def torq_mxint4_expand(packed, out=None, stream=None):
    """Stored form [rows,k/2] -> operand form [rows,k]."""
    _check(packed, torch.uint8, "packed")
    rows, k2 = packed.shape
    if out is None:
        out = torch.empty((rows, 2 * k2), dtype=torch.uint8, device=packed.device)
    _check(out, torch.uint8, "out")
    _raise(lib().torq_mxint4_expand(_ptr(packed), rows, 2 * k2, _ptr(out), _stream(stream)), "torq_mxint4_expand")
    return out


def torq_rotate_quantize_mxint4(X, R_inter, R_intra, out_bytes=None, out_scales=None, stream=None):
    """X [M,d] bf16, R_inter [d,d] bf16, R_intra [d/32,32,32] bf16 or None -> (operand bytes [M,d], scales)."""
    M, d = X.shape
    for t, n in ((X, "X"), (R_inter, "R_inter"), (R_intra, "R_intra")):
        _check(t, torch.bfloat16, n)
    if out_bytes is None:
        out_bytes = torch.empty((M, d), dtype=torch.uint8, device=X.device)
    if out_scales is None:
        out_scales = torch.empty(torq_scales_bytes(M, d), dtype=torch.uint8, device=X.device)
    _raise(lib().torq_rotate_quantize_mxint4(_ptr(X), _ptr(R_inter), _ptr(R_intra), M, d, _ptr(out_bytes),
                                             _ptr(out_scales), _stream(stream)), "torq_rotate_quantize_mxint4")
    return out_bytes, out_scales


def torq_rotate_quantize_structured_mxint4(X, R_B, R_intra, out_bytes=None, out_scales=None, stream=None):
    """The structured rotation (R_B [d/32,d/32], shared R_intra [32,32] or None) followed by the MXINT4 quantizer."""
    M, d = X.shape
    for t, n in ((X, "X"), (R_B, "R_B"), (R_intra, "R_intra")):
        _check(t, torch.bfloat16, n)
    if out_bytes is None:
        out_bytes = torch.empty((M, d), dtype=torch.uint8, device=X.device)
    if out_scales is None:
        out_scales = torch.empty(torq_scales_bytes(M, d), dtype=torch.uint8, device=X.device)
    _raise(lib().torq_rotate_quantize_structured_mxint4(_ptr(X), _ptr(R_B), _ptr(R_intra), M, d, _ptr(out_bytes),
                                                        _ptr(out_scales), _stream(stream)),
           "torq_rotate_quantize_structured_mxint4")
    return out_bytes, out_scales


def torq_mxint4_gemm(A8, As, W8, Ws, out_dtype=torch.bfloat16, Y=None, stream=None):
    """A8 [M,K], W8 [N,K] operand bytes; As, Ws tiled E8M0 scale bytes -> Y [M,N]."""
    M, K = A8.shape
    N = W8.shape[0]
    for t, n in ((A8, "A8"), (As, "As"), (W8, "W8"), (Ws, "Ws")):
        _check(t, torch.uint8, n)
    if Y is None:
        Y = torch.empty((M, N), dtype=out_dtype, device=A8.device)
    _check(Y, Y.dtype, "Y")
    dt = TORQ_F32 if Y.dtype == torch.float32 else TORQ_BF16
    _raise(lib().torq_mxint4_gemm(_ptr(A8), _ptr(As), _ptr(W8), _ptr(Ws), M, N, K, _ptr(Y), dt, _stream(stream)),
           "torq_mxint4_gemm")
    return Y


def torq_rotated_linear_mxint4(X, R_inter, R_intra, W8, Ws, out_dtype=torch.bfloat16, Y=None, workspace=None,
                               dbg_bytes=None, dbg_scales=None, stream=None):
    """Rotate, quantize to MXINT4 and multiply in one call.  Returns Y [M,N]."""
    M, d = X.shape
    N = W8.shape[0]
    for t, n in ((X, "X"), (R_inter, "R_inter"), (R_intra, "R_intra")):
        _check(t, torch.bfloat16, n)
    for t, n in ((W8, "W8"), (Ws, "Ws"), (dbg_bytes, "dbg_bytes"), (dbg_scales, "dbg_scales")):
        _check(t, torch.uint8, n)
    if Y is None:
        Y = torch.empty((M, N), dtype=out_dtype, device=X.device)
    if workspace is None:
        workspace = torch.empty(torq_mxint4_workspace_bytes(M, d, N), dtype=torch.uint8, device=X.device)
    dt = TORQ_F32 if Y.dtype == torch.float32 else TORQ_BF16
    _raise(lib().torq_rotated_linear_mxint4(_ptr(X), _ptr(R_inter), _ptr(R_intra), _ptr(W8), _ptr(Ws), M, d, N,
                                            _ptr(Y), dt, _ptr(workspace), workspace.numel(), _ptr(dbg_bytes),
                                            _ptr(dbg_scales), _stream(stream)), "torq_rotated_linear_mxint4")
    return Y


def torq_prepare_weights_mxint4(R_inter, R_intra, W, workspace=None, stream=None):
    """Offline weight side in MXINT4: returns (stored form [N,d/2], operand form [N,d], tiled scales)."""
    d, N, workspace = _prep_args(R_inter, R_intra, W, workspace)
    Wn = torch.empty((N, d // 2), dtype=torch.uint8, device=W.device)
    W8 = torch.empty((N, d), dtype=torch.uint8, device=W.device)
    Ws = torch.empty(torq_scales_bytes(N, d), dtype=torch.uint8, device=W.device)
    _raise(lib().torq_prepare_weights_mxint4(_ptr(W), _ptr(R_inter), _ptr(R_intra), d, N, _ptr(Wn), _ptr(W8), _ptr(Ws),
                                             _ptr(workspace), workspace.numel(), _stream(stream)),
           "torq_prepare_weights_mxint4")
    return Wn, W8, Ws


prepare_weights_mxint4 = torq_prepare_weights_mxint4


# ---- calibration of the inter-block rotation (Section 5.1, Algorithm 1; offline) -----------------------
def torq_block_covariance(X, out=None, stream=None):
    """X [T,d] bf16 -> Sigma [d/32,d/32] float64: covariance across blocks, pooled over tokens and positions."""
    _check(X, torch.bfloat16, "X")
    T, d = X.shape
    if out is None:
        out = torch.empty((d // 32, d // 32), dtype=torch.float64, device=X.device)
    _check(out, torch.float64, "out")
    _raise(lib().torq_block_covariance(_ptr(X), T, d, _ptr(out), _stream(stream)), "torq_block_covariance")
    return out


def torq_givens_equalize(Sigma, eps: float, stream=None):
    """Algorithm 1 on Sigma [B,B] float64 (overwritten with Q Sigma Q^T).
    Returns (Q float64 [B,B], Q bf16 [B,B], number of rotations as a device int32 tensor)."""
    _check(Sigma, torch.float64, "Sigma")
    B = Sigma.shape[0]
    Q = torch.empty((B, B), dtype=torch.float64, device=Sigma.device)
    Qb = torch.empty((B, B), dtype=torch.bfloat16, device=Sigma.device)
    n = torch.zeros(4, dtype=torch.int32, device=Sigma.device)
    _raise(lib().torq_givens_equalize(_ptr(Sigma), B, float(eps), _ptr(Q), _ptr(Qb), _ptr(n), _stream(stream)),
           "torq_givens_equalize")
    return Q, Qb, n[:1]


def torq_rotate_quantize_structured_nvfp4(X, R_B, R_intra, tensor_scale: float, out_codes=None, out_scales=None,
                                          stream=None):
    """The structured rotation (R_B [d/32,d/32], shared R_intra [32,32] or None) followed by the NVFP4 quantizer."""
    M, d = X.shape
    for t, n in ((X, "X"), (R_B, "R_B"), (R_intra, "R_intra")):
        _check(t, torch.bfloat16, n)
    if out_codes is None:
        out_codes = torch.empty((M, d // 2), dtype=torch.uint8, device=X.device)
    if out_scales is None:
        out_scales = torch.empty(torq_nvfp4_scales_bytes(M, d), dtype=torch.uint8, device=X.device)
    _raise(lib().torq_rotate_quantize_structured_nvfp4(_ptr(X), _ptr(R_B), _ptr(R_intra), M, d, tensor_scale,
                                                       _ptr(out_codes), _ptr(out_scales), _stream(stream)),
           "torq_rotate_quantize_structured_nvfp4")
    return out_codes, out_scales
