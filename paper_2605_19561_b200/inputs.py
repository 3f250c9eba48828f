"""Seeded synthetic inputs for the rotated-MXFP4 linear layer.

This module only *draws* data: activations, orthogonal matrices, weights, and their
bfloat16 bit patterns.  It contains none of the method's arithmetic (no rotation is
applied, nothing is quantized here) so that both the CUDA path and the CPU checker
can be fed from it without sharing any code that is under test.

The activations stand in for LLaMA3 / Qwen3 layer inputs: heavy-tailed (Student-t
with 3 degrees of freedom, or Laplace for the post-SwiGLU shape) with a handful of
channels scaled up to imitate outlier features.  Rotations are the Q factor of a
seeded Gaussian matrix with the sign convention diag(R_qr) > 0.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

BASE_SEED = 260519561
K_BLOCK = 32


@dataclass(frozen=True)
class LayerConfig:
    name: str
    cfg_id: int
    M: int
    d: int
    N: int
    dist: str            # "student_t3" | "laplace"
    n_outliers: int
    outlier_gain: float
    out_dtype: str       # "f32" | "bf16"


CONFIGS = {
    "tiny": LayerConfig("tiny", 1, 64, 256, 256, "student_t3", 4, 50.0, "f32"),
    "llama3_8b_qkv": LayerConfig("llama3_8b_qkv", 2, 2048, 4096, 6144, "student_t3", 4, 100.0, "bf16"),
    "llama3_8b_down": LayerConfig("llama3_8b_down", 3, 2048, 14336, 4096, "laplace", 8, 200.0, "bf16"),
    "qwen3_32b_gateup": LayerConfig("qwen3_32b_gateup", 4, 8192, 5120, 51200, "student_t3", 5, 100.0, "bf16"),
    "qwen3_32b_sweep": LayerConfig("qwen3_32b_sweep", 5, 1024, 5120, 5120, "student_t3", 0, 1.0, "bf16"),
}
SWEEP_M = (1, 4, 16, 64, 256, 1024, 4096, 16384)


def _rng(cfg_id: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(BASE_SEED + 100 * cfg_id + stream))


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float array -> bfloat16 bit patterns (uint16), round to nearest even."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_bits_to_tensor(bits: np.ndarray, device="cpu") -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.to(device)


def activations(cfg: LayerConfig, M: int | None = None, d: int | None = None) -> np.ndarray:
    """X [M,d] as bfloat16 bit patterns."""
    M = cfg.M if M is None else M
    d = cfg.d if d is None else d
    g = _rng(cfg.cfg_id, 0)
    if cfg.dist == "student_t3":
        x = g.standard_t(3.0, size=(M, d))
    elif cfg.dist == "laplace":
        x = g.laplace(0.0, 1.0, size=(M, d))
    else:
        raise ValueError(cfg.dist)
    if cfg.n_outliers:
        ch = _rng(cfg.cfg_id, 4).choice(d, size=min(cfg.n_outliers, d), replace=False)
        x[:, ch] *= cfg.outlier_gain
    return to_bf16_bits(x)


def orthogonal(n: int, g: np.random.Generator, batch: int | None = None, device: str = "cpu") -> np.ndarray:
    """Q factor (float64) of a seeded Gaussian matrix, columns sign-fixed so that the
    R factor has a positive diagonal.  With `batch`, a stack of independent matrices.
    `device` only chooses where LAPACK-style QR runs (large n is slow on few cores)."""
    shape = (n, n) if batch is None else (batch, n, n)
    a = g.standard_normal(size=shape)
    if device != "cpu":
        q, r = torch.linalg.qr(torch.from_numpy(a).to(device))
        q = q * torch.sign(torch.diagonal(r, dim1=-2, dim2=-1)).unsqueeze(-2)
        return q.cpu().numpy()
    q, r = np.linalg.qr(a)
    sgn = np.sign(np.diagonal(r, axis1=-2, axis2=-1))
    return q * sgn[..., None, :]


def rotations(cfg: LayerConfig, d: int | None = None, device: str = "cpu"):
    """(R_inter [d,d], R_intra [d/32,32,32]) as bfloat16 bit patterns, plus the float64
    matrices they were rounded from (for orthogonality checks)."""
    d = cfg.d if d is None else d
    r_inter = orthogonal(d, _rng(cfg.cfg_id, 1), device=device)
    r_intra = orthogonal(K_BLOCK, _rng(cfg.cfg_id, 2), batch=d // K_BLOCK)
    return to_bf16_bits(r_inter), to_bf16_bits(r_intra), r_inter, r_intra


def intra_rotations16(cfg: LayerConfig, d: int | None = None) -> np.ndarray:
    """R_intra [d/16,16,16] as bfloat16 bit patterns: the intra-block rotations of a format whose
    quantization block has 16 elements (stream 5 of the configuration)."""
    d = cfg.d if d is None else d
    return to_bf16_bits(orthogonal(16, _rng(cfg.cfg_id, 5), batch=d // 16))


def weights(cfg: LayerConfig, d: int | None = None, N: int | None = None) -> np.ndarray:
    """W [d,N] ~ N(0, 0.02^2), float32 (the un-rotated weight of out = x W)."""
    d = cfg.d if d is None else d
    N = cfg.N if N is None else N
    return (_rng(cfg.cfg_id, 3).standard_normal(size=(d, N)) * 0.02).astype(np.float32)


def random_codes(rows: int, k: int, seed: int):
    """Uniformly random packed e2m1 codes [rows,k/2] and scale bytes [rows,k/32] in a
    narrow range around 2^0 (for GEMM-only tests and benchmarks)."""
    g = np.random.Generator(np.random.PCG64(BASE_SEED + 7919 * seed))
    packed = g.integers(0, 256, size=(rows, k // 2), dtype=np.uint8)
    sb = g.integers(120, 131, size=(rows, k // K_BLOCK), dtype=np.uint8)
    return packed, sb
