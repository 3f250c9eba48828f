"""Shared test helpers: moving arrays to the device and the mismatch accounting used when the
CUDA path and the oracle may legitimately differ by accumulation order."""
import numpy as np
import torch

import oracle as O
from paper_2605_19561_b200 import inputs as I


def dev_bf16(bits):
    return I.bf16_bits_to_tensor(bits, "cuda").contiguous()


def dev_u8(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint8)).cuda()


def gpu_quantized_to_numpy(codes_t, scales_t, M, d):
    """(packed codes tensor, tiled scales tensor) -> (codes [M,d] 0..15, scale bytes [M,d/32])."""
    codes = O.unpack_codes(codes_t.cpu().numpy())
    sb = O.unswizzle_scales(scales_t.cpu().numpy(), M, d)
    return codes, sb


def lattice(codes):
    """Position on the 15-value signed e2m1 lattice (+0 and -0 coincide)."""
    mag = (codes & 7).astype(np.int64)
    return np.where(codes & 8, -mag, mag)


def mismatch_report(g_codes, g_sb, o_codes, o_sb):
    """Fractions of differing elements / blocks and whether every difference is benign:
    same scale -> codes at most one lattice step apart; scale differing by one step -> values
    at most one step of the coarser grid apart.  `elem_mismatch_frac` counts every element whose
    decoded value differs, inside blocks whose scale byte differs as well, so the acceptance
    bound on it covers all elements."""
    M, d = o_codes.shape
    same_scale = g_sb == o_sb
    same_scale_e = np.repeat(same_scale, 32, axis=1)
    lg, lo = lattice(g_codes), lattice(o_codes)
    diff = (lg != lo) & same_scale_e
    adjacent = np.abs(lg - lo) <= 1
    bad_elems = int((diff & ~adjacent).sum())
    # blocks whose scale differs
    nblk_diff = int((~same_scale).sum())
    scale_step = np.abs(g_sb.astype(np.int64) - o_sb.astype(np.int64))
    bad_blocks = int((scale_step > 1).sum())
    n_diff = int(diff.sum())
    if nblk_diff:
        dg, do = O.dequantize(g_codes, g_sb), O.dequantize(o_codes, o_sb)
        coarse = np.ldexp(1.0, np.maximum(g_sb, o_sb).astype(np.int64) - 127)   # grid step <= 2*2^e; use 2*s
        tol = 2.0 * np.repeat(coarse, 32, axis=1)
        bad_elems += int(((np.abs(dg - do) > tol) & ~same_scale_e).sum())
        n_diff += int(((dg != do) & ~same_scale_e).sum())
    return {
        "elem_mismatch_frac": float(n_diff) / (M * d),
        "block_scale_mismatch_frac": nblk_diff / (M * (d // 32)),
        "non_adjacent": bad_elems,
        "scale_off_by_more_than_one": bad_blocks,
    }
