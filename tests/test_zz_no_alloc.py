"""torq_rotated_linear_static: the layer for callers that are not allowed to allocate.

A custom operator inside someone else's inference engine, a server that gave all of its device
memory to a cache pool at start-up, or a decode loop that cannot tolerate the device-wide
synchronisation of cudaMalloc has no way to provide the scratch buffer torq_rotated_linear asks
for.  The static entry point keeps that scratch in a fixed array inside the library instead, and
every call on a device reuses it.  These tests go through the C ABI and check that

  * its result equals torq_rotated_linear's (caller-provided workspace) on the same inputs bit for
    bit: the two run the same kernels on the same data, so a single stale byte read from the
    shared array would show,
  * this holds on two calls in a row with different inputs and shapes, i.e. whatever the first
    call left in the shared array does not leak into the second,
  * the calls allocate nothing: free device memory is the same before and after,
  * each regime of the rotation is reached: split along the contraction (few tokens), CTA pairs
    (many tokens), and the single-pass kernel when the array has no room left for partial sums,
  * a problem too large for the array is refused with TORQ_ERR_WORKSPACE and launches nothing.

The file name sorts after every other test file on purpose: a run that stops at the first failure
has then already exercised everything else.  It needs nothing from the other tests and passes in a
fresh process as well.
"""
import numpy as np
import pytest
import torch

from paper_2605_19561_b200 import inputs as I
from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu

TORQ_ERR_WORKSPACE = 7


def _layer(M, d, N, seed):
    """Seeded operands on the device.  The weight codes are random bytes: this test compares two
    entry points with each other, so the weights need not come from a real W."""
    g = np.random.default_rng(seed)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    X = I.bf16_bits_to_tensor(I.to_bf16_bits(g.standard_t(3.0, size=(M, d))), "cuda")
    if d <= 1024:
        R = I.bf16_bits_to_tensor(I.to_bf16_bits(I.orthogonal(d, g)), "cuda")
    else:                                         # any matrix of the right scale serves a comparison of two entry points
        R = (torch.randn((d, d), device="cuda", generator=torch.Generator("cuda").manual_seed(seed)) / d ** 0.5
             ).to(torch.bfloat16)
    Ri = I.bf16_bits_to_tensor(I.to_bf16_bits(I.orthogonal(32, g, batch=d // 32)), "cuda")
    Wq = dev(g.integers(0, 256, size=(N, d // 2), dtype=np.uint8))
    Ws = torq.torq_swizzle_scales(dev(g.integers(118, 126, size=(N, d // 32), dtype=np.uint8)), d)
    return X, R, Ri, Wq, Ws


def _rel(a, b):
    a, b = a.double(), b.double()
    return float((a - b).norm() / b.norm())


def test_static_entry_point_matches_the_workspace_one_on_two_calls_in_a_row():
    # second shape is smaller than the first, so stale bytes of call one surround call two's data
    cases = [(300, 512, 392, torch.float32, 11), (77, 256, 136, torch.bfloat16, 12)]
    prepared = [(_layer(M, d, N, seed), torch.empty((M, N), dtype=dt, device="cuda")) for M, d, N, dt, seed in cases]
    expected = [torq.torq_rotated_linear(*ops, out_dtype=Y.dtype) for ops, Y in prepared]
    torq.torq_rotated_linear_static(*prepared[0][0], Y=prepared[0][1])      # first call on the device: set-up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    before = torq.torq_launch_count()
    for ops, Y in prepared:                       # back to back, same stream, no sync in between
        Y.zero_()
        torq.torq_rotated_linear_static(*ops, Y=Y)
    torch.cuda.synchronize()
    assert torq.torq_launch_count() - before >= 2 * len(cases)     # rotation + GEMM kernels per call
    assert torq.torq_last_device_error() == 0
    for (ops, Y), ref in zip(prepared, expected):
        assert torch.isfinite(Y.float()).all()
        assert torch.equal(Y, ref)
    # and once more in the opposite order: call one's shape after call two's
    for ops, Y in reversed(prepared):
        Y.zero_()
        torq.torq_rotated_linear_static(*ops, Y=Y)
    torch.cuda.synchronize()
    for (ops, Y), ref in zip(prepared, expected):
        assert torch.equal(Y, ref)
    assert torch.cuda.mem_get_info()[0] == free_before             # nothing was allocated, nothing freed


def test_static_entry_point_in_every_regime_of_the_rotation():
    """Many tokens (CTA pairs, single pass: exactly two launches), several waves of tiles whose quantized
    activations nearly fill the array, and a 128-token problem whose partial sums do not fit behind the
    quantized activations in the array, which must fall back to the single pass."""
    # (M, d, N, dtype, seed, exact, launches)
    cases = [(2048, 4096, 512, torch.bfloat16, 21, True, 2),
             (4096, 5120, 5120, torch.bfloat16, 22, True, 2),
             (128, 16384, 256, torch.float32, 23, None, 2)]
    for M, d, N, dt, seed, exact, launches in cases:
        ops = _layer(M, d, N, seed)
        Y = torch.zeros((M, N), dtype=dt, device="cuda")
        if exact is None:
            # the workspace entry point splits this rotation (other summation order): compare with the
            # single-pass kernels instead, which is what the static entry point must have run
            codes, scales = torq.torq_rotate_quantize(*ops[:3])
            ref = torq.torq_mxfp4_gemm(codes, scales, ops[3], ops[4], out_dtype=dt)
            exact = True
        else:
            ref = torq.torq_rotated_linear(*ops, out_dtype=dt)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        before = torq.torq_launch_count()
        torq.torq_rotated_linear_static(*ops, Y=Y)
        torch.cuda.synchronize()
        assert torq.torq_launch_count() - before == launches, (M, d, N)
        assert torq.torq_last_device_error() == 0
        assert torch.cuda.mem_get_info()[0] == free_before
        if exact:
            assert torch.equal(Y, ref), (M, d, N)
        else:
            assert _rel(Y, ref) <= 1e-3, (M, d, N)
        del ops, Y, ref
        torch.cuda.empty_cache()


def test_static_entry_point_refuses_what_does_not_fit():
    M, d, N = 4096, 14336, 8
    assert torq.torq_workspace_bytes(M, d, N) > torq.TORQ_STATIC_WORKSPACE_BYTES
    X = torch.zeros((M, d), dtype=torch.bfloat16, device="cuda")
    Wq = torch.zeros((N, d // 2), dtype=torch.uint8, device="cuda")
    Ws = torch.zeros(torq.torq_scales_bytes(N, d), dtype=torch.uint8, device="cuda")
    Y = torch.full((M, N), 7.0, dtype=torch.float32, device="cuda")
    before = torq.torq_launch_count()
    with pytest.raises(torq.TorqError) as e:
        torq.torq_rotated_linear_static(X, None, None, Wq, Ws, Y=Y)
    assert e.value.code == TORQ_ERR_WORKSPACE
    assert torq.torq_launch_count() == before
    torch.cuda.synchronize()
    assert bool((Y == 7.0).all())
    # the largest LLaMA3-8B shape of the workloads still fits
    assert torq.torq_workspace_bytes(2048, 14336, 4096) <= torq.TORQ_STATIC_WORKSPACE_BYTES
