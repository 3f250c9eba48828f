"""torq_rotated_linear_static: the layer for callers that are not allowed to allocate.

A custom operator inside someone else's inference engine, a server that gave all of its device
memory to a cache pool at start-up, or a decode loop that cannot tolerate the device-wide
synchronisation of cudaMalloc has no way to provide the scratch buffer torq_rotated_linear asks
for.  The static entry point keeps that scratch in a fixed array inside the library instead, and
every call on a device reuses it.  These tests go through the C ABI and check that

  * its result matches torq_rotated_linear (caller-provided workspace) on the same inputs, within
    the bound the other GEMM tests use (relative Frobenius error <= 1e-3; the two run the same
    kernels, so in practice the outputs are identical),
  * this holds on two calls in a row with different inputs and shapes, i.e. whatever the first
    call left in the shared array does not leak into the second,
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
    R = I.bf16_bits_to_tensor(I.to_bf16_bits(I.orthogonal(d, g)), "cuda")
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
    torch.cuda.synchronize()
    before = torq.torq_launch_count()
    for ops, Y in prepared:                       # back to back, same stream, no sync in between
        torq.torq_rotated_linear_static(*ops, Y=Y)
    torch.cuda.synchronize()
    assert torq.torq_launch_count() - before >= 2 * len(cases)     # rotation + GEMM kernels per call
    assert torq.torq_last_device_error() == 0
    for (ops, Y), ref in zip(prepared, expected):
        assert torch.isfinite(Y.float()).all()
        assert _rel(Y, ref) <= 1e-3
    # and once more in the opposite order: call one's shape after call two's
    for ops, Y in reversed(prepared):
        Y.zero_()
        torq.torq_rotated_linear_static(*ops, Y=Y)
    torch.cuda.synchronize()
    for (ops, Y), ref in zip(prepared, expected):
        assert _rel(Y, ref) <= 1e-3


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
