"""Run-to-run determinism of the whole layer: every reduction in the path (tensor-core accumulation inside
a tile, the K splits of the few-token kernels added in cluster-rank order, the split-K partials added in split
order) has a fixed order, so repeated calls on the same inputs must return the same bits -- codes, scales and
outputs -- whatever else the GPU is doing.  One shape per dispatch regime."""
import pytest
import torch

from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,d,N", [(1, 5120, 5120), (64, 1536, 640), (128, 2560, 1024), (200, 1280, 512),
                                   (384, 1024, 256), (1024, 5120, 1024), (3840, 1280, 1280), (2048, 4096, 6144)])
def test_repeated_calls_return_the_same_bits(M, d, N):
    g = torch.Generator(device="cuda").manual_seed(1000 * M + d)
    X = (torch.randn(M, d, device="cuda", generator=g) * 2).bfloat16()
    R = (torch.randn(d, d, device="cuda", generator=g) / d ** 0.5).bfloat16()
    Ri = (torch.randn(d // 32, 32, 32, device="cuda", generator=g) / 32 ** 0.5).bfloat16()
    Wq = torch.randint(0, 256, (N, d // 2), dtype=torch.uint8, device="cuda", generator=g)
    Ws = torch.randint(120, 132, (torq.torq_scales_bytes(N, d),), dtype=torch.uint8, device="cuda", generator=g)
    first = None
    for it in range(12):
        dbg_c = torch.empty((M, d // 2), dtype=torch.uint8, device="cuda")
        dbg_s = torch.empty(torq.torq_scales_bytes(M, d), dtype=torch.uint8, device="cuda")
        y = torq.torq_rotated_linear(X, R, Ri, Wq, Ws, out_dtype=torch.bfloat16, dbg_codes=dbg_c, dbg_scales=dbg_s)
        torch.cuda.synchronize()
        if first is None:
            first = (y.clone(), dbg_c.clone(), dbg_s.clone())
            assert bool(torch.isfinite(y.float()).all())
        else:
            assert torch.equal(y, first[0]) and torch.equal(dbg_c, first[1]) and torch.equal(dbg_s, first[2]), it
    assert torq.torq_last_device_error() == 0
