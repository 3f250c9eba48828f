"""The multi-GPU form of the path on CPU: two gloo ranks split a batch by rows, each runs the
whole layer on its rows with replicated rotations and weights, and nothing is exchanged but the
timings.  The oracle stands in for the per-rank computation (no GPU here); what is under test is
the host logic: the partition, that row shards reproduce the unsharded result exactly (the
property that makes the path collective-free), and the max-over-ranks reduction."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle as O
from paper_2605_19561_b200 import inputs as I
from paper_2605_19561_b200.sharding import max_over_ranks, row_range


def test_row_range_is_a_balanced_partition():
    for M in (0, 1, 2, 7, 64, 2048, 16385):
        for world in (1, 2, 3, 8):
            spans = [row_range(M, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == M
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        row_range(4, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = I.CONFIGS["tiny"]
        xb = I.activations(cfg, M=67)                       # odd row count: shards of 34 and 33
        rb, rib, _, _ = I.rotations(cfg)
        w_codes, w_sb = O.prepare_weights(rb, rib, I.weights(cfg))
        lo, hi = row_range(xb.shape[0], rank, world)
        out, codes, sb = O.rotated_linear(xb[lo:hi], rb, rib, w_codes, w_sb)
        np.savez(os.path.join(out_dir, f"shard{rank}.npz"), lo=lo, hi=hi, out=out, codes=codes, sb=sb)
        # timings: every rank reports its own, all must see the maximum
        mine = [1.0 + rank, 10.0 - rank]
        got = max_over_ranks(mine)
        assert got == [float(world), 10.0], got
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_rows_without_any_exchange(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg, M=67)
    rb, rib, _, _ = I.rotations(cfg)
    w_codes, w_sb = O.prepare_weights(rb, rib, I.weights(cfg))
    out, codes, sb = O.rotated_linear(xb, rb, rib, w_codes, w_sb)
    shards = [np.load(os.path.join(tmp_path, f"shard{r}.npz")) for r in range(world)]
    assert [int(s["lo"]) for s in shards] == [0, 34] and int(shards[-1]["hi"]) == 67
    assert np.array_equal(np.concatenate([s["codes"] for s in shards]), codes)
    assert np.array_equal(np.concatenate([s["sb"] for s in shards]), sb)
    # the fp64 matrix product may block differently for 34 rows than for 67: rounding-level slack
    np.testing.assert_allclose(np.concatenate([s["out"] for s in shards]), out, rtol=1e-12, atol=1e-12)


def test_max_over_ranks_without_a_process_group_is_the_identity():
    assert max_over_ranks([3.0, 1.5]) == [3.0, 1.5]
