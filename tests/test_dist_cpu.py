"""The N > 1 path on CPU: two gloo ranks shard the rows, each computes its share with no exchange of
data, and the shares concatenate to the single-rank result bit for bit; the timing reduction takes
the slowest rank."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import workloads as wl
from paper_2609_39056_b200.dist_util import max_over_ranks, shard_rows, whole_job_value


def test_shard_rows_partitions_and_keeps_streams():
    off, st = wl.segments([(192, 0), (16, 1), (48, 2)])
    for world in (1, 2, 3, 5, 8):
        covered = []
        for rank in range(world):
            lo, hi, o, s = shard_rows(256, off, st, rank, world)
            assert o[0] == 0 and o[-1] == hi - lo and np.all(np.diff(o) > 0)
            row_stream_full = np.repeat(st, np.diff(off))[lo:hi]
            assert np.array_equal(np.repeat(s, np.diff(o)), row_stream_full)
            covered.extend(range(lo, hi))
        assert covered == list(range(256))
    lo, hi, o, s = shard_rows(3, [0, 3], [2], 3, 4)          # more ranks than rows: empty shard
    assert lo == hi and list(o) == [0, 0]


def _worker(rank, world, port, result_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    inp = wl.tiny(seed=31, M=50, K=256, N=64, T=2)
    pw = oracle.pack_int4(inp.W, inp.d, 64)
    lo, hi, o, s = shard_rows(inp.M, inp.seg_offsets, inp.seg_stream, rank, world)
    out = oracle.rudder_linear(inp.X_bf16[lo:hi], pw, inp.gamma, None, 1, 0, o, s, "w4a8", inp.bias)
    np.save(os.path.join(result_dir, f"y{rank}.npy"), out["y"])
    slowest = max_over_ranks(10.0 + rank)                     # rank 1 is "slower"
    np.save(os.path.join(result_dir, f"t{rank}.npy"), np.array([slowest]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_compose_without_a_collective(tmp_path):
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    import oracle
    inp = wl.tiny(seed=31, M=50, K=256, N=64, T=2)
    pw = oracle.pack_int4(inp.W, inp.d, 64)
    full = oracle.rudder_linear(inp.X_bf16, pw, inp.gamma, None, 1, 0, inp.seg_offsets, inp.seg_stream, "w4a8", inp.bias)
    got = np.concatenate([np.load(tmp_path / "y0.npy"), np.load(tmp_path / "y1.npy")])
    assert np.array_equal(got, full["y"])
    assert np.load(tmp_path / "t0.npy")[0] == 11.0 and np.load(tmp_path / "t1.npy")[0] == 11.0
    assert whole_job_value(100.0, 2, 11.0) == pytest.approx(200.0 / 0.011)
