"""The N > 1 path on CPU: two gloo ranks shard rows, run the (oracle) layer on their shard, and
the max-over-ranks timing / whole-job throughput reduction works.  Sharded results equal the
unsharded ones because rows are independent under per-row scales."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle as orc
from paper_2203_15952_b200 import inputs as gen
from paper_2203_15952_b200.shard import aggregate_throughput, row_shard


def test_row_shard_covers_rows_once():
    for M, world in ((12800, 2), (12800, 8), (1000, 3), (65536, 8), (5, 2)):
        spans = [row_shard(M, r, world) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == M
        assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
        tiles = [(b - a + 127) // 128 for a, b in spans]
        assert max(tiles) - min(tiles) <= 1
    assert aggregate_throughput([10.0, 10.0], 2.0) == 10.0


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, M, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = gen.WORKLOADS[2]
    spec = gen.workload_layers(w)[0]
    wq, sw = orc.quantize(gen.layer_weight(w, 0, 0, spec), 4, orc.AXIS_ROW)       # replicated weights
    a, b = row_shard(M, rank, world)
    x = gen.workload_input(w, row_subset=range(a, b))
    y = orc.linear_fwd(x, wq, sw, act=orc.ACT_SWISH)
    np.save(os.path.join(out_dir, "y%d.npy" % rank), y)
    t = torch.tensor([0.5 + rank], dtype=torch.float64)                           # pretend step times
    dist.barrier()
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        np.save(os.path.join(out_dir, "tmax.npy"), t.numpy())
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_rows_without_a_collective(tmp_path):
    M, world = 300, 2
    mp.spawn(_worker, args=(world, _free_port(), M, str(tmp_path)), nprocs=world, join=True)
    w = gen.WORKLOADS[2]
    spec = gen.workload_layers(w)[0]
    wq, sw = orc.quantize(gen.layer_weight(w, 0, 0, spec), 4, orc.AXIS_ROW)
    y_full = orc.linear_fwd(gen.workload_input(w, row_subset=range(M)), wq, sw, act=orc.ACT_SWISH)
    y_sharded = np.concatenate([np.load(tmp_path / ("y%d.npy" % r)) for r in range(world)])
    assert np.array_equal(y_full.view(np.uint32), y_sharded.view(np.uint32))
    assert float(np.load(tmp_path / "tmax.npy")[0]) == 1.5
