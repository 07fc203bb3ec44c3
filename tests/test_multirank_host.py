"""Host-side logic of the N > 1 bench path on CPU: two gloo ranks, each with its own batch (replicas, no
data-path collective); the whole-job number is total units over the slowest rank's time."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    import bench
    from paper_1901_06887_b200 import synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    models = synth.make_models(1)
    ids, x = synth.make_requests(1, models, salt=1000 * rank)
    local_ms = 10.0 * (rank + 1)                    # rank 1 is the slow one
    units, ms = bench.aggregate(len(ids) * 5, local_ms, world)
    line = bench.result_line(units, ms, 5)
    ret[rank] = (units, ms, line["value"], int(ids.sum()), int(x.astype(np.int64).sum()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_and_independent_batches():
    world = 2
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
    assert set(ret.keys()) == {0, 1}
    for r in (0, 1):
        units, ms, value, _, _ = ret[r]
        assert units == 2 * 64 * 5 and ms == 20.0
        assert abs(value - 640 / 0.020) < 1e-6
    assert ret[0][3:] != ret[1][3:]                 # ranks draw different batches


def test_single_rank_aggregate_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate(128, 3.5, 1) == (128.0, 3.5)
    line = bench.result_line(128, 4.0, 2)
    assert line["value"] == 32000.0 and line["ms_per_step"] == 2.0 and line["unit"] == "requests/s"
