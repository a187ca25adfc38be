"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own layer
(independent problems, no data-path collective); only the timing is reduced (max)."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    sys.path.insert(0, ROOT)
    import bench
    import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, world, rank)
    layer = synth.make_layer("c2", 8, 64, 128, seed=bench.layer_seed(rank))
    ms = bench.max_over_ranks(torch.tensor([10.0 + rank, 3.0 - rank], dtype=torch.float64), world)
    out[rank] = (float(layer.W.float().sum()), ms.tolist())
    dist.destroy_process_group()


def test_two_ranks_get_distinct_layers_and_max_time():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29731, out), nprocs=2, join=True)
    assert out[0][0] != out[1][0]                 # different seeds -> different layers
    assert out[0][1] == out[1][1] == [11.0, 3.0]  # every rank sees the max over ranks
