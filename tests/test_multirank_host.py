"""The multi-rank part of the benchmark on CPU: two gloo ranks, no exchange on the data path (every rank
runs its own batch), the job time is the maximum over ranks and the job value the sum of the work."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = [10.0 + 5.0 * rank, 3.0 - rank, 7.0]            # rank 1 is slower on the first, faster on the second
    got = bench.reduce_max(ms, world, "cpu")
    # every rank draws its own activations: different seeds per rank, same weights
    from paper_2407_09453_b200 import synth
    layer = synth.Layer("t", 16, 16, 1, 1, 2, 2, 2)
    W0, X0, _ = synth.make_layer_tensors(layer, "bf16", config=2, layer_id=0)
    Wr, Xr, _ = synth.make_layer_tensors(layer, "bf16", config=2, layer_id=rank)
    same_x = bool((X0 == Xr).all())
    out[rank] = (got, bench.job_tflops(1e12, world, got[0]), same_x)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_max_time_and_sum_the_work():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        got, value, same_x = res[rank]
        assert got == [15.0, 3.0, 7.0]
        assert abs(value - 2 * 1e12 / 15e-3 / 1e12) < 1e-9         # two ranks' work over the slower rank's time
    assert res[0][2] is True and res[1][2] is False                  # rank 1 has its own batch


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max([1.5, 2.5], 1, "cpu") == [1.5, 2.5]
    assert bench.job_tflops(2e12, 1, 1000.0) == 2.0
