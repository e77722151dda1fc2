"""The benchmark's multi-process bookkeeping on CPU: the layer does not shard (replicas only),
so the job's step time is the max over ranks and its work the sum.  Run as two gloo ranks."""
import os
import socket
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench

    bench.barrier(world)
    ms, units = bench.reduce_max_and_sum(1.0 + rank, 768.0, world)   # rank 1 is the slow replica
    out[rank] = (ms, units)
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_world_size_2():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1] == (2.0, 1536.0)


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.reduce_max_and_sum(3.5, 64.0, 1) == (3.5, 64.0)


def test_reference_arm_exits_quietly_on_other_ranks(capsys):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2308_14352_b200 import inputs

    class A:
        steps, warmup, gpus = 1, 0, 2

    bench.run_reference(A, inputs.WORKLOADS["switch_base_decode"], 64, 12, rank=1, world=2)
    assert capsys.readouterr().out == ""
