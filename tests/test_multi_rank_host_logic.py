"""Host-side logic of the multi-GPU benchmark path on CPU: two gloo ranks shard the batch (no exchange step on
the data path) and reduce their timings with MAX."""
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
    r0, r1 = bench.shard_rows(world, rank, batch_per_gpu=3, seq=197)
    spans = [None] * world
    dist.all_gather_object(spans, (r0, r1))
    slowest = bench.max_over_ranks([10.0 + rank, 5.0 - rank], torch.device("cpu"), world)
    if rank == 0:
        out.put((spans, slowest))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_the_batch_and_take_the_slowest_timing():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    spans, slowest = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert spans == [(0, 3 * 197), (3 * 197, 6 * 197)]          # disjoint, contiguous, whole batch items
    assert slowest == [11.0, 5.0]


def test_bench_starts_its_own_ranks_when_not_launched_as_ranks():
    """`bench.py --gpus N` without a launcher's environment hands over to N ranks on this node (one per GPU,
    rendezvous on 127.0.0.1); the command line it builds is checked here, nothing is started."""
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.spawn_command(4, ["--gpus", "4", "--steps", "20"], 29555)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert cmd[cmd.index("--nproc-per-node") + 1] == "4"
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29555"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "20"] and cmd[-5].endswith("bench.py")
