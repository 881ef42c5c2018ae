"""The multi-GPU mode of the bench is N independent replicas (the layer is not sharded): rank-0's
line must carry all ranks' work over the slowest rank's time.  Checked with 2 gloo ranks on CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 if rank == 0 else 12.5          # rank 1 is the slow replica
    value, ms = bench.replica_throughput(local_ms, 2.0e12, world, device="cpu")
    dist.barrier()
    q.put((rank, value, ms))
    dist.destroy_process_group()


def test_two_replicas_report_whole_job_throughput_over_slowest_rank():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, ms in res:
        assert ms == 12.5
        assert abs(value - 2 * 2.0e12 / 12.5e-3 / 1e12) < 1e-9   # 320 TFLOP/s for the whole job


def test_single_replica_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    value, ms = bench.replica_throughput(4.0, 1.0e12, 1)
    assert ms == 4.0 and abs(value - 250.0) < 1e-9
