"""The N > 1 path on CPU: two gloo ranks run the replica bookkeeping bench.py uses (barrier, max over ranks
of the timed region, whole-job throughput = bytes of all replicas / slowest replica's time)."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2608_00358_b200 import multi
    multi.barrier(dist)
    local_ms = 10.0 if rank == 0 else 25.0            # rank 1 is the slow replica
    gbs, worst = multi.replica_throughput_gbs(local_ms, bytes_per_step=1_000_000_000, steps=5, dist=dist)
    out[rank] = (gbs, worst)
    multi.barrier(dist)
    dist.destroy_process_group()


def test_two_gloo_replicas_report_sum_of_bytes_over_slowest_rank():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert len(out) == 2
    for rank in range(world):
        gbs, worst = out[rank]
        assert worst == 25.0                                          # max over ranks, on every rank
        assert abs(gbs - 2 * 1e9 * 5 / 25e-3 / 1e9) < 1e-9            # 2 replicas x 5 GB / 25 ms = 400 GB/s


def test_single_process_is_its_own_figure():
    from paper_2608_00358_b200 import multi
    gbs, worst = multi.replica_throughput_gbs(2.0, 1 << 30, 3)
    assert worst == 2.0 and abs(gbs - 3 * (1 << 30) / 2e-3 / 1e9) < 1e-9
