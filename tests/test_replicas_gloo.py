"""world_size-2 check (gloo, CPU) of the multi-GPU plumbing: disjoint clients per rank, max-over-ranks timing."""
import os
import socket

import torch
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
    from paper_2402_03770_b200 import replica as R
    from paper_2402_03770_b200 import workloads as W
    clients = R.replica_clients(rank, 3)
    w = W.WORKLOADS["small_cnn"]
    x0 = W.client_update(w, clients[0], d=1000)
    my_ms = 5.0 + 2.0 * rank
    slowest = R.max_over_ranks(my_ms, torch.device("cpu"))
    dist.barrier()
    out[rank] = (clients, float(x0[:8].sum()), slowest, R.job_throughput(100, world, slowest))
    dist.destroy_process_group()


def test_two_replicas_have_disjoint_clients_and_agree_on_the_slowest_time():
    world = 2
    port = _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        a, b = out[0], out[1]
    assert a[0] == [0, 1, 2] and b[0] == [3, 4, 5]
    assert a[1] != b[1]                      # different seeds, different data
    assert a[2] == b[2] == 7.0               # max over ranks
    assert a[3] == b[3] == 100 * 2 / 7.0e-3
