"""The N>1 path is 'replicas only': ranks own disjoint tensors and only meet for a barrier and a
max-reduction of the time.  Exercised here with two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2501_02379_b200 import replicas, synth


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close(); return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ids = replicas.tensor_ids_for_rank(rank, world, 2)
    wl = synth.WORKLOADS["tiny4"]
    # each rank draws its own tensors; different ids give different data
    norms = [float(abs(synth.GradientSource(wl, i).gradient(0)).sum()) for i in ids]
    my_time = 1.0 + rank           # rank 1 is the slow one
    dist.barrier()
    tmax = replicas.max_over_ranks(my_time, dist)
    gathered = [None] * world
    dist.all_gather_object(gathered, (ids, norms))
    if rank == 0:
        out.put((tmax, gathered, replicas.aggregate_throughput(10.0, world, tmax)))
    dist.destroy_process_group()


def test_two_ranks_disjoint_tensors_and_max_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    tmax, gathered, thr = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert tmax == 2.0
    assert gathered[0][0] == [0, 1] and gathered[1][0] == [2, 3]
    all_norms = gathered[0][1] + gathered[1][1]
    assert len(set(all_norms)) == 4
    assert thr == 10.0 * 2 / 2.0


def test_single_process_identity():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.tensor_ids_for_rank(0, 1, 4) == [0, 1, 2, 3]
