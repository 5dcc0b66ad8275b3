"""The replica logic of the multi-GPU benchmark path on two CPU processes (gloo)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2402_17227_b200 import dist_util


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = dist_util.rank_batches(rank, 8)
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    slowest = dist_util.max_over_ranks(10.0 + 5.0 * rank)
    dist.barrier()
    if rank == 0:
        flat = [b for g in gathered for b in g]
        out.put((len(flat) == len(set(flat)) == 8 * world, slowest))
    dist.destroy_process_group()


def test_two_replicas_disjoint_batches_and_max_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    disjoint, slowest = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert disjoint and slowest == 15.0


def test_metric_is_whole_job():
    # two replicas finishing 100 calls each in 5 ms: 0.025 ms per layer backward over the job
    assert dist_util.ms_per_layer(5.0, 100, 2) == 0.025
    assert dist_util.max_over_ranks(3.0) == 3.0          # no process group: identity


def _reduce_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    red = dist_util.GradReducer()
    # three "layers": the gradient of layer l on replica r is (r + 1) * (l + 1); reductions are issued layer by
    # layer while the "backward" goes on, and waited for once at the end of the pass
    grads = [torch.full((4, 3), float((rank + 1) * (l + 1))) for l in range(3)]
    for g in grads:
        red.reduce_async(g)
    assert red.active and len(red.works) == 3
    red.wait()
    ok = all(torch.all(g == float(sum(r + 1 for r in range(world)) * (l + 1))) for l, g in enumerate(grads))
    ok = ok and len(red.works) == 0
    dist.barrier()
    if rank == 0:
        out.put(bool(ok))
    dist.destroy_process_group()


def test_two_replicas_sum_their_weight_gradients():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_reduce_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ok = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ok
    red = dist_util.GradReducer()                         # no process group: nothing to do
    red.reduce_async(torch.ones(2)); red.wait()
    assert not red.active
