"""World-size-2 check (gloo, CPU) of the data-parallel plumbing: every rank differentiates its own batch
shard, the core gradients are summed with one all-reduce, and the sum equals the gradient of the whole
batch.  The per-rank gradients come from the fp64 oracle here (no GPU in this test); on GPUs the same
helpers are fed by the CUDA backward."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

import oracle
import workloads


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    import torch.distributed as dist
    from paper_2609_03459_b200 import dist as ttd
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # same tables and cores on every rank, own batch shard
        mine = workloads.make(5, tiny=True, batch_seed=None if rank == 0 else ttd.rank_seed(workloads.BASE_SEED, rank))
        grads = oracle.backward_workload(mine)
        flat = torch.from_numpy(np.concatenate([g.reshape(-1) for tg in grads for g in tg]))
        local = flat.clone()
        ttd.allreduce_core_grads(flat)
        t_max = ttd.max_over_ranks(10.0 + rank)
        n_sum = ttd.sum_over_ranks(mine.L)
        q.put((rank, local.numpy(), flat.numpy(), t_max, n_sum, mine.L))
    finally:
        dist.destroy_process_group()


def test_two_rank_gradient_allreduce_equals_whole_batch_gradient():
    world = 2
    port = _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted([q.get(timeout=180) for _ in range(world)], key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    locals_, reduced = [r[1] for r in res], [r[2] for r in res]
    np.testing.assert_array_equal(reduced[0], reduced[1])                  # every rank ends with the same sum
    np.testing.assert_allclose(reduced[0], locals_[0] + locals_[1], rtol=1e-12, atol=1e-14)
    assert np.abs(locals_[0] - locals_[1]).max() > 0                       # the shards really differ
    assert res[0][3] == res[1][3] == 11.0                                  # max over ranks of the step time
    assert res[0][4] == res[0][5] + res[1][5]                              # lookups of all ranks


def test_rank_seed_keeps_rank0_on_the_single_gpu_stream():
    from paper_2609_03459_b200 import dist as ttd
    assert ttd.rank_seed(123, 0) == 123
    assert len({ttd.rank_seed(123, r) for r in range(8)}) == 8
    assert ttd.world() == 1
    assert ttd.max_over_ranks(3.5) == 3.5 and ttd.sum_over_ranks(2) == 2.0
    x = torch.ones(4)
    assert ttd.allreduce_core_grads(x) is x
