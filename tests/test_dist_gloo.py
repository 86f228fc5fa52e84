"""World-size-2 checks of the data-parallel path (batch-sharded replicas, one all-reduce of the core gradients).

CPU (gloo): every rank differentiates its own batch shard with the fp64 oracle, the flat gradients are summed
with the library's all-reduce helper, and the sum is compared with the oracle's gradient of the CONCATENATED
batch (the bags of both shards in one call), which is what data parallelism has to reproduce.

GPU (marked gpu; two processes share the one GPU, gloo carries the CUDA tensors): each rank runs the CUDA forward
and backward on its shard, all-reduces its flat gradient buffer, applies tt_emb_sgd_step; both ranks must end with
the cores the oracle gets from one SGD step on the concatenated batch.  No kernel of one rank waits for the other:
the exchange is a host-side collective between the backward and the update."""
import os
import socket

import numpy as np
import pytest
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


def _shard(rank):
    from paper_2609_03459_b200 import dist as ttd
    # same tables and cores on every rank, own batch shard
    return workloads.make(5, tiny=True, batch_seed=None if rank == 0 else ttd.rank_seed(workloads.BASE_SEED, rank))


def _concatenated(shards):
    """One workload holding the bags of all shards: per table the bags of shard 0, then those of shard 1, ..."""
    first = shards[0]
    T, Bs = first.T, [s.B for s in shards]
    idx_parts, lens = [], []
    for t in range(T):
        for s in shards:
            i, o = s.table_slice(t)
            idx_parts.append(i)
            lens.append(o[1:] - o[:-1])
    offsets = np.concatenate([[0], np.cumsum(np.concatenate(lens))]).astype(np.int64)
    grad = np.concatenate([s.grad_out for s in shards], axis=0)
    return workloads.Workload(name="concat", tables=first.tables, B=sum(Bs), indices=np.concatenate(idx_parts).astype(np.int64),
                              offsets=offsets, cores=first.cores, grad_out=grad, lr=first.lr)


def _flat(grads):
    return np.concatenate([g.reshape(-1) for tg in grads for g in tg])


def _worker(rank, world, port, q):
    import torch.distributed as dist
    from paper_2609_03459_b200 import dist as ttd
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = _shard(rank)
        grads = oracle.backward_workload(mine)
        flat = torch.from_numpy(_flat(grads))
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
    assert np.abs(locals_[0] - locals_[1]).max() > 0                       # the shards really differ
    # the gradient of the whole batch, computed by the oracle in one call over the bags of both shards
    whole = _concatenated([_shard(r) for r in range(world)])
    assert whole.B == 2 * _shard(0).B and whole.L == res[0][5] + res[1][5]
    want = _flat(oracle.backward_workload(whole))
    np.testing.assert_allclose(reduced[0], want, rtol=1e-11, atol=1e-13 * np.abs(want).max())
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


def _gpu_worker(rank, world, port, q):
    import torch.distributed as dist
    from paper_2609_03459_b200 import binding
    from paper_2609_03459_b200 import dist as ttd
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = _shard(rank)
        emb = binding.from_workload(mine, enable_backward=True)
        out = emb.forward(torch.from_numpy(mine.indices).cuda(), torch.from_numpy(mine.offsets).cuda(), mine.B)
        emb.backward(torch.from_numpy(mine.grad_out).cuda())
        torch.cuda.synchronize()
        ttd.allreduce_core_grads(emb.flat_grads)      # the one exchange of the path
        emb.sgd_step(mine.lr)
        torch.cuda.synchronize()
        q.put((rank, out.cpu().numpy(), emb.get_grads(), emb.get_cores(), emb.status()))
    finally:
        dist.destroy_process_group()


@pytest.mark.gpu
def test_two_ranks_on_the_gpu_reproduce_the_whole_batch_training_step():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import __graft_entry__ as entry
    entry.build()
    world = 2
    port = _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_gpu_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted([q.get(timeout=600) for _ in range(world)], key=lambda x: x[0])
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    shards = [_shard(r) for r in range(world)]
    whole = _concatenated(shards)
    ref_g = oracle.backward_workload(whole)
    for rank, out, grads, cores, status in res:
        assert status == 0
        ref_out = oracle.forward_workload(shards[rank])
        assert np.abs(out - ref_out).max() <= 1e-5 * np.abs(ref_out).max()
        for t in range(whole.T):
            want = oracle.sgd(whole.cores[t], ref_g[t], whole.lr)
            for k in range(len(want)):
                scale = max(np.abs(ref_g[t][k]).max(), 1e-300)
                assert np.abs(grads[t][k] - ref_g[t][k]).max() <= 1e-5 * scale, ("grad", rank, t, k)
                assert np.abs(cores[t][k] - want[k]).max() <= 1e-5 * np.abs(want[k]).max(), ("core", rank, t, k)
