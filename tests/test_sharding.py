"""Multi-GPU host logic on CPU: partitions are disjoint, cover everything, and are balanced.
The two-rank test runs real processes over the gloo backend and cross-checks the ranks' shards."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_29010_b200 import inputs, sharding


@pytest.mark.parametrize("total,world,multiple", [(4096, 8, 128), (100352, 8, 128), (1000, 3, 128), (5, 8, 1), (0, 2, 128),
                                                  (129, 2, 128)])
def test_split_range_covers_disjointly(total, world, multiple):
    cuts = [sharding.split_range(total, world, r, multiple) for r in range(world)]
    assert cuts[0][0] == 0 and cuts[-1][1] == total
    for (b0, e0), (b1, e1) in zip(cuts, cuts[1:]):
        assert e0 == b1 and b0 <= e0
    for b, e in cuts[:-1]:
        assert b % multiple == 0 and (e % multiple == 0 or e == total)
    sizes = [-(-(e - b) // multiple) for b, e in cuts]
    assert max(sizes) - min(sizes) <= 1


def test_group_assignment_is_balanced_and_complete():
    Ms = inputs.grouped_sizes(16, 128, 4096)
    for world in (1, 2, 4, 8):
        owned = sharding.assign_groups(Ms, world)
        assert sorted(g for lst in owned for g in lst) == list(range(16))
        loads = [sum(Ms[g] for g in lst) for lst in owned]
        assert max(loads) - min(loads) <= max(Ms)
    assert sharding.assign_groups([], 2) == [[], []]
    with pytest.raises(ValueError):
        sharding.split_range(10, 0, 0)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, M, batch, Ms):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rows = sharding.gemm_rows(M, world, rank)
        bat = sharding.batch_entries(batch, world, rank)
        groups = sharding.assign_groups(Ms, world)[rank]
        # mark what this rank owns; the sum over ranks must be exactly one everywhere
        own_rows = torch.zeros(M, dtype=torch.int64)
        own_rows[rows[0]:rows[1]] = 1
        own_batch = torch.zeros(batch, dtype=torch.int64)
        own_batch[bat[0]:bat[1]] = 1
        own_groups = torch.zeros(len(Ms), dtype=torch.int64)
        own_groups[groups] = 1
        for t in (own_rows, own_batch, own_groups):
            dist.all_reduce(t)
            assert bool((t == 1).all())
        # weak-scaling bookkeeping of the benchmark: the job's time is the slowest rank's
        t = torch.tensor([1.0 + rank], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert float(t) == float(world)
    finally:
        dist.destroy_process_group()


def test_two_ranks_partition_every_operation_over_gloo():
    world = 2
    Ms = inputs.grouped_sizes(16, 128, 4096)
    mp.spawn(_worker, args=(world, _free_port(), 4096, 128, Ms), nprocs=world, join=True)


def _wgrad_worker(rank, world, port):
    from oracle import oracle as orc
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        N, H, W, C, K, R, S = 5, 6, 7, 8, 8, 3, 3
        X = inputs.small_integers([N, H, W, C], 51, 1, -2, 2)
        dY = inputs.small_integers([N, H, W, K], 51, 3, -2, 2)
        n0, n1 = sharding.conv_images(N, world, rank)
        part, _ = orc.conv2d_wgrad(dY[n0:n1].contiguous(), X[n0:n1].contiguous(), (R, S), pad=(1, 1))
        dW = part.to(torch.float32)               # integers: exact in fp32
        sharding.reduce_weight_gradient(dW)
        full, _ = orc.conv2d_wgrad(dY, X, (R, S), pad=(1, 1))
        assert torch.equal(dW.double(), full)
        # the data gradient needs no exchange: each rank's images are its own rows of dX
        Wf = inputs.small_integers([K, R, S, C], 51, 2, -2, 2)
        mine, _ = orc.conv2d_dgrad(dY[n0:n1].contiguous(), Wf, (H, W), pad=(1, 1))
        whole, _ = orc.conv2d_dgrad(dY, Wf, (H, W), pad=(1, 1))
        assert torch.equal(mine, whole[n0:n1])
    finally:
        dist.destroy_process_group()


def test_two_ranks_data_parallel_conv_gradients_over_gloo():
    mp.spawn(_wgrad_worker, args=(2, _free_port()), nprocs=2, join=True)


def _shard_worker(rank, world, port):
    """Each rank computes its shard of a small GEMM, batched GEMM, convolution and grouped GEMM (the oracle stands in for
    the per-rank kernel); gathered over gloo, the shards must reproduce the whole problem exactly."""
    from oracle import oracle as orc
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        def gather(mine, full_rows):
            # pad every rank's rows to the same count so that all_gather applies, then cut the padding off again
            pad = torch.zeros((full_rows,) + tuple(mine.shape[1:]), dtype=torch.float64)
            pad[:mine.shape[0]] = mine
            outs = [torch.zeros_like(pad) for _ in range(world)]
            dist.all_gather(outs, pad)
            return outs
        # GEMM: rows of A and D (cuts on the 256-row tile)
        M, N, K = 700, 40, 24
        A, B = inputs.small_integers([M, K], 61, 1), inputs.small_integers([N, K], 61, 2)
        whole, _ = orc.gemm(A, B, epi="relu")
        r0, r1 = sharding.gemm_rows(M, world, rank, 256)
        mine, _ = orc.gemm(A[r0:r1].contiguous(), B, epi="relu")
        parts = gather(mine, M)
        cuts = [sharding.gemm_rows(M, world, r, 256) for r in range(world)]
        assert torch.equal(torch.cat([parts[r][:c1 - c0] for r, (c0, c1) in enumerate(cuts)]), whole)
        # batched: batch entries
        Ab, Bb = inputs.small_integers([5, 16, 8], 62, 1), inputs.small_integers([5, 24, 8], 62, 2)
        wholeb, _ = orc.batched_gemm(Ab, Bb)
        b0, b1 = sharding.batch_entries(5, world, rank)
        mineb, _ = orc.batched_gemm(Ab[b0:b1].contiguous(), Bb[b0:b1].contiguous())
        partsb = gather(mineb, 5)
        cutsb = [sharding.batch_entries(5, world, r) for r in range(world)]
        assert torch.equal(torch.cat([partsb[r][:c1 - c0] for r, (c0, c1) in enumerate(cutsb)]), wholeb)
        # convolution: images
        X, Wf = inputs.small_integers([3, 6, 5, 8], 63, 6), inputs.small_integers([8, 3, 3, 8], 63, 7)
        wholec, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1))
        n0, n1 = sharding.conv_images(3, world, rank)
        minec, _ = orc.conv2d_fprop(X[n0:n1].contiguous(), Wf, pad=(1, 1))
        partsc = gather(minec, 3)
        cutsc = [sharding.conv_images(3, world, r) for r in range(world)]
        assert torch.equal(torch.cat([partsc[r][:c1 - c0] for r, (c0, c1) in enumerate(cutsc)]), wholec)
        # grouped: whole groups; every group is computed by exactly one rank
        Ms = [5, 0, 17, 9, 3]
        As = [inputs.small_integers([m, 8], 64 + g, 1) for g, m in enumerate(Ms)]
        Bs = [inputs.small_integers([12, 8], 64 + g, 2) for g in range(len(Ms))]
        owned = sharding.assign_groups(Ms, world)
        flags = torch.zeros(len(Ms))
        for g in owned[rank]:
            flags[g] = 1
        dist.all_reduce(flags)
        assert bool((flags == 1).all())
        for g in owned[rank]:
            if Ms[g]:
                assert torch.equal(orc.gemm(As[g], Bs[g])[0], orc.grouped_gemm(As, Bs)[0][g])
    finally:
        dist.destroy_process_group()


def test_two_ranks_shards_concatenate_to_the_whole_problem():
    mp.spawn(_shard_worker, args=(2, _free_port()), nprocs=2, join=True)
