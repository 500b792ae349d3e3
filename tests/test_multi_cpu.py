"""Multi-GPU layout of the path, exercised on CPU: two gloo ranks each hold a subset of the nodes,
compute their partial weighted combination (the chains stand in for the kernels through the CPU
checker, which tests may use) and add the partials with the single all-reduce the method has."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
import wpsgd_inputs as wi


def test_partition_covers_every_node_once_and_balances(wpsgd_lib):
    from paper_1708_04801_b200 import multi

    n = np.array([20000, 10000, 5000] * 5 + [20000])
    for G in (1, 2, 3, 8):
        parts = multi.partition_nodes(n, G)
        allj = np.sort(np.concatenate(parts))
        assert np.array_equal(allj, np.arange(len(n)))
        loads = [int(n[p].sum()) for p in parts]
        assert max(loads) - min(loads) <= int(n.max())
    a, b = multi.partition_nodes(n, 2), multi.partition_nodes(n, 2)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))


def test_local_weights_are_the_global_weights_restricted(wpsgd_lib):
    from paper_1708_04801_b200 import multi

    n = np.array([1000, 800, 500, 250, 1000, 10])
    parts = multi.partition_nodes(n, 2)
    full, _, _ = oracle.weights(n, 0.01, 0, 1e-3)
    tot = 0.0
    for p in parts:
        w = multi.local_weights(n, p, 0.01, 0, 1e-3)
        np.testing.assert_allclose(w, full[p], rtol=1e-12)
        tot += w.sum()
    assert abs(tot - 1.0) < 1e-14


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank_main(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_1708_04801_b200 import multi

        wl = wi.config1(k=5, d=16, m=32, n_steps=(120, 90, 60, 30, 0))
        parts = multi.partition_nodes(wl.n_steps, world)
        mine = parts[rank]
        # this rank runs only its nodes (others get zero steps); node numbers stay global
        n_local = np.zeros_like(wl.n_steps)
        n_local[mine] = wl.n_steps[mine]
        W = oracle.run_dense(wl.X, wl.y, wl.shard_off, n_local, wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
        w_local = multi.local_weights(wl.n_steps, mine, wl.eta0, wl.sched, wl.lam)
        partial = torch.from_numpy((w_local[:, None] * W[mine]).sum(0))
        v = multi.allreduce_sum(partial)
        if rank == 0:
            q.put(v.numpy())
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_process_combination(wpsgd_lib):
    wl = wi.config1(k=5, d=16, m=32, n_steps=(120, 90, 60, 30, 0))
    want, _, _ = oracle.solve(wl)
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)
