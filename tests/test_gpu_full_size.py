"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (default options).

Every node's final model and the combined model are compared with the CPU oracle. The large workloads live in
device memory only, so the oracle is fed one shard at a time: the rows of node j are copied back from the device
and the oracle runs that node alone (its number still enters the sample stream); nodes are independent until the
combination, which the oracle then forms from its own models and its own weights. Several nodes are checked at a
time on host threads (the oracle itself stays single-threaded per call)."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle
import wpsgd_inputs as wi

pytestmark = pytest.mark.gpu

TOL = {0: 1e-3, 1: 1e-4, 2: 1e-4}


@pytest.fixture(scope="module")
def P(wpsgd_lib):
    import paper_1708_04801_b200 as pkg

    return pkg


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def run_gpu(P, wl):
    with P.Context(wl.k, wl.d) as ctx:
        ctx.run_workload(wl)
        v = ctx.combine().cpu().numpy()
        W = ctx.get_models()
        wts, _ = ctx.get_weights()
        ctx.check()
    return v, W, wts


def one_node_layout(wl, j):
    """Shard offsets and step counts that keep node j's number (it enters the sample stream) while only its
    shard is present in the arrays handed to the oracle."""
    m = int(wl.shard_off[j + 1] - wl.shard_off[j])
    off = np.zeros(wl.k + 1, dtype=np.int64)
    off[j + 1:] = m
    n = np.zeros(wl.k, dtype=np.int64)
    n[j] = wl.n_steps[j]
    return off, n, m


WORKERS = max(1, min(16, (os.cpu_count() or 2) - 1))


def oracle_all_nodes(wl, fetch):
    """Oracle models of every node, [k, d] float64; fetch(j) copies node j's shard to the host and returns the
    oracle's final model of that node."""
    oW = np.zeros((wl.k, wl.d), dtype=np.float64)

    def one(j):
        oW[j] = fetch(j)
        return j

    with ThreadPoolExecutor(max_workers=WORKERS) as ex:
        list(ex.map(one, range(wl.k)))
    return oW


def dense_node(wl, j):
    off, n, m = one_node_layout(wl, j)
    lo = int(wl.shard_off[j])
    Xj, yj = wl.X[lo:lo + m].cpu(), wl.y[lo:lo + m].cpu()
    return oracle.run_dense(Xj, yj, off, n, wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)[j]


def csr_node(wl, j):
    off, n, m = one_node_layout(wl, j)
    lo = int(wl.shard_off[j])
    rp = wl.row_ptr[lo:lo + m + 1]
    p0, p1 = int(rp[0]), int(rp[-1])
    return oracle.run_csr((rp - p0).cpu(), wl.col_idx[p0:p1].cpu(), wl.val[p0:p1].cpu(), wl.y[lo:lo + m].cpu(), off, n,
                          wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed, one_node=j)


def assert_all_nodes_and_combination(v, W_dev, wts, wl, node_fn):
    tol = TOL[wl.loss]
    owts, _, _ = oracle.weights(wl.n_steps, wl.eta0, wl.sched, wl.lam)
    np.testing.assert_allclose(wts, owts, rtol=1e-12)
    oW = oracle_all_nodes(wl, lambda j: node_fn(wl, j))
    W = W_dev.cpu().numpy()
    errs = np.array([rel_l2(W[j], oW[j]) for j in range(wl.k)])
    worst = int(np.argmax(errs))
    assert errs[worst] <= tol, f"node {worst}: {errs[worst]:.3e} > {tol} (steps {int(wl.n_steps[worst])})"
    ov = oracle.combine(oW, owts)
    assert rel_l2(v, ov) <= tol, f"combined model: {rel_l2(v, ov):.3e} > {tol}"


def test_config2_full(P):
    wl_cpu = wi.config2()
    v, W, wts = run_gpu(P, wl_cpu.to("cuda"))
    ov, oW, owts = oracle.solve(wl_cpu)
    W = W.cpu().numpy()
    assert max(rel_l2(W[j], oW[j]) for j in range(wl_cpu.k)) <= TOL[wl_cpu.loss]
    assert rel_l2(v, ov) <= TOL[wl_cpu.loss]


@pytest.mark.parametrize("rho", [1.0, 4.0, 16.0])
def test_config5_full_every_node(P, rho):
    wl = wi.config5(rho=rho, device="cuda")
    assert wl.total_steps == 1 << 24 and wl.k == 1024
    v, W, wts = run_gpu(P, wl)
    assert_all_nodes_and_combination(v, W, wts, wl, dense_node)


def test_config3_full_every_node(P):
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs 40 GiB of free device memory")
    wl = wi.config3(device="cuda")
    assert wl.k == 128 and wl.d == 4096 and wl.X.dtype == torch.bfloat16
    v, W, wts = run_gpu(P, wl)
    assert_all_nodes_and_combination(v, W, wts, wl, dense_node)
    del wl
    torch.cuda.empty_cache()


def test_config4_full_every_node(P):
    wl = wi.config4(device="cuda")
    assert wl.k == 64 and wl.d == 1 << 20
    v, W, wts = run_gpu(P, wl)
    assert_all_nodes_and_combination(v, W, wts, wl, csr_node)
    del wl
    torch.cuda.empty_cache()
