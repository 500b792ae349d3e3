"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (default options).

The CPU oracle cannot run every chain of the large workloads in reasonable time or memory, so for
those it is run on sampled nodes, one by one, on exactly the rows the GPU used (copied back from the
device), and the combined model is checked through the property that ties it to the per-node models:
v = sum_j weight_j w_j with the oracle's weights."""
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


def check_combination(v, W_dev, wts, wl):
    owts, _, _ = oracle.weights(wl.n_steps, wl.eta0, wl.sched, wl.lam)
    np.testing.assert_allclose(wts, owts, rtol=1e-12)
    want = (torch.from_numpy(owts).to(W_dev.device)[:, None] * W_dev.double()).sum(0).cpu().numpy()
    np.testing.assert_allclose(v, want, rtol=1e-5, atol=1e-9)


def test_config2_full(P):
    wl_cpu = wi.config2()
    v, W, wts = run_gpu(P, wl_cpu.to("cuda"))
    ov, oW, owts = oracle.solve(wl_cpu)
    W = W.cpu().numpy()
    assert max(rel_l2(W[j], oW[j]) for j in range(wl_cpu.k)) <= TOL[wl_cpu.loss]
    assert rel_l2(v, ov) <= TOL[wl_cpu.loss]


@pytest.mark.parametrize("rho", [1.0, 16.0])
def test_config5_full_sampled_nodes(P, rho):
    wl = wi.config5(rho=rho, device="cuda")
    assert wl.total_steps == 1 << 24
    v, W, wts = run_gpu(P, wl)
    check_combination(v, W, wts, wl)
    for j in (0, 1, 511, 1023):
        off, n, m = one_node_layout(wl, j)
        lo = int(wl.shard_off[j])
        Xj, yj = wl.X[lo:lo + m].cpu(), wl.y[lo:lo + m].cpu()
        oW = oracle.run_dense(Xj, yj, off, n, wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
        assert rel_l2(W[j].cpu().numpy(), oW[j]) <= TOL[wl.loss], f"node {j}"


def test_config3_full_sampled_nodes(P):
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs 40 GiB of free device memory")
    wl = wi.config3(device="cuda")
    v, W, wts = run_gpu(P, wl)
    check_combination(v, W, wts, wl)
    longest, shortest = int(np.argmax(wl.n_steps)), int(np.argmin(wl.n_steps))
    for j in sorted({0, longest, shortest, 127}):
        off, n, m = one_node_layout(wl, j)
        lo = int(wl.shard_off[j])
        Xj, yj = wl.X[lo:lo + m].cpu(), wl.y[lo:lo + m].cpu()
        oW = oracle.run_dense(Xj, yj, off, n, wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
        assert rel_l2(W[j].cpu().numpy(), oW[j]) <= TOL[wl.loss], f"node {j}"
    del wl
    torch.cuda.empty_cache()


def test_config4_full_sampled_nodes(P):
    wl = wi.config4(device="cuda")
    assert wl.k == 64 and wl.d == 1 << 20
    v, W, wts = run_gpu(P, wl)
    check_combination(v, W, wts, wl)
    for j in (0, 3, 62):
        off, n, m = one_node_layout(wl, j)
        lo = int(wl.shard_off[j])
        rp = wl.row_ptr[lo:lo + m + 1]
        p0, p1 = int(rp[0]), int(rp[-1])
        oWj = oracle.run_csr((rp - p0).cpu(), wl.col_idx[p0:p1].cpu(), wl.val[p0:p1].cpu(), wl.y[lo:lo + m].cpu(), off, n,
                             wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed, one_node=j)
        assert rel_l2(W[j].cpu().numpy(), oWj) <= TOL[wl.loss], f"node {j}"
    del wl
    torch.cuda.empty_cache()
