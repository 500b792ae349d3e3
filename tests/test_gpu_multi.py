"""The device side of the multi-GPU layout, on one GPU: every "rank" is a context that holds only its own nodes'
shards, tells the library their global numbers (wpsgd_set_node_ids) and combines them with their global Eq. 6
weights (wpsgd_combine_weighted); the partial combinations are then added, which is all the exchange Algorithm 1's
last line needs. The sum must be the single-context result, and each rank's models must be the same nodes' models
of the single-context run bit for bit (same sample stream, same kernel, same arithmetic)."""
import numpy as np
import pytest
import torch

import oracle
import wpsgd_inputs as wi

pytestmark = pytest.mark.gpu

TOL = {0: 1e-3, 1: 1e-4, 2: 1e-4}


def rel_l2(a, b):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def rank_view_dense(wl, owned):
    """Rows, labels, shard offsets and step counts of the owned nodes only, packed."""
    rows = [torch.arange(int(wl.shard_off[j]), int(wl.shard_off[j + 1])) for j in owned]
    sel = torch.cat(rows)
    off = np.zeros(len(owned) + 1, dtype=np.int64)
    off[1:] = np.cumsum([r.numel() for r in rows])
    return wl.X[sel].contiguous(), wl.y[sel].contiguous(), off, wl.n_steps[owned]


def rank_view_csr(wl, owned):
    rps, cols, vals, ys = [torch.zeros(1, dtype=torch.int64)], [], [], []
    off = [0]
    base = 0
    for j in owned:
        lo, hi = int(wl.shard_off[j]), int(wl.shard_off[j + 1])
        rp = wl.row_ptr[lo:hi + 1]
        p0, p1 = int(rp[0]), int(rp[-1])
        rps.append(rp[1:] - p0 + base)
        base += p1 - p0
        cols.append(wl.col_idx[p0:p1])
        vals.append(wl.val[p0:p1])
        ys.append(wl.y[lo:hi])
        off.append(off[-1] + hi - lo)
    return (torch.cat(rps), torch.cat(cols).contiguous(), torch.cat(vals).contiguous(), torch.cat(ys).contiguous(),
            np.array(off, dtype=np.int64), wl.n_steps[owned])


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("kind", ["fp32", "bf16", "small_d", "csr"])
def test_partitioned_contexts_add_up_to_the_single_context_result(wpsgd_lib, world, kind):
    import paper_1708_04801_b200 as P
    from paper_1708_04801_b200 import multi

    if kind == "fp32":
        wl = wi.config2(k=12, d=1024, m=96, base_steps=400)
    elif kind == "bf16":
        wl = wi.config3(k=12, d=2048, m=64, n_lo=100, n_hi=500)
    elif kind == "small_d":
        wl = wi.config5(k=12, d=256, m=64, total_steps=12 * 300, rho=5.0)
    else:
        wl = wi.config4(k=12, d=4096, m=128, base_steps=400, mean_nnz=25.0)
    wl.n_steps[5] = 0  # a node that did no work still takes part in the combination
    ov, oW, owts = oracle.solve(wl)
    dev = wl.to("cuda")
    with P.Context(wl.k, wl.d) as ctx:
        ctx.run_workload(dev)
        v_single = ctx.combine().cpu().numpy()
        W_single = ctx.get_models().cpu().numpy()
        ctx.check()
    parts = multi.partition_nodes(wl.n_steps, world)
    assert sorted(np.concatenate(parts).tolist()) == list(range(wl.k))
    total = np.zeros(wl.d, dtype=np.float64)
    for owned in parts:
        w_local = multi.local_weights(wl.n_steps, owned, wl.eta0, wl.sched, wl.lam)
        np.testing.assert_allclose(w_local, owts[owned], rtol=1e-12)
        with P.Context(len(owned), wl.d) as ctx:
            ctx.set_node_ids(owned)
            if kind == "csr":
                rp, ci, va, y, off, n = rank_view_csr(wl, owned)
                ctx.run_csr(rp.cuda(), ci.cuda(), va.cuda(), y.cuda(), off, n, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
            else:
                X, y, off, n = rank_view_dense(wl, owned)
                ctx.run(X.cuda(), y.cuda(), off, n, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
            part = ctx.combine_weighted(w_local).cpu().numpy()
            W_part = ctx.get_models().cpu().numpy()
            ctx.check()
        np.testing.assert_array_equal(W_part, W_single[owned])  # placement does not change a node's chain
        total += part.astype(np.float64)
    assert rel_l2(total, v_single) <= 1e-6
    assert rel_l2(total, ov) <= TOL[wl.loss]


def test_set_node_ids_rejects_bad_input_and_can_be_reset(wpsgd_lib):
    import paper_1708_04801_b200 as P

    wl = wi.config1(k=3, d=64, m=32, n_steps=(40, 20, 10)).to("cuda")
    with P.Context(3, 64) as ctx:
        with pytest.raises(P.WpsgdError) as e:
            ctx.set_node_ids([0, -1, 2])
        assert e.value.status_name == "INVALID_ARG"
        ctx.run_workload(wl)
        base = ctx.get_models().cpu().numpy()
        ctx.set_node_ids([7, 8, 9])
        ctx.run_workload(wl)
        moved = ctx.get_models().cpu().numpy()
        assert not np.array_equal(moved, base)  # other node numbers, other draws
        ctx.set_node_ids(None)
        ctx.run_workload(wl)
        np.testing.assert_array_equal(ctx.get_models().cpu().numpy(), base)
        with pytest.raises(P.WpsgdError) as e:
            ctx.combine_weighted([0.5, float("nan"), 0.5])
        assert e.value.status_name == "INVALID_ARG"
        ctx.check()
