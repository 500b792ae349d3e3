"""Evaluation measures on sparse rows, and the qualitative claim of the paper's experiments on data regenerated
from its "analog data" recipe: with two of ten nodes consuming a fifth of the data, the weighted combination
(Eq. 6) stays close to the balanced run and clearly beats averaging the models directly (Table II and
Fig. 6 show this ordering; their numbers need the paper's own data and are not reproduced)."""
import numpy as np
import pytest
import torch

import oracle
import wpsgd_inputs as wi

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P(wpsgd_lib):
    import paper_1708_04801_b200 as pkg

    return pkg


@pytest.mark.parametrize("loss", [0, 1, 2])
def test_objective_csr_matches_oracle(P, loss):
    rp, ci, va, y = wi.analog_rows(777, 5000, data_seed=5)
    w = torch.randn(5000, generator=torch.Generator().manual_seed(1)) / 4
    with P.Context(2, 5000) as ctx:
        out = ctx.objective_csr(rp.cuda(), ci.cuda(), va.cuda(), y.cuda(), w.cuda(), 0.01, loss).cpu().numpy()
        ctx.check()
    obj, err = oracle.objective_csr(rp, ci, va, y, w.numpy().astype(np.float64), 0.01, loss)
    assert out[0] == pytest.approx(obj, rel=1e-5)
    assert abs(out[1] - err) <= 2.0 / 777


def test_weighted_combination_tracks_the_balanced_run_on_analog_data(P):
    d, lam, eta, t = 100000, 0.01, 0.01, 20000
    rows = [4000] * 8 + [800] * 2  # two slow nodes hold a fifth of the data
    n_train = sum(rows)
    rp, ci, va, y = wi.analog_rows(n_train + 4000, d, data_seed=2001)
    off = np.concatenate([[0], np.cumsum(rows)]).astype(np.int64)
    p0 = int(rp[n_train])
    test = ((rp[n_train:] - p0).cuda(), ci[p0:].cuda(), va[p0:].cuda(), y[n_train:].cuda())
    train = (rp[:n_train + 1].cuda(), ci[:p0].cuda(), va[:p0].cuda(), y[:n_train].cuda())
    w0 = torch.full((d,), 4.0, device="cuda")  # the paper's experiments start from the constant vector 4
    unbalanced = np.array([t] * 8 + [t // 5] * 2, dtype=np.int64)
    balanced = np.full(10, t, dtype=np.int64)
    obj = {}
    with P.Context(10, d) as ctx:
        for name, n, r in (("balanced", balanced, 0.0), ("weighted", unbalanced, 0.0), ("direct", unbalanced, 1.0)):
            ctx.run_csr(*train, off, n, eta, 0, lam, 0, 7, w0)
            v = ctx.combine(r)
            obj[name] = float(ctx.objective_csr(*test, v, lam, 0).cpu()[0])
            if name == "weighted":
                v_weighted = v.cpu().numpy()
        ctx.check()
    assert obj["balanced"] < obj["weighted"] < obj["direct"]
    assert obj["weighted"] - obj["balanced"] < 0.35 * (obj["direct"] - obj["balanced"])
    # and the GPU's weighted model is the oracle's
    W = oracle.run_csr(rp[:n_train + 1], ci[:p0], va[:p0], y[:n_train], off, unbalanced, d, eta, 0, lam, 0, 7, w0.cpu())
    wts, _, _ = oracle.weights(unbalanced, eta, 0, lam)
    ov = oracle.combine(W, wts)
    assert np.linalg.norm(v_weighted - ov) / np.linalg.norm(ov) <= 1e-3
