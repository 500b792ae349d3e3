"""Pins for the oracle's arithmetic against what the paper and the mathematics fix (not GPU).

Each test names the passage it rests on. None of them re-types the oracle's loop: they use
closed forms, hand-computed steps, finite differences of the objective's *definition*
(Eq. 4), an equivalent linear-map formulation, exact rational/decimal evaluation of Eq. 6,
and cross-checks between independently written oracle variants.
"""
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
import wpsgd_inputs as wi

HINGE, LOGISTIC, SQUARED = 0, 1, 2
CONST, INV_SQRT = 0, 1


def one_shard(m):
    return np.array([0, m], dtype=np.int64)


def f32(x):
    return float(np.float32(x))


# ---- Eq. 5 with the loss term switched off: pure contraction (1 - eta lambda)^n (cf. Eq. 16) -------
@pytest.mark.parametrize("loss", [HINGE, LOGISTIC, SQUARED])
def test_pure_regulariser_decay(loss):
    d, m, n = 5, 7, 300
    X = np.zeros((m, d), dtype=np.float32)
    y = np.ones(m, dtype=np.float32)
    w0 = np.array([1.0, -2.0, 0.5, 4.0, -0.25], dtype=np.float32)
    eta, lam = f32(0.01), f32(0.3)
    W = oracle.run_dense(X, y, one_shard(m), np.array([n]), d, eta, CONST, lam, loss, 5, w0)
    want = (1.0 - eta * lam) ** n * w0.astype(np.float64)
    np.testing.assert_allclose(W[0], want, rtol=1e-12)


def test_pure_regulariser_decay_inv_sqrt_schedule():
    d, m, n = 3, 4, 200
    X = np.zeros((m, d), dtype=np.float32)
    y = np.ones(m, dtype=np.float32)
    w0 = np.array([4.0, 4.0, -1.0], dtype=np.float32)
    eta0, lam = f32(0.1), f32(0.5)
    W = oracle.run_dense(X, y, one_shard(m), np.array([n]), d, eta0, INV_SQRT, lam, HINGE, 1, w0)
    fac = 1.0
    for s in range(1, n + 1):
        fac *= 1.0 - eta0 / np.sqrt(s) * lam
    np.testing.assert_allclose(W[0], fac * w0.astype(np.float64), rtol=1e-12)


# ---- squared loss, d = 1, constant example: geometric convergence to the ridge solution ----------
def test_squared_loss_scalar_closed_form():
    x, yv = f32(1.5), f32(-0.7)
    eta, lam = f32(0.05), f32(0.2)
    m, n = 3, 40
    X = np.full((m, 1), x, dtype=np.float32)
    y = np.full(m, yv, dtype=np.float32)
    w0 = np.array([2.0], dtype=np.float32)
    W = oracle.run_dense(X, y, one_shard(m), np.array([n]), 1, eta, CONST, lam, SQUARED, 9, w0)
    w_star = x * yv / (lam + x * x)
    want = w_star + (1.0 - eta * lam - eta * x * x) ** n * (2.0 - w_star)
    assert W[0, 0] == pytest.approx(want, rel=1e-12)


# ---- one step from w = 0 ---------------------------------------------------------------------------
def test_first_step_from_zero():
    x = np.array([[0.5, -1.0, 2.0]], dtype=np.float32)
    eta, lam = f32(0.1), f32(0.01)
    for yv in (1.0, -1.0):
        y = np.array([yv], dtype=np.float32)
        run = lambda loss: oracle.run_dense(x, y, one_shard(1), np.array([1]), 3, eta, CONST, lam, loss, 0)[0]
        np.testing.assert_allclose(run(HINGE), eta * yv * x[0].astype(np.float64), rtol=1e-14)
        np.testing.assert_allclose(run(LOGISTIC), 0.5 * eta * yv * x[0].astype(np.float64), rtol=1e-14)
        np.testing.assert_allclose(run(SQUARED), eta * yv * x[0].astype(np.float64), rtol=1e-14)


# ---- four hinge steps worked by hand (Eq. 5; the last one has margin > 1, so only the regulariser acts)
def test_hinge_four_steps_by_hand():
    X = np.array([[1.0, 2.0]], dtype=np.float32)
    y = np.array([1.0], dtype=np.float32)
    eta, lam = f32(0.125), f32(0.5)  # exactly representable
    # step 1: z=0   -> w = eta*x                      = [0.125, 0.25]
    # step 2: z=.625 -> w = w(1-eta*lam) + eta*x       = [0.2421875, 0.484375]
    # step 3: z=1.2109375 >= 1 -> w = w(1-eta*lam)     = [0.22705078125, 0.4541015625]
    # step 4: z=1.13525390625 >= 1 -> again decay      = [0.212860107421875, 0.42572021484375]
    hand = {1: [0.125, 0.25], 2: [0.2421875, 0.484375], 3: [0.22705078125, 0.4541015625],
            4: [0.212860107421875, 0.42572021484375]}
    for n, want in hand.items():
        W = oracle.run_dense(X, y, one_shard(1), np.array([n]), 2, eta, CONST, lam, HINGE, 3)
        np.testing.assert_allclose(W[0], want, rtol=1e-15)


def test_hinge_tie_margin_exactly_one_takes_no_loss_step():
    X = np.array([[1.0, 0.0]], dtype=np.float32)
    y = np.array([1.0], dtype=np.float32)
    w0 = np.array([1.0, 3.0], dtype=np.float32)  # y z = 1 exactly
    W = oracle.run_dense(X, y, one_shard(1), np.array([1]), 2, f32(0.5), CONST, f32(0.5), HINGE, 0, w0)
    np.testing.assert_allclose(W[0], [0.75, 2.25], rtol=1e-15)


# ---- Eq. 4/5 through finite differences of the objective's definition ----------------------------
def _objective(loss, lam, x, yv, w):
    z = float(np.dot(w, x))
    if loss == HINGE:
        L = max(0.0, 1.0 - yv * z)
    elif loss == LOGISTIC:
        L = np.log1p(np.exp(-yv * z))
    else:
        L = 0.5 * (z - yv) ** 2
    return 0.5 * lam * float(np.dot(w, w)) + L


@pytest.mark.parametrize("loss", [HINGE, LOGISTIC, SQUARED])
@pytest.mark.parametrize("sched", [CONST, INV_SQRT])
def test_steps_follow_numerical_gradient_of_eq4(loss, sched):
    rng = np.random.default_rng(12 + loss)
    d, n_steps = 6, 6
    x = rng.normal(size=d).astype(np.float32)
    yv = -1.0
    X, y = x[None, :].copy(), np.array([yv], dtype=np.float32)
    w0 = (0.3 * rng.normal(size=d)).astype(np.float32)
    eta0, lam = f32(0.07), f32(0.4)
    w = w0.astype(np.float64)
    xd = x.astype(np.float64)
    h = 1e-6
    for n in range(1, n_steps + 1):
        grad = np.zeros(d)
        for c in range(d):
            e = np.zeros(d)
            e[c] = h
            grad[c] = (_objective(loss, lam, xd, yv, w + e) - _objective(loss, lam, xd, yv, w - e)) / (2 * h)
        eta = eta0 / np.sqrt(n) if sched == INV_SQRT else eta0
        w = w - eta * grad
        W = oracle.run_dense(X, y, one_shard(1), np.array([n]), d, eta0, sched, lam, loss, 77, w0)
        np.testing.assert_allclose(W[0], w, rtol=0, atol=2e-8 * n)
        w = W[0].copy()  # restart from the oracle's iterate so finite-difference error does not pile up


# ---- squared-loss chain == product of affine maps along the drawn index sequence ------------------
def test_squared_chain_equals_affine_map_product():
    rng = np.random.default_rng(5)
    k, d, m = 3, 4, 6
    X = rng.normal(size=(k * m, d)).astype(np.float32)
    y = rng.normal(size=k * m).astype(np.float32)
    off = np.arange(k + 1, dtype=np.int64) * m
    n_steps = np.array([9, 0, 4], dtype=np.int64)
    eta, lam, seed = f32(0.05), f32(0.1), 42
    w0 = rng.normal(size=d).astype(np.float32)
    W = oracle.run_dense(X, y, off, n_steps, d, eta, CONST, lam, SQUARED, seed, w0)
    for j in range(k):
        idx = oracle.sample_indices(seed, j, m, 0, int(n_steps[j]))
        A = np.eye(d + 1)  # homogeneous coordinates
        for i in idx:
            x = X[off[j] + i].astype(np.float64)
            M = np.eye(d + 1)
            M[:d, :d] = (1 - eta * lam) * np.eye(d) - eta * np.outer(x, x)
            M[:d, d] = eta * float(y[off[j] + i]) * x
            A = M @ A
        want = (A @ np.append(w0.astype(np.float64), 1.0))[:d]
        np.testing.assert_allclose(W[j], want, rtol=1e-11, atol=1e-13)
    np.testing.assert_array_equal(W[1], w0.astype(np.float64))  # a node that did no work keeps w0


def test_each_node_reads_only_its_own_shard():
    rng = np.random.default_rng(8)
    k, d, m = 3, 5, 10
    X = rng.normal(size=(k * m, d)).astype(np.float32)
    y = np.sign(rng.normal(size=k * m)).astype(np.float32)
    off = np.array([0, 10, 13, 30], dtype=np.int64)  # unequal shards
    n_steps = np.array([50, 50, 50], dtype=np.int64)
    base = oracle.run_dense(X, y, off, n_steps, d, f32(0.05), CONST, f32(0.01), LOGISTIC, 3)
    for j in range(k):
        Xp, yp = X.copy(), y.copy()
        mask = np.ones(k * m, dtype=bool)
        mask[off[j]:off[j + 1]] = False
        Xp[mask] = np.nan
        yp[mask] = np.nan
        Wp = oracle.run_dense(Xp, yp, off, n_steps, d, f32(0.05), CONST, f32(0.01), LOGISTIC, 3)
        np.testing.assert_array_equal(Wp[j], base[j])
        assert np.isfinite(Wp[j]).all()


def test_bf16_rows_are_widened_exactly():
    rng = np.random.default_rng(2)
    d, m = 16, 12
    Xb = torch.from_numpy(rng.normal(size=(m, d)).astype(np.float32)).to(torch.bfloat16)
    y = rng.normal(size=m).astype(np.float32)
    a = oracle.run_dense(Xb, y, one_shard(m), np.array([30]), d, f32(0.05), CONST, f32(0.1), SQUARED, 6)
    b = oracle.run_dense(Xb.float().numpy(), y, one_shard(m), np.array([30]), d, f32(0.05), CONST, f32(0.1), SQUARED, 6)
    np.testing.assert_array_equal(a, b)


def test_row_stride_is_honoured():
    rng = np.random.default_rng(3)
    d, ld, m = 5, 8, 9
    Xp = rng.normal(size=(m, ld)).astype(np.float32)
    y = np.sign(rng.normal(size=m)).astype(np.float32)
    a = oracle.run_dense(Xp, y, one_shard(m), np.array([25]), d, f32(0.1), CONST, f32(0.1), HINGE, 4)
    b = oracle.run_dense(np.ascontiguousarray(Xp[:, :d]), y, one_shard(m), np.array([25]), d, f32(0.1), CONST, f32(0.1),
                         HINGE, 4)
    np.testing.assert_array_equal(a, b)


def test_segmented_run_equals_one_run():
    wl = wi.config1(k=3, d=8, m=32, n_steps=(40, 25, 10))
    full = oracle.run_dense(wl.X, wl.y, wl.shard_off, wl.n_steps, wl.d, wl.eta0, INV_SQRT, wl.lam, wl.loss, wl.seed)
    first = np.minimum(wl.n_steps, 15)
    W = oracle.run_dense(wl.X, wl.y, wl.shard_off, first, wl.d, wl.eta0, INV_SQRT, wl.lam, wl.loss, wl.seed)
    rest = wl.n_steps - first
    # all nodes ran 15 steps or finished; continue the ones that have steps left
    assert (first[rest > 0] == 15).all()
    W2 = oracle.run_dense(wl.X, wl.y, wl.shard_off, rest, wl.d, wl.eta0, INV_SQRT, wl.lam, wl.loss, wl.seed,
                          step_begin=15, W_resume=W)
    np.testing.assert_array_equal(W2, full)


# ---- sparse variants ---------------------------------------------------------------------------------
def _small_sparse(loss=HINGE, sched=INV_SQRT):
    wl = wi.config4(k=3, d=64, m=40, base_steps=120, mean_nnz=6.0, max_nnz=16)
    wl.loss, wl.sched = loss, sched
    if loss == SQUARED:
        wl.eta0 = 0.05
    return wl


@pytest.mark.parametrize("loss", [HINGE, LOGISTIC, SQUARED])
@pytest.mark.parametrize("sched", [CONST, INV_SQRT])
def test_csr_literal_equals_dense_on_densified_rows(loss, sched):
    wl = _small_sparse(loss, sched)
    wl.lam = 0.05
    w0 = torch.full((wl.d,), 0.25)
    dn = wi.densify(wl)
    a = oracle.run_csr(wl.row_ptr, wl.col_idx, wl.val, wl.y, wl.shard_off, wl.n_steps, wl.d, wl.eta0, sched, wl.lam,
                       loss, wl.seed, w0, literal=True)
    b = oracle.run_dense(dn.X, dn.y, dn.shard_off, dn.n_steps, dn.d, wl.eta0, sched, wl.lam, loss, wl.seed, w0)
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-15)
    assert np.abs(a).max() > 0


@pytest.mark.parametrize("loss", [HINGE, LOGISTIC, SQUARED])
def test_csr_scaled_form_equals_literal(loss):
    wl = _small_sparse(loss)
    wl.lam = 0.05
    w0 = torch.full((wl.d,), -0.5)
    a = oracle.run_csr(wl.row_ptr, wl.col_idx, wl.val, wl.y, wl.shard_off, wl.n_steps, wl.d, wl.eta0, wl.sched,
                       wl.lam, loss, wl.seed, w0, literal=True)
    b = oracle.run_csr(wl.row_ptr, wl.col_idx, wl.val, wl.y, wl.shard_off, wl.n_steps, wl.d, wl.eta0, wl.sched,
                       wl.lam, loss, wl.seed, w0, literal=False)
    np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-14)
    one = oracle.run_csr(wl.row_ptr, wl.col_idx, wl.val, wl.y, wl.shard_off, wl.n_steps, wl.d, wl.eta0, wl.sched,
                         wl.lam, loss, wl.seed, w0, literal=False, one_node=2)
    np.testing.assert_array_equal(one, b[2])


@pytest.mark.parametrize("loss", [HINGE, LOGISTIC, SQUARED])
def test_csr_scaled_form_folds_its_scale_back_and_still_equals_literal(loss):
    """eta*lambda = 0.5 for 400 steps: the scale factor passes 1e-100 after 333 steps (0.5^333 = 5.7e-101), so the
    scaled form multiplies it back into u on the way; the literal O(d) form has no scale at all."""
    wl = _small_sparse(loss)
    wl.sched, wl.eta0, wl.lam = 0, 0.5, 1.0
    wl.n_steps = np.array([400, 340, 5], dtype=np.int64)[: wl.k] if wl.k <= 3 else np.array(
        [400, 340, 5] + [332] * (wl.k - 3), dtype=np.int64)
    assert 0.5 ** int(wl.n_steps.max()) < 1e-100
    w0 = torch.full((wl.d,), 2.0)
    a = oracle.run_csr(wl.row_ptr, wl.col_idx, wl.val, wl.y, wl.shard_off, wl.n_steps, wl.d, wl.eta0, wl.sched,
                       wl.lam, loss, wl.seed, w0, literal=True)
    b = oracle.run_csr(wl.row_ptr, wl.col_idx, wl.val, wl.y, wl.shard_off, wl.n_steps, wl.d, wl.eta0, wl.sched,
                       wl.lam, loss, wl.seed, w0, literal=False)
    for j in range(wl.k):
        assert np.linalg.norm(a[j]) > 0
        assert np.linalg.norm(a[j] - b[j]) <= 1e-11 * np.linalg.norm(a[j]), j
    # and the chains really went through the branch: untouched coordinates carry w0 * 0.5^n, far below 1e-100
    assert 0 < np.abs(a[0]).min() < 1e-100


# ---- Eq. 6 / Eq. 8 weights, Eq. 7 / Eq. 9 condition --------------------------------------------------
def _decimal_weights(n_steps, r):
    getcontext().prec = 60
    t = max(n_steps)
    p = [Decimal(r) ** (t - n) for n in n_steps]
    s = sum(p)
    return [float(x / s) for x in p], float(s)


def test_weights_sum_to_one_and_ratios():
    n = np.array([1000, 800, 500, 250, 1000], dtype=np.int64)
    eta, lam = f32(0.01), f32(1e-3)
    w, _, tot = oracle.weights(n, eta, CONST, lam)
    assert abs(w.sum() - 1.0) < 1e-15  # premise of Lemma 2
    r = 1.0 - eta * lam
    for i in range(5):
        for j in range(5):
            assert w[i] / w[j] == pytest.approx(r ** float(n[j] - n[i]), rel=1e-12)
    assert w[0] == w[4] and w[0] > w[1] > w[2] > w[3]  # the fastest node weighs most
    assert tot == pytest.approx(sum(r ** float(1000 - x) for x in n), rel=1e-13)


def test_weights_worked_values_exact_arithmetic():
    # config 1: eta*lambda = 1e-5 up to fp32 rounding of the two factors
    for n, eta, lam in [([1000, 800, 500, 250], f32(0.01), f32(1e-3)),
                        ([20000, 10000, 5000] * 5 + [20000], f32(0.05), f32(1e-4))]:
        r_exact = Fraction(1) - Fraction(eta) * Fraction(lam)
        want, tot = _decimal_weights(n, Decimal(r_exact.numerator) / Decimal(r_exact.denominator))
        got, _, gtot = oracle.weights(np.array(n, dtype=np.int64), eta, CONST, lam)
        np.testing.assert_allclose(got, want, rtol=1e-12)
        assert gtot == pytest.approx(tot, rel=1e-12)
    # values one gets from Eq. 6 with r = 1 - 1e-5 and delays 0, 200, 500, 750
    got, _, _ = oracle.weights(np.array([1000, 800, 500, 250]), f32(0.01), CONST, f32(1e-3))
    np.testing.assert_allclose(got, [0.250906874, 0.250405559, 0.249655465, 0.249032102], atol=2e-9)


def test_weights_paper_experiment_setting_with_fitted_rate():
    # Section "Real-world data": 8 fast nodes, 2 slow nodes with one fifth of the data, r = 0.99999 (Eq. 8);
    # at t = 800000 a slow node has run 160000 steps, delay 640000.
    n = np.array([800000] * 8 + [160000] * 2, dtype=np.int64)
    got, holds, tot = oracle.weights(n, f32(1e-4), CONST, f32(0.01), r=0.99999)
    want, wtot = _decimal_weights(list(n), Decimal(0.99999))  # the double nearest to 0.99999, exactly
    np.testing.assert_allclose(got, want, rtol=1e-11)
    assert got[0] == pytest.approx(0.124948100, abs=1e-8)
    assert got[9] == pytest.approx(2.07602e-4, rel=1e-4)
    # Eq. 9: 2 * (8 + 2 * 0.99999^640000) > sqrt(10) + 10
    assert holds and 2 * tot > np.sqrt(10) + 10
    # default rate r = 1 - eta*lambda = 0.999999 instead
    got2, _, _ = oracle.weights(n, f32(1e-4), CONST, f32(0.01))
    assert got2[0] == pytest.approx(0.110441, abs=2e-6)
    assert got2[9] == pytest.approx(0.058235, abs=2e-6)


def test_equal_work_gives_simuparallel_average():
    # all delays zero: Eq. 6 gives 1/k, i.e. Algorithm 2's plain average
    for k in (1, 2, 7, 16):
        w, _, _ = oracle.weights(np.full(k, 123, dtype=np.int64), f32(0.1), CONST, f32(0.1))
        np.testing.assert_array_equal(w, np.full(k, 1.0 / k))
    wl = wi.config2(k=4, d=16, m=64, base_steps=60)
    wl.n_steps[:] = 60
    v, W, wts = oracle.solve(wl)
    np.testing.assert_allclose(v, W.mean(axis=0), rtol=1e-14, atol=1e-16)


def test_rate_one_is_direct_averaging_and_single_node_is_sequential_sgd():
    n = np.array([100, 10, 55], dtype=np.int64)
    w, _, _ = oracle.weights(n, f32(0.1), CONST, f32(0.1), r=1.0)
    np.testing.assert_array_equal(w, np.full(3, 1.0 / 3))
    wl = wi.config1(k=1, d=8, m=32, n_steps=(50,))
    v, W, wts = oracle.solve(wl)
    assert wts[0] == 1.0
    np.testing.assert_array_equal(v, W[0])


def test_condition_of_corollary_3():
    # k = 1: 2 * 1 > 1 + 1 is false
    assert oracle.weights(np.array([10]), f32(0.1), CONST, f32(0.1))[1] is False
    # config 1 and 2 settings
    _, h1, t1 = oracle.weights(np.array([1000, 800, 500, 250]), f32(0.01), CONST, f32(1e-3))
    assert h1 and t1 == pytest.approx(3.985542, abs=1e-6)
    n2 = (20000 * np.array([1.0, 0.5, 0.25])[np.arange(16) % 3]).astype(np.int64)
    _, h2, t2 = oracle.weights(n2, f32(0.05), CONST, f32(1e-4))
    assert h2 and 2 * t2 == pytest.approx(30.79, abs=0.01)
    # heavy delays break it: sum r^T ~ 1 for k = 4 -> 2 > 6 false
    assert oracle.weights(np.array([10 ** 6, 1, 1, 1]), f32(0.1), CONST, f32(0.1))[1] is False


def test_weights_decaying_schedule_product_form():
    n = np.array([400, 130, 0, 399], dtype=np.int64)
    eta0, lam = f32(0.1), f32(0.5)
    got, _, _ = oracle.weights(n, eta0, INV_SQRT, lam)
    getcontext().prec = 50
    t = 400
    p = []
    for nj in n:
        f = Decimal(1)
        for s in range(int(nj) + 1, t + 1):
            f *= Decimal(1) - Decimal(eta0) * Decimal(lam) / Decimal(s).sqrt()
        p.append(f)
    want = [float(x / sum(p)) for x in p]
    np.testing.assert_allclose(got, want, rtol=1e-11)
    # a node that did nothing still gets a (small) weight and keeps w0
    assert 0 < got[2] < got[1] < got[3] < got[0]


def test_weights_reject_negative_steps():
    with pytest.raises(ValueError):
        oracle.weights(np.array([5, -1]), f32(0.1), CONST, f32(0.1))


def test_combine_is_the_weighted_sum():
    rng = np.random.default_rng(1)
    W = rng.normal(size=(5, 9))
    wts = rng.random(5)
    wts /= wts.sum()
    v = oracle.combine(W, wts)
    np.testing.assert_allclose(v, wts @ W, rtol=1e-14)
    # not the transpose, not unweighted
    e = np.zeros(5)
    e[3] = 1.0
    np.testing.assert_array_equal(oracle.combine(W, e), W[3])


def test_whole_path_relabelling_nodes_permutes_nothing_but_order():
    # v does not depend on how nodes are numbered when their streams move with them: build the same
    # problem with shards swapped and per-node results must swap (k=2, node id enters the stream,
    # so compare W of node j with a run where that shard sits at the same node position).
    wl = wi.config1(k=2, d=8, m=16, n_steps=(30, 12))
    v, W, wts = oracle.solve(wl)
    np.testing.assert_allclose(v, wts[0] * W[0] + wts[1] * W[1], rtol=1e-15)
    assert wts[0] > wts[1]


def test_objective_and_error_rate_by_hand():
    X = np.array([[1.0, 0.0], [0.0, 2.0], [1.0, 1.0]], dtype=np.float32)
    y = np.array([1.0, -1.0, 1.0], dtype=np.float32)
    w = np.array([0.5, 0.25])
    # margins z = .5, .5, .75 ; hinge losses: .5, 1.5, .25 -> mean .75 ; reg = .5*lam*(.3125)
    obj, err = oracle.objective_dense(X, y, w, f32(0.5), HINGE)
    assert obj == pytest.approx(0.75 + 0.5 * 0.5 * 0.3125, rel=1e-14)
    assert err == pytest.approx(1.0 / 3.0)
    obj, _ = oracle.objective_dense(X, y, w, f32(0.0), SQUARED)
    assert obj == pytest.approx((0.125 + 0.5 * 2.25 + 0.5 * 0.0625) / 3, rel=1e-14)
    obj, _ = oracle.objective_dense(X, y, w, f32(0.0), LOGISTIC)
    assert obj == pytest.approx((np.log1p(np.exp(-0.5)) + np.log1p(np.exp(0.5)) + np.log1p(np.exp(-0.75))) / 3,
                                rel=1e-14)


def test_csr_objective_by_hand_and_against_dense():
    # rows: [1, 0], [0, 2], [1, 1] as CSR; same numbers as the dense hand example above
    rp = np.array([0, 1, 2, 4], dtype=np.int64)
    ci = np.array([0, 1, 0, 1], dtype=np.int32)
    va = np.array([1.0, 2.0, 1.0, 1.0], dtype=np.float32)
    y = np.array([1.0, -1.0, 1.0], dtype=np.float32)
    w = np.array([0.5, 0.25])
    obj, err = oracle.objective_csr(rp, ci, va, y, w, f32(0.5), HINGE)
    assert obj == pytest.approx(0.75 + 0.5 * 0.5 * 0.3125, rel=1e-14)
    assert err == pytest.approx(1.0 / 3.0)
    wl = _small_sparse()
    dn = wi.densify(wl)
    wv = np.random.default_rng(0).normal(size=wl.d)
    for loss in (HINGE, LOGISTIC, SQUARED):
        a = oracle.objective_csr(wl.row_ptr, wl.col_idx, wl.val, wl.y, wv, f32(0.1), loss)
        b = oracle.objective_dense(dn.X, dn.y, wv, f32(0.1), loss)
        assert a[0] == pytest.approx(b[0], rel=1e-12) and a[1] == b[1]
