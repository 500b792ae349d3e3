"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs. Sample streams bit-exact; models within relative L2 error 1e-4 (logistic, squared)
or 1e-3 (hinge: a margin within rounding of 1 may flip one subgradient)."""
import numpy as np
import pytest
import torch

import oracle
import wpsgd_inputs as wi

pytestmark = pytest.mark.gpu

HINGE, LOGISTIC, SQUARED = 0, 1, 2
TOL = {HINGE: 1e-3, LOGISTIC: 1e-4, SQUARED: 1e-4}


@pytest.fixture(scope="module")
def P(wpsgd_lib):
    import paper_1708_04801_b200 as pkg

    return pkg


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a))


def gpu_solve(P, wl_cpu, options=None, r=0.0):
    wl = wl_cpu.to("cuda")
    with P.Context(wl.k, wl.d) as ctx:
        for k_, v_ in (options or {}).items():
            ctx.set_option(k_, v_)
        ctx.run_workload(wl)
        v = ctx.combine(r)
        W = ctx.get_models()
        wts, flag = ctx.get_weights(r)
        ctx.check()
        return v.cpu().numpy(), W.cpu().numpy(), wts, flag


def assert_parity(P, wl, options=None, r=0.0, tol=None):
    v, W, wts, flag = gpu_solve(P, wl, options, r)
    ov, oW, owts = oracle.solve(wl, r)
    tol = tol or TOL[wl.loss]
    np.testing.assert_allclose(wts, owts, rtol=1e-12)
    worst = max(rel_l2(W[j], oW[j]) for j in range(wl.k) if np.linalg.norm(oW[j]) > 0)
    assert worst <= tol, f"per-node model error {worst:.3e} > {tol}"
    err = rel_l2(v, ov)
    assert err <= tol, f"combined model error {err:.3e} > {tol}"
    return err


# ---- sample stream ------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed,node,m,n_begin,count", [
    (0, 0, 4096, 0, 1000), (0, 3, 4096, 0, 250), (1, 15, 8192, 0, 20001), (7, 2, 1, 0, 17),
    (0xFFFFFFFFFFFFFFFF, 1023, (1 << 32) - 1, 0, 4099), (5, 9, 65536, 1, 1), (5, 9, 65536, 2, 3), (5, 9, 65536, 3, 6),
    (5, 9, 65536, 1237, 3763), (0x123456789ABCDEF1, 77, 2047, 999999999, 1025), (3, 1, 10, 0, 0),
    (2, 4, 3, (1 << 34) + 1, 13),
])
def test_sample_stream_bit_exact(P, seed, node, m, n_begin, count):
    with P.Context(2, 8) as ctx:
        got = ctx.sample_indices(seed, node, m, n_begin, count).cpu().numpy().view(np.uint32)
        ctx.check()
    want = oracle.sample_indices(seed, node, m, n_begin, count)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("seed,node,m,n_begin,count", [
    (0, 0, 4096, 0, 9000), (3, 7, 1, 0, 5), (3, 7, 2, 1, 9), (9, 1023, 1000, 998, 1005), (5, 2, 65537, 0, 70000),
    (0xFFFFFFFFFFFFFFFF, 4, (1 << 32) - 1, (1 << 33) + 3, 257), (1, 1, 5, 0, 0),
])
def test_shuffled_sample_stream_bit_exact(P, seed, node, m, n_begin, count):
    oracle.set_sampling(1)
    try:
        want = oracle.sample_indices(seed, node, m, n_begin, count)
    finally:
        oracle.set_sampling(0)
    with P.Context(2, 8) as ctx:
        ctx.set_option("sampling", 1)
        got = ctx.sample_indices(seed, node, m, n_begin, count).cpu().numpy().view(np.uint32)
        ctx.check()
    assert np.array_equal(got, want)


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_small_workloads_shuffled_order(P, cfg):
    oracle.set_sampling(1)
    try:
        assert_parity(P, wi.small(cfg), {"sampling": 1})
    finally:
        oracle.set_sampling(0)


# ---- the five workloads, scaled down, default kernel choice ---------------------------------------------
@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_small_workloads_default_kernels(P, cfg):
    assert_parity(P, wi.small(cfg))


# ---- every dense kernel variant ----------------------------------------------------------------------
@pytest.mark.parametrize("variant,threads,prefetch", [(1, 0, 0), (2, 0, 2), (2, 0, 4), (2, 0, 8), (2, 128, 4), (2, 64, 8),
                                                      (2, 32, 2), (3, 0, 2), (3, 0, 4), (3, 0, 8), (4, 0, 0)])
@pytest.mark.parametrize("bf16", [False, True])
def test_dense_variants(P, variant, threads, prefetch, bf16):
    # d = 480: 120 fp32 / 60 bf16 16-byte chunks: ragged against 32-lane and 128-thread tiles
    wl = wi.config2(k=5, d=480, m=96, base_steps=333)
    if bf16:
        wl.X = wl.X.to(torch.bfloat16)
    assert_parity(P, wl, {"dense_variant": variant, "threads": threads, "prefetch": prefetch})


@pytest.mark.parametrize("loss", [HINGE, LOGISTIC, SQUARED])
@pytest.mark.parametrize("sched", [0, 1])
@pytest.mark.parametrize("variant", [1, 2, 3, 4, 5])
def test_losses_and_schedules(P, loss, sched, variant):
    wl = wi.config1(k=3, d=64, m=128, n_steps=(300, 150, 40))
    wl.loss, wl.sched = loss, sched
    wl.eta0 = 0.05 if sched else 0.01
    if loss == SQUARED:
        wl.y = (wl.y * 0.5 + 0.1).contiguous()
    assert_parity(P, wl, {"dense_variant": variant})


def test_generic_kernel_handles_unaligned_shapes(P):
    # d = 67 (not a multiple of 4), row stride 71: only the generic kernel applies, and auto must pick it
    g = torch.Generator().manual_seed(3)
    k, d, ld, m = 3, 67, 71, 50
    Xp = torch.randn(k * m, ld, generator=g) / 8
    y = torch.sign(torch.randn(k * m, generator=g))
    off = np.arange(k + 1, dtype=np.int64) * m
    n = np.array([200, 77, 0], dtype=np.int64)
    oW = oracle.run_dense(Xp, y, off, n, d, 0.05, 0, 1e-2, LOGISTIC, 11)
    Xd = Xp.cuda()
    with P.Context(k, d) as ctx:
        ctx.run(Xd[:, :d], y.cuda(), off, n, 0.05, 0, 1e-2, LOGISTIC, 11)
        W = ctx.get_models().cpu().numpy()
        ctx.check()
        with pytest.raises(P.WpsgdError) as e:
            ctx.set_option("dense_variant", 2)
            ctx.run(Xd[:, :d], y.cuda(), off, n, 0.05, 0, 1e-2, LOGISTIC, 11)
        assert e.value.status_name == "UNSUPPORTED"
    for j in range(2):
        assert rel_l2(W[j], oW[j]) <= 1e-4
    assert np.all(W[2] == 0)


def test_large_d_falls_back_and_matches(P):
    wl = wi.config2(k=2, d=8200, m=16, base_steps=40)  # beyond the register kernels' reach
    assert_parity(P, wl)


# ---- blocked kernels with the decaying step size eta0 / sqrt(n): per-block tables instead of powers of one factor -------
@pytest.mark.parametrize("loss", [HINGE, LOGISTIC, SQUARED])
@pytest.mark.parametrize("kind", ["block_fp32", "block_bf16", "warp", "mma8", "mma16", "f32x16"])
def test_blocked_kernels_decaying_step_size(P, kind, loss):
    d = {"block_fp32": 1024, "block_bf16": 1000, "warp": 256, "mma8": 2048, "mma16": 2048, "f32x16": 1024}[kind]
    wl = wi.config2(k=4, d=d, m=96, base_steps=333)
    wl.n_steps[3] = 0
    wl.loss, wl.sched, wl.eta0, wl.lam = loss, 1, 0.3, 0.05  # eta_n lambda from 1.5e-2 down: the factors differ step by step
    if loss == SQUARED:
        wl.y = (wl.y * 0.3).contiguous()
    wl.w0 = torch.full((d,), 0.05)
    if kind not in ("block_fp32", "warp", "f32x16"):
        wl.X = wl.X.to(torch.bfloat16)
    opts = {"block_fp32": {"dense_variant": 4}, "block_bf16": {"dense_variant": 4}, "warp": {"dense_variant": 5},
            "mma8": {"dense_variant": 8, "block_samples": 8, "cluster": 2},
            "mma16": {"dense_variant": 8, "block_samples": 16, "cluster": 2},
            "f32x16": {"dense_variant": 9, "cluster": 4}}[kind]
    assert_parity(P, wl, opts)


def test_decaying_step_size_continue_keeps_the_step_numbers(P):
    # a continued chain must take eta of its own step numbers (first + n), also inside the per-block tables
    wl_cpu = wi.config2(k=3, d=1024, m=64, base_steps=8)
    wl_cpu.n_steps = np.array([203, 101, 50], dtype=np.int64)
    wl_cpu.sched, wl_cpu.eta0, wl_cpu.lam = 1, 0.3, 0.05
    wl = wl_cpu.to("cuda")
    with P.Context(wl.k, wl.d) as ctx:
        ctx.run(wl.X, wl.y, wl.shard_off, np.array([50, 50, 50]), wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
        ctx.continue_(wl.X, wl.y, wl.shard_off, np.array([153, 51, 0]))
        seg = ctx.get_models().cpu().numpy()
        ctx.check()
    oW = oracle.run_dense(wl_cpu.X, wl_cpu.y, wl.shard_off, wl_cpu.n_steps, wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
    for j in range(wl.k):
        assert rel_l2(seg[j], oW[j]) <= 1e-4


# ---- blocked kernel: block boundaries, ring depths, column tilings ----------------------------------------
@pytest.mark.parametrize("n_steps", [(1, 7, 8), (9, 15, 16), (17, 0, 64), (333, 250, 3)])
@pytest.mark.parametrize("stages", [2, 3, 4])
def test_blocked_kernel_block_boundaries_and_ring_depths(P, n_steps, stages):
    wl = wi.config2(k=3, d=1024, m=64, base_steps=8)
    wl.n_steps = np.array(n_steps, dtype=np.int64)
    wl.w0 = torch.full((1024,), 0.1)
    assert_parity(P, wl, {"dense_variant": 4, "stages": stages})


@pytest.mark.parametrize("d,bf16", [(64, False), (480, False), (1024, False), (2048, False), (1536, False), (64, True),
                                     (1000, True), (4096, True), (3008, True)])
@pytest.mark.parametrize("loss", [HINGE, LOGISTIC, SQUARED])
def test_blocked_kernel_column_tilings(P, d, bf16, loss):
    wl = wi.config2(k=3, d=d, m=48, base_steps=210)
    wl.loss = loss
    if loss == SQUARED:
        wl.y = (wl.y * 0.3).contiguous()
    if bf16:
        wl.X = wl.X.to(torch.bfloat16)
    assert_parity(P, wl, {"dense_variant": 4})


@pytest.mark.parametrize("d,bf16", [(64, False), (200, False), (256, False), (8, False), (72, True), (512, True)])
@pytest.mark.parametrize("loss", [HINGE, LOGISTIC, SQUARED])
@pytest.mark.parametrize("stages", [2, 3])
def test_blocked_warp_kernel(P, d, bf16, loss, stages):
    # k = 11: three CTAs of four warps, the last one with an idle warp; step counts with ragged last blocks
    wl = wi.config5(k=11, d=d, m=40, total_steps=11 * 131, rho=6.0)
    wl.n_steps[3] = 0
    wl.n_steps[7] = 5
    wl.loss = loss
    if loss == SQUARED:
        wl.y = (wl.y * 0.3).contiguous()
    if bf16:
        wl.X = wl.X.to(torch.bfloat16)
    wl.w0 = torch.full((d,), 0.05)
    assert_parity(P, wl, {"dense_variant": 5, "stages": stages})


def test_blocked_warp_kernel_limits(P):
    wl = wi.config2(k=2, d=480, m=16, base_steps=20)  # 120 chunks: too wide for a warp
    with pytest.raises(P.WpsgdError) as e:
        gpu_solve(P, wl, {"dense_variant": 5})
    assert e.value.status_name == "UNSUPPORTED"


@pytest.mark.parametrize("d,bf16", [(1024, False), (2048, False), (4096, True)])
def test_bounded_wait_for_rows_reports_timeout_and_context_survives(P, d, bf16):
    # Failure detection without a fault: the rows of block 3 are never requested (test hook), so the bounded
    # wait for them runs out; the kernel flags it, leaves in step and returns, and the next run is clean.
    wl_cpu = wi.config2(k=3, d=d, m=32, base_steps=120)
    if bf16:
        wl_cpu.X = wl_cpu.X.to(torch.bfloat16)
    wl = wl_cpu.to("cuda")
    with P.Context(wl.k, wl.d) as ctx:
        ctx.set_option("dense_variant", 4)
        ctx.set_option("spin_limit", 2000)
        ctx.set_option("test_drop_block", 3)
        ctx.run_workload(wl)
        with pytest.raises(P.WpsgdError) as e:
            ctx.check()
        assert e.value.status_name == "TIMEOUT"
        ctx.set_option("test_drop_block", -1)
        ctx.set_option("spin_limit", 1 << 20)
        ctx.run_workload(wl)
        v = ctx.combine().cpu().numpy()
        ctx.check()
    ov, _, _ = oracle.solve(wl_cpu)
    assert rel_l2(v, ov) <= 1e-4


# ---- tensor-core cluster kernel (bf16 rows): Gram block and margins from mma, model split into three bf16 rows; blocks
# of 8 samples (every loss) or 16 samples (squared and hinge) -----------------------------------------------------------
MMA_BLOCKS = [8, 16]


def _mma(block, wl, **more):
    """Options that select the tensor-core kernel with the given block size."""
    return dict({"dense_variant": 8, "block_samples": block}, **more)


@pytest.mark.parametrize("cluster", [1, 2, 4])
@pytest.mark.parametrize("d", [480, 488, 8, 264])
@pytest.mark.parametrize("block", MMA_BLOCKS)
def test_mma_kernel_ragged_shapes(P, cluster, d, block):
    # 60 / 61 / 1 / 33 chunks of 8 columns: odd chunk counts leave half a 16-column tile empty, the last CTA of a
    # cluster owns a ragged slice, and with d = 8 only one CTA can exist
    if d == 8 and cluster > 1:
        pytest.skip("fewer chunks than CTAs")
    wl = wi.config2(k=5, d=d, m=96, base_steps=333)
    wl.n_steps[2] = 0
    wl.w0 = torch.full((d,), 0.05)
    wl.X = wl.X.to(torch.bfloat16)
    assert_parity(P, wl, _mma(block, wl, cluster=cluster))


@pytest.mark.parametrize("d,cluster", [(4096, 2), (4096, 4), (2048, 1), (4096, 8), (3008, 2), (1024, 8)])
@pytest.mark.parametrize("loss", [HINGE, LOGISTIC, SQUARED])
@pytest.mark.parametrize("block", MMA_BLOCKS)
def test_mma_kernel_losses_and_widths(P, d, cluster, loss, block):
    wl = wi.config2(k=3, d=d, m=48, base_steps=210)
    wl.loss = loss
    if loss == SQUARED:
        wl.y = (wl.y * 0.3).contiguous()
    wl.X = wl.X.to(torch.bfloat16)
    assert_parity(P, wl, _mma(block, wl, cluster=cluster))


@pytest.mark.parametrize("n_steps", [(1, 7, 8), (9, 15, 16), (17, 0, 64), (333, 250, 3), (31, 32, 33)])
@pytest.mark.parametrize("stages", [2, 3, 4])
@pytest.mark.parametrize("block", MMA_BLOCKS)
def test_mma_kernel_block_boundaries_and_ring_depths(P, n_steps, stages, block):
    wl = wi.config2(k=3, d=1024, m=64, base_steps=8)
    wl.n_steps = np.array(n_steps, dtype=np.int64)
    wl.w0 = torch.full((1024,), 0.1)
    wl.X = wl.X.to(torch.bfloat16)
    assert_parity(P, wl, _mma(block, wl, cluster=2, stages=stages))


@pytest.mark.parametrize("block", MMA_BLOCKS)
def test_mma_kernel_model_split_keeps_fp32_accuracy(P, block):
    # a model with a wide spread of magnitudes (w0 from 1e-6 to 1e3): the three bf16 rows must carry all 24 bits of
    # every entry, or the margins of the first steps are off by far more than the tolerance
    wl = wi.config3(k=4, d=2048, m=64, n_lo=40, n_hi=90)
    g = torch.Generator().manual_seed(11)
    wl.w0 = (torch.randn(2048, generator=g) * torch.logspace(-6, 3, 2048)).contiguous()
    assert_parity(P, wl, _mma(block, wl, cluster=2))


@pytest.mark.parametrize("block", MMA_BLOCKS)
def test_mma_kernel_default_shape_and_continue(P, block):
    wl_cpu = wi.small(3)
    wl = wl_cpu.to("cuda")
    with P.Context(wl.k, wl.d) as ctx:
        ctx.set_option("dense_variant", 8)
        ctx.set_option("block_samples", block)
        first = np.minimum(wl.n_steps, 301)
        ctx.run(wl.X, wl.y, wl.shard_off, first, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
        ctx.continue_(wl.X, wl.y, wl.shard_off, wl.n_steps - first)
        seg = ctx.get_models().cpu().numpy()
        ctx.check()
    oW = oracle.run_dense(wl_cpu.X, wl_cpu.y, wl.shard_off, wl.n_steps, wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
    for j in range(wl.k):
        assert rel_l2(seg[j], oW[j]) <= 1e-4


@pytest.mark.parametrize("block", MMA_BLOCKS)
def test_mma_kernel_limits(P, block):
    wl = wi.config2(k=2, d=64, m=16, base_steps=20)  # fp32 rows
    with pytest.raises(P.WpsgdError) as e:
        gpu_solve(P, wl, {"dense_variant": 8, "block_samples": block})
    assert e.value.status_name == "UNSUPPORTED"
    wl.X = wl.X.to(torch.bfloat16)  # 8 chunks: a cluster of 8 needs 8 non-empty slices; 16 CTAs cannot exist
    with pytest.raises(P.WpsgdError) as e:
        gpu_solve(P, wl, {"dense_variant": 8, "block_samples": block, "cluster": 16})
    assert e.value.status_name == "INVALID_ARG"


@pytest.mark.parametrize("d,cluster", [(1024, 1), (4096, 2), (4096, 4)])
@pytest.mark.parametrize("block", MMA_BLOCKS)
def test_mma_kernel_bounded_waits_report_timeout_and_context_survives(P, d, cluster, block):
    # Failure detection without a fault: the rows of block 3 are never requested (test hook), so the bounded wait
    # for them runs out; every CTA of the cluster is told, all leave in step, and the next run is clean.
    wl_cpu = wi.config2(k=3, d=d, m=32, base_steps=120)
    wl_cpu.X = wl_cpu.X.to(torch.bfloat16)
    opts = _mma(block, wl_cpu, cluster=cluster)
    wl = wl_cpu.to("cuda")
    with P.Context(wl.k, wl.d) as ctx:
        for k_, v_ in opts.items():
            ctx.set_option(k_, v_)
        ctx.set_option("spin_limit", 2000)
        ctx.set_option("test_drop_block", 3)
        ctx.run_workload(wl)
        with pytest.raises(P.WpsgdError) as e:
            ctx.check()
        assert e.value.status_name == "TIMEOUT"
        ctx.set_option("test_drop_block", -1)
        ctx.set_option("spin_limit", 1 << 20)
        ctx.run_workload(wl)
        v = ctx.combine().cpu().numpy()
        ctx.check()
    ov, _, _ = oracle.solve(wl_cpu)
    assert rel_l2(v, ov) <= 1e-4


# ---- fp32 rows, 16 samples per block, a chain spread over a cluster (Gram block on the fp32 pipes) ----------------------
@pytest.mark.parametrize("d,cluster", [(1024, 8), (1024, 4), (512, 2), (256, 1), (1000, 8), (36, 1), (2048, 8)])
@pytest.mark.parametrize("loss", [HINGE, LOGISTIC, SQUARED])
def test_f32_cluster_kernel_losses_and_widths(P, d, cluster, loss):
    wl = wi.config2(k=3, d=d, m=48, base_steps=210)
    wl.loss = loss
    if loss == SQUARED:
        wl.y = (wl.y * 0.3).contiguous()
    assert_parity(P, wl, {"dense_variant": 9, "cluster": cluster})


@pytest.mark.parametrize("n_steps", [(1, 7, 8), (9, 15, 16), (17, 0, 64), (333, 250, 3), (31, 32, 33)])
@pytest.mark.parametrize("cluster", [1, 4])
def test_f32_cluster_kernel_block_boundaries_and_empty_chains(P, n_steps, cluster):
    wl = wi.config2(k=3, d=256, m=64, base_steps=8)
    wl.n_steps = np.array(n_steps, dtype=np.int64)
    wl.w0 = torch.full((256,), 0.1)
    assert_parity(P, wl, {"dense_variant": 9, "cluster": cluster})


def test_f32_cluster_kernel_default_shape_and_continue(P):
    wl_cpu = wi.config2(k=5, d=1024, m=96, base_steps=700)
    wl = wl_cpu.to("cuda")
    with P.Context(wl.k, wl.d) as ctx:
        ctx.set_option("dense_variant", 9)
        first = np.minimum(wl.n_steps, 301)
        ctx.run(wl.X, wl.y, wl.shard_off, first, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
        ctx.continue_(wl.X, wl.y, wl.shard_off, wl.n_steps - first)
        seg = ctx.get_models().cpu().numpy()
        ctx.check()
    oW = oracle.run_dense(wl_cpu.X, wl_cpu.y, wl.shard_off, wl.n_steps, wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
    for j in range(wl.k):
        assert rel_l2(seg[j], oW[j]) <= 1e-4


def test_f32_cluster_kernel_limits(P):
    wl = wi.config2(k=2, d=2048, m=16, base_steps=20)  # 512 chunks: one CTA would hold more than 64
    with pytest.raises(P.WpsgdError) as e:
        gpu_solve(P, wl, {"dense_variant": 9, "cluster": 4})
    assert e.value.status_name == "UNSUPPORTED"
    wl.X = wl.X.to(torch.bfloat16)
    with pytest.raises(P.WpsgdError) as e:
        gpu_solve(P, wl, {"dense_variant": 9})
    assert e.value.status_name == "UNSUPPORTED"


@pytest.mark.parametrize("d,cluster", [(256, 1), (1024, 4), (1024, 8)])
def test_f32_cluster_kernel_bounded_waits_report_timeout_and_context_survives(P, d, cluster):
    # the rows of block 3 are never requested (test hook): the bounded wait for them runs out, every CTA of the
    # cluster is told, all leave in step, and the next run is clean
    wl_cpu = wi.config2(k=3, d=d, m=32, base_steps=120)
    wl = wl_cpu.to("cuda")
    with P.Context(wl.k, wl.d) as ctx:
        ctx.set_option("dense_variant", 9)
        ctx.set_option("cluster", cluster)
        ctx.set_option("spin_limit", 2000)
        ctx.set_option("test_drop_block", 3)
        ctx.run_workload(wl)
        with pytest.raises(P.WpsgdError) as e:
            ctx.check()
        assert e.value.status_name == "TIMEOUT"
        ctx.set_option("test_drop_block", -1)
        ctx.set_option("spin_limit", 1 << 20)
        ctx.run_workload(wl)
        v = ctx.combine().cpu().numpy()
        ctx.check()
    ov, _, _ = oracle.solve(wl_cpu)
    assert rel_l2(v, ov) <= 1e-4


# ---- logistic loss: blocks whose steps move the margins far take the direct evaluation ---------------------------------
@pytest.mark.parametrize("variant,d", [(4, 1024), (5, 128), (8, 1024), (9, 1024)])
def test_logistic_large_steps_between_correlated_rows(P, variant, d):
    # rows that are nearly parallel (large Gram entries) and a large step size: inside a block of 8 samples the
    # margins move by much more than the range of the cubic expansion of the logistic factor
    wl = wi.config2(k=3, d=d, m=64, base_steps=160)
    g = torch.Generator().manual_seed(5)
    base = torch.randn(d, generator=g) / np.sqrt(d)
    wl.X = (2.0 * base[None, :] + 0.3 * wl.X).contiguous()
    wl.eta0 = 0.4
    if variant == 8:
        wl.X = wl.X.to(torch.bfloat16)
    assert_parity(P, wl, {"dense_variant": variant})


@pytest.mark.parametrize("k,variant", [(4, 9), (40, 4)])
def test_default_kernels_for_large_aligned_fp32_rows(P, k, variant):
    # few chains: each spread over a cluster of idle SMs (16 samples per block); many chains: one CTA each (8 per block)
    wl = wi.config2(k=k, d=1024, m=64, base_steps=100).to("cuda")
    with P.Context(wl.k, wl.d) as a, P.Context(wl.k, wl.d) as b:
        a.run_workload(wl)
        b.set_option("dense_variant", variant)
        b.run_workload(wl)
        np.testing.assert_array_equal(a.get_models().cpu().numpy(), b.get_models().cpu().numpy())
        a.check()
        b.check()


def test_tensor_core_cluster_kernel_is_the_default_for_wide_bf16_rows(P):
    wl = wi.config3(k=4, d=2048, m=64, n_lo=60, n_hi=120).to("cuda")
    with P.Context(wl.k, wl.d) as a, P.Context(wl.k, wl.d) as b:
        a.run_workload(wl)
        b.set_option("dense_variant", 8)
        b.run_workload(wl)
        np.testing.assert_array_equal(a.get_models().cpu().numpy(), b.get_models().cpu().numpy())
        a.check()
        b.check()


# ---- degenerate cases -----------------------------------------------------------------------------------
def test_nodes_without_work_keep_w0(P):
    wl = wi.config1(k=4, d=64, m=64, n_steps=(120, 0, 30, 0))
    wl.w0 = torch.full((64,), 4.0)  # the paper's experiments start from the constant vector 4
    v, W, wts, _ = gpu_solve(P, wl)
    assert np.all(W[1] == 4.0) and np.all(W[3] == 4.0)
    assert_parity(P, wl)


def test_no_work_at_all_returns_w0(P):
    wl = wi.config1(k=3, d=64, m=8, n_steps=(0, 0, 0))
    wl.w0 = torch.arange(64, dtype=torch.float32)
    v, W, wts, _ = gpu_solve(P, wl)
    np.testing.assert_array_equal(wts, np.full(3, 1 / 3))
    np.testing.assert_allclose(v, np.arange(64), rtol=1e-6)
    wl.w0 = None
    v, W, _, _ = gpu_solve(P, wl)
    assert np.all(v == 0) and np.all(W == 0)


def test_single_node_is_sequential_sgd(P):
    wl = wi.config1(k=1, d=64, m=256, n_steps=(500,))
    v, W, wts, flag = gpu_solve(P, wl)
    assert wts[0] == 1.0 and flag is False  # Eq. 7 with k = 1: 2 > 2 is false
    np.testing.assert_array_equal(v, W[0])
    assert_parity(P, wl)


def test_single_row_shards_and_unequal_shards(P):
    g = torch.Generator().manual_seed(5)
    d = 32
    off = np.array([0, 1, 4, 4, 40], dtype=np.int64)  # shard sizes 1, 3, 0, 36
    X = torch.randn(40, d, generator=g) / 4
    y = torch.sign(torch.randn(40, generator=g))
    n = np.array([25, 60, 0, 100], dtype=np.int64)
    wl = wi.Workload("ragged", 4, d, off, n, 0.05, 0, 0.01, LOGISTIC, 9, y, X=X)
    assert_parity(P, wl)
    for variant in (1, 2, 3):
        assert_parity(P, wl, {"dense_variant": variant})


def test_equal_work_reduces_to_plain_average(P):
    wl = wi.config2(k=6, d=128, m=64, base_steps=90)
    wl.n_steps[:] = 90
    v, W, wts, _ = gpu_solve(P, wl)
    np.testing.assert_array_equal(wts, np.full(6, 1 / 6))
    np.testing.assert_allclose(v, W.astype(np.float64).mean(0), rtol=1e-6, atol=1e-9)


def test_relabelling_a_node_changes_only_its_stream(P):
    # the same shard at node position j must see the oracle's stream for node j
    wl = wi.config1(k=3, d=64, m=64, n_steps=(50, 50, 50))
    _, W, _, _ = gpu_solve(P, wl)
    assert not np.array_equal(W[0], W[1])
    assert_parity(P, wl)


# ---- combination --------------------------------------------------------------------------------------
@pytest.mark.parametrize("r", [0.0, 1.0, 0.99999, 0.9])
def test_combine_rates(P, r):
    wl = wi.config1(k=4, d=64, m=64, n_steps=(400, 300, 100, 7))
    v, W, wts, flag = gpu_solve(P, wl, r=r)
    owts, oflag, _ = oracle.weights(wl.n_steps, wl.eta0, wl.sched, wl.lam, r)
    np.testing.assert_allclose(wts, owts, rtol=1e-12)
    assert flag == oflag
    want = oracle.combine(W.astype(np.float64), owts)  # the GPU's own models, so this isolates the reduction
    np.testing.assert_allclose(v, want, rtol=2e-7, atol=1e-12)


def test_combine_many_nodes_ragged_d(P):
    k, d = 37, 1001
    g = torch.Generator().manual_seed(1)
    X = torch.randn(k * 4, d, generator=g)
    y = torch.sign(torch.randn(k * 4, generator=g))
    n = (np.arange(k) % 5).astype(np.int64)
    wl = wi.Workload("wide", k, d, np.arange(k + 1, dtype=np.int64) * 4, n, 0.01, 0, 0.1, HINGE, 2, y, X=X)
    assert_parity(P, wl)


# ---- segmented runs and periodic averaging ----------------------------------------------------------------
def test_continue_blocked_kernel(P):
    # the blocked kernel groups samples by eight from wherever a segment starts, so a cut run agrees with the
    # uncut one up to rounding order (not bit for bit)
    wl_cpu = wi.config2(k=3, d=256, m=128, base_steps=203)
    wl = wl_cpu.to("cuda")
    with P.Context(wl.k, wl.d) as ctx:
        ctx.set_option("dense_variant", 4)
        first = np.minimum(wl.n_steps, 37)
        ctx.run(wl.X, wl.y, wl.shard_off, first, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
        ctx.continue_(wl.X, wl.y, wl.shard_off, wl.n_steps - first)
        seg = ctx.get_models().cpu().numpy()
        ctx.check()
    oW = oracle.run_dense(wl_cpu.X, wl_cpu.y, wl.shard_off, wl.n_steps, wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
    for j in range(wl.k):
        assert rel_l2(seg[j], oW[j]) <= 1e-4


@pytest.mark.parametrize("variant", [1, 2, 3])
def test_continue_equals_one_run(P, variant):
    wl = wi.config1(k=3, d=64, m=128, n_steps=(203, 101, 50)).to("cuda")
    wl.sched = 1  # the step number matters for eta_n, so a wrong restart shows
    with P.Context(wl.k, wl.d) as ctx:
        ctx.set_option("dense_variant", variant)
        ctx.run_workload(wl)
        full = ctx.get_models().cpu().numpy()
        cuts = [np.array([50, 50, 50]), np.array([1, 1, 0]), np.array([152, 50, 0])]
        ctx.run(wl.X, wl.y, wl.shard_off, cuts[0], wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
        for c in cuts[1:]:
            ctx.continue_(wl.X, wl.y, wl.shard_off, c)
        seg = ctx.get_models().cpu().numpy()
        wts, _ = ctx.get_weights()
        ctx.check()
    np.testing.assert_array_equal(seg, full)  # same arithmetic in the same order
    owts, _, _ = oracle.weights(wl.n_steps, wl.eta0, wl.sched, wl.lam)
    np.testing.assert_allclose(wts, owts, rtol=1e-12)


def test_periodic_weighted_averaging(P):
    # average every `span` fastest-node steps, then continue from the average on every node
    wl = wi.config2(k=4, d=128, m=64, base_steps=120)
    span_steps = [np.array([40, 20, 10, 40]), np.array([40, 20, 10, 40]), np.array([40, 20, 10, 40])]
    dev = wl.to("cuda")
    with P.Context(wl.k, wl.d) as ctx:
        ctx.run(dev.X, dev.y, wl.shard_off, span_steps[0], wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
        for seg in span_steps[1:]:
            ctx.set_models(ctx.combine())
            ctx.continue_(dev.X, dev.y, wl.shard_off, seg)
        v = ctx.combine().cpu().numpy()
        ctx.check()
    # oracle: same schedule; weights of each round come from that round's step counts
    W = oracle.run_dense(wl.X, wl.y, wl.shard_off, span_steps[0], wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
    done = span_steps[0].copy()
    for seg in span_steps[1:]:
        wts, _, _ = oracle.weights(done, wl.eta0, wl.sched, wl.lam)
        vv = oracle.combine(W, wts)
        # steps continue from each node's own count: run node by node with its own step_begin
        Wn = np.zeros_like(W)
        for j in range(wl.k):
            only = np.zeros(wl.k, dtype=np.int64)
            only[j] = seg[j]
            Wn[j] = oracle.run_dense(wl.X, wl.y, wl.shard_off, only, wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed,
                                     step_begin=int(done[j]), W_resume=np.tile(vv.astype(np.float32).astype(np.float64), (wl.k, 1)))[j]
        W = Wn
        done = done + seg
    wts, _, _ = oracle.weights(done, wl.eta0, wl.sched, wl.lam)
    assert rel_l2(v, oracle.combine(W, wts)) <= 1e-4


# ---- evaluation measures ---------------------------------------------------------------------------------
@pytest.mark.parametrize("loss", [HINGE, LOGISTIC, SQUARED])
@pytest.mark.parametrize("bf16", [False, True])
def test_objective_and_error_rate(P, loss, bf16):
    wl = wi.config1(k=2, d=64, m=333, n_steps=(10, 10))
    X = wl.X.to(torch.bfloat16) if bf16 else wl.X
    w = (torch.randn(64, generator=torch.Generator().manual_seed(4)) / 8)
    with P.Context(2, 64) as ctx:
        out = ctx.objective(X.cuda(), wl.y.cuda(), w.cuda(), 0.01, loss).cpu().numpy()
        ctx.check()
    obj, err = oracle.objective_dense(X, wl.y, w.numpy().astype(np.float64), 0.01, loss)
    assert out[0] == pytest.approx(obj, rel=1e-5)
    assert abs(out[1] - err) <= 2.0 / 666  # a margin within fp32 rounding of 0 may flip


# ---- host-buffer entry point --------------------------------------------------------------------------------
def test_solve_host_equals_device_path(P):
    wl = wi.config2(k=5, d=256, m=128, base_steps=200)
    wl.w0 = torch.full((256,), 0.5)
    v_dev, _, _, _ = gpu_solve(P, wl)
    with P.Context(wl.k, wl.d) as ctx:
        out = ctx.solve_host(wl.X.pin_memory(), wl.y.pin_memory(), wl.shard_off, wl.n_steps, wl.eta0, wl.sched, wl.lam,
                             wl.loss, wl.seed, w0=wl.w0)
        again = ctx.solve_host(wl.X, wl.y, wl.shard_off, wl.n_steps, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed,
                               w0=wl.w0)  # pageable source, buffers reused
        ctx.check()
    np.testing.assert_array_equal(out.numpy(), v_dev)
    np.testing.assert_array_equal(again.numpy(), v_dev)


@pytest.mark.parametrize("d,bf16,k", [(1024, False, 5), (1024, False, 2), (2048, True, 7), (480, False, 3)])
@pytest.mark.parametrize("pipeline", [0, 1])
def test_solve_host_pipelined_equals_device_path(P, d, bf16, k, pipeline):
    # rows wide enough for the pipelined form: shards copied in groups (longest chains first), chains of a group
    # launched when its rows have arrived; the per-node arithmetic is the same, so the result is bit for bit that of
    # the device path
    wl = wi.config2(k=k, d=d, m=96, base_steps=230)
    wl.n_steps[k - 1] = 0
    if bf16:
        wl.X = wl.X.to(torch.bfloat16)
    wl.w0 = torch.full((d,), 0.25)
    v_dev, _, _, _ = gpu_solve(P, wl)
    with P.Context(wl.k, wl.d) as ctx:
        ctx.set_option("host_pipeline", pipeline)
        for _ in range(2):
            out = ctx.solve_host(wl.X.pin_memory(), wl.y.pin_memory(), wl.shard_off, wl.n_steps, wl.eta0, wl.sched, wl.lam,
                                 wl.loss, wl.seed, w0=wl.w0)
            np.testing.assert_array_equal(out.numpy(), v_dev)
        ctx.check()


def test_solve_host_csr_equals_device_path(P):
    wl = wi.config4(k=5, d=4096, m=200, base_steps=500, mean_nnz=25.0)
    wl.w0 = torch.full((4096,), 0.02)
    v_dev, _, _, _ = gpu_solve(P, wl)
    with P.Context(wl.k, wl.d) as ctx:
        for _ in range(2):
            out = ctx.solve_host_csr(wl.row_ptr.pin_memory(), wl.col_idx.pin_memory(), wl.val.pin_memory(), wl.y.pin_memory(),
                                     wl.shard_off, wl.n_steps, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed, w0=wl.w0)
            np.testing.assert_array_equal(out.numpy(), v_dev)
        ctx.check()
    ov, _, _ = oracle.solve(wl)
    assert rel_l2(out.numpy(), ov) <= TOL[wl.loss]


# ---- sparse path --------------------------------------------------------------------------------------------
# sparse_variant 1: one step per round trip to the model in global memory; 2 (the default): blocks of steps run in a
# shared-memory cache of the model entries they touch
@pytest.mark.parametrize("loss", [HINGE, LOGISTIC, SQUARED])
@pytest.mark.parametrize("variant,prefetch", [(1, 2), (1, 4), (1, 8), (2, 0)])
def test_csr_losses_and_kernels(P, loss, variant, prefetch):
    wl = wi.config4(k=5, d=4096, m=300, base_steps=700, mean_nnz=30.0)
    wl.loss = loss
    if loss == SQUARED:
        wl.eta0 = 0.05
    wl.w0 = torch.full((4096,), 0.01)
    assert_parity(P, wl, {"sparse_variant": variant, "prefetch": prefetch})


@pytest.mark.parametrize("variant", [1, 2])
def test_csr_long_rows_and_strong_regulariser(P, variant):
    # rows with up to 128 nonzeros (beyond the 64 kept in registers); eta*lambda large enough that the
    # scale factor is folded back into the model several times
    wl = wi.config4(k=3, d=512, m=64, base_steps=400, mean_nnz=90.0, max_nnz=128)
    wl.sched, wl.eta0, wl.lam = 0, 0.5, 0.5  # (1 - 0.25)^400 ~ 1e-50
    wl.w0 = torch.full((512,), 1.0)
    assert_parity(P, wl, {"sparse_variant": variant})


@pytest.mark.parametrize("n_steps", [(1, 63, 64), (65, 127, 128), (129, 0, 200), (333, 250, 3)])
@pytest.mark.parametrize("mean_nnz", [8.0, 100.0])
def test_csr_block_kernel_block_boundaries(P, n_steps, mean_nnz):
    # short rows: a block ends after 64 steps; long rows: it ends when its 4096 table entries are used up
    wl = wi.config4(k=3, d=2048, m=96, base_steps=10, mean_nnz=mean_nnz, max_nnz=128)
    wl.n_steps = np.array(n_steps, dtype=np.int64)
    wl.w0 = torch.full((2048,), 0.02)
    assert_parity(P, wl, {"sparse_variant": 2})


def _rows_with_given_lengths(lengths, d, seed):
    """Hand-built CSR rows of the given lengths: distinct sorted random columns, values 1/sqrt(nnz), labels +-1."""
    g = torch.Generator().manual_seed(seed)
    cols, vals = [], []
    for n in lengths:
        c, _ = torch.sort(torch.randperm(d, generator=g)[:n])
        cols.append(c.to(torch.int32))
        vals.append(torch.full((n,), 1.0 / np.sqrt(max(n, 1))))
    rp = torch.zeros(len(lengths) + 1, dtype=torch.int64)
    rp[1:] = torch.cumsum(torch.tensor(lengths), 0)
    y = torch.where(torch.rand(len(lengths), generator=g) < 0.5, 1.0, -1.0)
    return rp, torch.cat(cols), torch.cat(vals), y


@pytest.mark.parametrize("loss", [HINGE, SQUARED])
def test_csr_rows_longer_than_the_block_tables(P, loss):
    # rows of 5000 and 6000 nonzeros do not fit the 4096 table entries of a block: such a step is run on global
    # memory, between ordinary blocks of short rows
    d = 8192
    lengths = [5000, 12, 30, 6000, 7, 4096, 4097, 64, 1, 0, 33, 65]
    rp, ci, va, y = _rows_with_given_lengths(lengths, d, 11)
    wl = wi.Workload("long", 2, d, np.array([0, 6, 12]), np.array([150, 90]), 0.2, 1, 0.01, loss, 5, y, row_ptr=rp,
                     col_idx=ci, val=va, w0=torch.full((d,), 0.01))
    assert_parity(P, wl, {"sparse_variant": 2})


@pytest.mark.parametrize("variant", [1, 2])
def test_continue_csr_equals_one_run(P, variant):
    wl_cpu = wi.config4(k=3, d=4096, m=128, base_steps=10, mean_nnz=30.0)
    wl_cpu.n_steps = np.array([203, 101, 50], dtype=np.int64)
    wl_cpu.lam = 0.01
    wl = wl_cpu.to("cuda")
    with P.Context(wl.k, wl.d) as ctx:
        ctx.set_option("sparse_variant", variant)
        ctx.run_workload(wl)
        full = ctx.get_models().cpu().numpy()
        cuts = [np.array([50, 50, 50]), np.array([1, 1, 0]), np.array([152, 50, 0])]
        ctx.run_csr(wl.row_ptr, wl.col_idx, wl.val, wl.y, wl.shard_off, cuts[0], wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
        for c in cuts[1:]:
            ctx.continue_csr(wl.row_ptr, wl.col_idx, wl.val, wl.y, wl.shard_off, c)
        seg = ctx.get_models().cpu().numpy()
        wts, _ = ctx.get_weights()
        ctx.check()
    if variant == 1:
        np.testing.assert_array_equal(seg, full)  # same arithmetic in the same order
    else:
        # the fp64 scale is a product over the steps of a block, so cutting the chain changes its last bits only
        for j in range(wl.k):
            assert rel_l2(seg[j], full[j]) <= 1e-6
    owts, _, _ = oracle.weights(wl_cpu.n_steps, wl_cpu.eta0, wl_cpu.sched, wl_cpu.lam)
    np.testing.assert_allclose(wts, owts, rtol=1e-12)
    oW = oracle.run_csr(wl_cpu.row_ptr, wl_cpu.col_idx, wl_cpu.val, wl_cpu.y, wl_cpu.shard_off, wl_cpu.n_steps, wl_cpu.d,
                        wl_cpu.eta0, wl_cpu.sched, wl_cpu.lam, wl_cpu.loss, wl_cpu.seed)
    for j in range(wl.k):
        assert rel_l2(seg[j], oW[j]) <= TOL[wl_cpu.loss]


def test_periodic_weighted_averaging_on_csr_rows(P):
    # average every span of fastest-node steps, broadcast, continue: the paper's bucket-style WP-SGD on sparse rows.
    # The checker runs the same schedule on the densified rows (its dense loop can start from a given model and step).
    wl = wi.config4(k=4, d=256, m=64, base_steps=10, mean_nnz=12.0, max_nnz=32)
    wl.loss, wl.sched, wl.eta0, wl.lam = LOGISTIC, 0, 0.1, 0.01
    span_steps = [np.array([40, 20, 10, 40]), np.array([40, 20, 10, 40]), np.array([40, 20, 10, 40])]
    dev = wl.to("cuda")
    with P.Context(wl.k, wl.d) as ctx:
        ctx.run_csr(dev.row_ptr, dev.col_idx, dev.val, dev.y, wl.shard_off, span_steps[0], wl.eta0, wl.sched, wl.lam,
                    wl.loss, wl.seed)
        for seg in span_steps[1:]:
            ctx.set_models(ctx.combine())
            ctx.continue_csr(dev.row_ptr, dev.col_idx, dev.val, dev.y, wl.shard_off, seg)
        v = ctx.combine().cpu().numpy()
        ctx.check()
    dn = wi.densify(wl)
    W = oracle.run_dense(dn.X, dn.y, wl.shard_off, span_steps[0], wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
    done = span_steps[0].copy()
    for seg in span_steps[1:]:
        wts, _, _ = oracle.weights(done, wl.eta0, wl.sched, wl.lam)
        vv = oracle.combine(W, wts)
        Wn = np.zeros_like(W)
        for j in range(wl.k):
            only = np.zeros(wl.k, dtype=np.int64)
            only[j] = seg[j]
            Wn[j] = oracle.run_dense(dn.X, dn.y, wl.shard_off, only, wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed,
                                     step_begin=int(done[j]),
                                     W_resume=np.tile(vv.astype(np.float32).astype(np.float64), (wl.k, 1)))[j]
        W = Wn
        done = done + seg
    wts, _, _ = oracle.weights(done, wl.eta0, wl.sched, wl.lam)
    assert rel_l2(v, oracle.combine(W, wts)) <= 1e-4


def test_validate_csr_accepts_good_input_and_names_the_bad_row(P):
    # the malformed arrays below are only ever read by the validator (which reads nothing outside [0, nnz)); they
    # are never handed to a chain kernel
    good = wi.config4(k=2, d=512, m=40, base_steps=10, mean_nnz=9.0, max_nnz=20).to("cuda")
    with P.Context(2, 512) as ctx:
        ctx.validate_csr(good.row_ptr, good.col_idx)
        ctx.check()
        nnz = int(good.col_idx.numel())
        row7 = slice(int(good.row_ptr[7]), int(good.row_ptr[8]))
        assert row7.stop - row7.start >= 2
        cases = []
        bad = good.col_idx.clone(); bad[row7.start] = 512            # column == d
        cases.append((good.row_ptr, bad, "detail 7"))
        bad = good.col_idx.clone(); bad[row7.start + 1] = -3          # negative column
        cases.append((good.row_ptr, bad, "detail 7"))
        bad = good.col_idx.clone(); bad[row7.start + 1] = bad[row7.start]   # a column twice in a row
        cases.append((good.row_ptr, bad, "detail 7"))
        rp = good.row_ptr.clone(); rp[0] = -1                         # row 0 starts before the arrays
        cases.append((rp, good.col_idx, "detail 0"))
        rp = good.row_ptr.clone(); rp[-1] = nnz + 10                  # last row claims entries beyond the arrays
        cases.append((rp, good.col_idx, f"detail {rp.numel() - 2}"))
        for rp_, ci_, where in cases:
            ctx.validate_csr(rp_, ci_)
            with pytest.raises(P.WpsgdError) as e:
                ctx.check()
            assert e.value.status_name == "CUDA" and where in str(e.value), str(e.value)
        ctx.validate_csr(good.row_ptr, good.col_idx)  # the context is clean again
        ctx.check()


def test_csr_equals_dense_kernels_on_densified_rows(P):
    wl = wi.config4(k=4, d=1024, m=128, base_steps=300, mean_nnz=20.0)
    wl.loss = LOGISTIC
    v_s, W_s, _, _ = gpu_solve(P, wl)
    v_d, W_d, _, _ = gpu_solve(P, wi.densify(wl))
    assert rel_l2(v_s, v_d) <= 1e-4


# ---- argument checking ----------------------------------------------------------------------------------------
def test_errors_are_reported_not_thrown_from_c(P):
    wl = wi.config1(k=2, d=64, m=16, n_steps=(5, 5)).to("cuda")
    with P.Context(2, 64) as ctx:
        with pytest.raises(P.WpsgdError) as e:
            ctx.combine()
        assert e.value.status_name == "STATE"
        with pytest.raises(P.WpsgdError) as e:
            ctx.get_models()
        assert e.value.status_name == "STATE"
        bad = [dict(n_steps=np.array([5, -1])), dict(shard_off=np.array([0, 16, 8])), dict(eta0=float("nan")),
               dict(lam=-1.0), dict(eta0=10.0, lam=0.2), dict(loss=9), dict(sched=5),
               dict(shard_off=np.array([0, 0, 32]), n_steps=np.array([3, 3]))]
        for kw in bad:
            args = dict(shard_off=wl.shard_off, n_steps=wl.n_steps, eta0=wl.eta0, sched=wl.sched, lam=wl.lam,
                        loss=wl.loss)
            args.update(kw)
            with pytest.raises(P.WpsgdError) as e:
                ctx.run(wl.X, wl.y, args["shard_off"], args["n_steps"], args["eta0"], args["sched"], args["lam"],
                        args["loss"], 0)
            assert e.value.status_name == "INVALID_ARG", kw
        with pytest.raises(P.WpsgdError):
            ctx.set_option("no_such_option", 1)
        with pytest.raises(P.WpsgdError):
            ctx.sample_indices(0, 0, 0, 0, 4)
        ctx.run_workload(wl)  # the context is still usable afterwards
        ctx.combine()
        ctx.check()
        assert ctx.launch_count() >= 3


# ---- shapes at the edges of the launch configurations ---------------------------------------------------------------
def test_many_nodes_with_few_steps(P):
    k, d, m = 3000, 64, 4
    g = torch.Generator().manual_seed(11)
    X = torch.randn(k * m, d, generator=g) / 8
    y = torch.sign(torch.randn(k * m, generator=g))
    n = (np.arange(k) % 7).astype(np.int64)  # 0..6 steps, many idle nodes, ragged last CTA
    wl = wi.Workload("many", k, d, np.arange(k + 1, dtype=np.int64) * m, n, 0.05, 0, 0.01, LOGISTIC, 5, y, X=X)
    assert_parity(P, wl)
    assert_parity(P, wl, {"dense_variant": 3})


@pytest.mark.parametrize("d", [1, 2, 3, 5])
def test_tiny_feature_counts(P, d):
    g = torch.Generator().manual_seed(d)
    k, m = 3, 20
    X = torch.randn(k * m, d, generator=g)
    y = torch.sign(torch.randn(k * m, generator=g))
    wl = wi.Workload("tiny", k, d, np.arange(k + 1, dtype=np.int64) * m, np.array([60, 1, 33]), 0.05, 0, 0.01, LOGISTIC, 3,
                     y, X=X)
    assert_parity(P, wl)


def test_one_long_chain(P):
    wl = wi.config2(k=1, d=256, m=512, base_steps=60000)
    assert_parity(P, wl)


def test_csr_rows_without_nonzeros_and_single_nonzero(P):
    # hand-built CSR: rows 0 and 3 are empty, row 1 has one nonzero, row 2 three
    rp = torch.tensor([0, 0, 1, 4, 4, 6], dtype=torch.int64)
    ci = torch.tensor([5, 0, 3, 7, 1, 6], dtype=torch.int32)
    va = torch.tensor([2.0, 0.5, -1.0, 0.25, 1.5, -0.75])
    y = torch.tensor([1.0, -1.0, 1.0, -1.0, 1.0])
    wl = wi.Workload("gaps", 1, 8, np.array([0, 5]), np.array([200]), 0.1, 1, 0.05, LOGISTIC, 2, y, row_ptr=rp, col_idx=ci,
                     val=va, w0=torch.full((8,), 0.3))
    assert_parity(P, wl)
