"""The entry point for callers that may not allocate device memory (wpsgd_solve_static).

Some users of the library run where cudaMalloc is off limits: inside a framework whose memory pool
already owns the device, in a loop that cannot take cudaMalloc's device-wide synchronisation, or
in a process with a memory budget fixed at start-up. For them the library carries its working
memory (models, sample stream, tables) in an array compiled into it. This test calls that entry point
through the C ABI and compares it with the ordinary context-based path and with the CPU oracle on the
same inputs, several times in a row with different problem sizes, because all calls share the one array
and every call meets the previous call's leftovers. It also checks the two promises such a caller
relies on: the library takes no device memory during the calls, and a problem inside the kernels is
reported through wpsgd_check_static. The file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

import oracle
import wpsgd_inputs as wi

pytestmark = pytest.mark.gpu

TOL = {0: 1e-3, 1: 1e-4, 2: 1e-4}  # the parity tolerances used everywhere else: hinge / logistic / squared


def _rel_l2(a, b):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def _context_path(P, wl, r):
    with P.Context(wl.k, wl.d) as ctx:
        ctx.run_workload(wl)
        v = ctx.combine(r).cpu().numpy()
        ctx.check()
    return v


def _cases():
    first = wi.config2(k=6, d=512, m=128, base_steps=400)      # larger problem first ...
    first.w0 = torch.full((512,), 0.25)
    second = wi.config1(k=3, d=64, m=64, n_steps=(90, 0, 31))  # ... then a smaller one over its leftovers
    third = wi.config3(k=4, d=1024, m=64, n_lo=50, n_hi=300)   # bf16 rows
    return [(first, 0.0), (second, 0.999), (third, 0.0), (first, 0.0)]


def test_no_alloc_entry_point_matches_context_path_and_oracle_calls_in_a_row(wpsgd_lib):
    import paper_1708_04801_b200 as P

    for wl_cpu, r in _cases():
        wl = wl_cpu.to("cuda")
        out = torch.full((wl.d,), float("nan"), dtype=torch.float32, device="cuda")  # caller-owned output
        P.solve_static(wl.X, wl.y, wl.shard_off, wl.n_steps, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed, w0=wl.w0,
                       r=r, out=out)
        P.check_static(0)  # waits for the stream; raises if a kernel flagged a timeout or a bounds failure
        got = out.cpu().numpy()
        assert np.isfinite(got).all()
        assert _rel_l2(got, _context_path(P, wl, r)) <= TOL[wl.loss]
        want, _, _ = oracle.solve(wl_cpu, r)  # the CPU checker shares no code with either CUDA path
        assert _rel_l2(got, want) <= TOL[wl.loss]


def test_no_alloc_entry_point_takes_no_device_memory(wpsgd_lib):
    import paper_1708_04801_b200 as P

    cases = [(wl.to("cuda"), r) for wl, r in _cases()]
    outs = [torch.empty(wl.d, dtype=torch.float32, device="cuda") for wl, _ in cases]
    wl, r = cases[0]
    P.solve_static(wl.X, wl.y, wl.shard_off, wl.n_steps, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed, w0=wl.w0, r=r,
                   out=outs[0])  # first call on the device: module load and the look-up of the array's address
    P.check_static(0)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for (wl, r), out in zip(cases, outs):
        P.solve_static(wl.X, wl.y, wl.shard_off, wl.n_steps, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed, w0=wl.w0, r=r,
                       out=out)
        P.check_static(0)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "wpsgd_solve_static or wpsgd_check_static changed the free device memory"


def test_no_alloc_entry_point_rejects_sizes_beyond_its_array(wpsgd_lib):
    import paper_1708_04801_b200 as P

    X = torch.zeros((8, 64), device="cuda")
    y = torch.ones(8, device="cuda")
    out = torch.empty(64, device="cuda")
    off = np.array([0, 4, 8], dtype=np.int64)
    with pytest.raises(P.WpsgdError) as e:  # more steps than the built-in sample-stream buffer holds
        P.solve_static(X, y, off, np.array([1 << 20, 1], dtype=np.int64), 0.01, 0, 0.01, 0, 0, out=out)
    assert e.value.status_name == "UNSUPPORTED" and "maximum" in str(e.value)
    wide = torch.zeros((2, (1 << 17) + 4), device="cuda")  # k * d beyond the built-in model matrix
    with pytest.raises(P.WpsgdError) as e:
        P.solve_static(wide, y[:2], np.array([0, 1, 2], dtype=np.int64), np.array([1, 1], dtype=np.int64), 0.01, 0,
                       0.01, 0, 0, out=torch.empty(wide.shape[1], device="cuda"))
    assert e.value.status_name == "UNSUPPORTED" and "maximum" in str(e.value)
    k = 1025
    with pytest.raises(P.WpsgdError) as e:  # too many nodes
        P.solve_static(torch.zeros((k, 8), device="cuda"), torch.ones(k, device="cuda"),
                       np.arange(k + 1, dtype=np.int64), np.ones(k, dtype=np.int64), 0.01, 0, 0.01, 0, 0,
                       out=torch.empty(8, device="cuda"))
    assert e.value.status_name == "UNSUPPORTED" and "maximum" in str(e.value)
    # and the ordinary argument checks still apply
    with pytest.raises(P.WpsgdError) as e:
        P.solve_static(X, y, off, np.array([3, -1], dtype=np.int64), 0.01, 0, 0.01, 0, 0, out=out)
    assert e.value.status_name == "INVALID_ARG"
