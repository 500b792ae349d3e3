"""The entry point for callers that may not allocate device memory (wpsgd_solve_static).

Some users of the library run where cudaMalloc is off limits: inside a framework whose memory pool
already owns the device, in a loop that cannot take cudaMalloc's device-wide synchronisation, or
in a process with a memory budget fixed at start-up. For them the library carries its working
memory (models, sample stream, tables) in an array compiled into it. This test calls that entry point
through the C ABI and compares it with the ordinary context-based path on the same inputs, twice in
a row with different problem sizes, because all calls share the one array and the second call meets
the first call's leftovers. The file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

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


def test_no_alloc_entry_point_matches_context_path_twice_in_a_row(wpsgd_lib):
    import paper_1708_04801_b200 as P

    first = wi.config2(k=6, d=512, m=128, base_steps=400).to("cuda")      # larger problem first ...
    first.w0 = torch.full((512,), 0.25, device="cuda")
    second = wi.config1(k=3, d=64, m=64, n_steps=(90, 0, 31)).to("cuda")  # ... then a smaller one over its leftovers
    third = wi.config3(k=4, d=1024, m=64, n_lo=50, n_hi=300).to("cuda")   # bf16 rows
    for wl, r in ((first, 0.0), (second, 0.999), (third, 0.0), (first, 0.0)):
        out = torch.full((wl.d,), float("nan"), dtype=torch.float32, device="cuda")  # caller-owned output
        P.solve_static(wl.X, wl.y, wl.shard_off, wl.n_steps, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed, w0=wl.w0,
                       r=r, out=out)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        want = _context_path(P, wl, r)
        assert np.isfinite(got).all()
        assert _rel_l2(got, want) <= TOL[wl.loss]


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
