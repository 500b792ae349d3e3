"""The C-ABI library: it builds, loads and exports every symbol the header declares; its host-side
logic (weights, argument checks) is checked against the oracle. No GPU compute here."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = []
    for f in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if f.endswith(".h"):
            src = open(os.path.join(ROOT, "include", f)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names += re.findall(r"\b(wpsgd_[a-z0-9_]+)\s*\(", src)
    return sorted(set(names))


def test_library_exports_every_declared_symbol(wpsgd_lib):
    import paper_1708_04801_b200 as P

    declared = _declared()
    assert len(declared) >= 15
    for name in declared:
        assert hasattr(wpsgd_lib, name), f"{name} declared in include/ but not exported"
    assert sorted(P.EXPORTED_SYMBOLS) == declared


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    import paper_1708_04801_b200.binding as B

    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "_HERE", str(tmp_path))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.load_library()


def test_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_1708_04801_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"
    text = open(os.path.join(ROOT, "oracle", "wpsgd_oracle.cpp")).read() + open(os.path.join(ROOT, "oracle", "__init__.py")).read()
    assert "paper_1708_04801_b200" not in text and "wpsgd.h" not in text


@pytest.mark.parametrize("case", [
    dict(n=[1000, 800, 500, 250], eta=0.01, sched=0, lam=1e-3, r=0.0),
    dict(n=[20000, 10000, 5000] * 5 + [20000], eta=0.05, sched=0, lam=1e-4, r=0.0),
    dict(n=[800000] * 8 + [160000] * 2, eta=1e-4, sched=0, lam=0.01, r=0.99999),
    dict(n=[65536, 45875, 26214, 6553, 0], eta=0.1, sched=1, lam=1e-5, r=0.0),
    dict(n=[400, 130, 0, 399], eta=0.1, sched=1, lam=0.5, r=0.0),
    dict(n=[7, 7, 7], eta=0.1, sched=0, lam=0.5, r=0.0),
    dict(n=[100, 10, 55], eta=0.1, sched=0, lam=0.1, r=1.0),
    dict(n=[5], eta=0.1, sched=0, lam=0.1, r=float("nan")),
    dict(n=[10 ** 6, 1, 1, 1], eta=0.1, sched=0, lam=0.1, r=0.0),
    dict(n=[100, 90], eta=0.1, sched=0, lam=0.1, r=1.5),
])
def test_host_weights_match_oracle(wpsgd_lib, case):
    import paper_1708_04801_b200 as P

    n = np.array(case["n"], dtype=np.int64)
    got, holds, tot = P.weights(n, case["eta"], case["sched"], case["lam"], case["r"])
    want, wholds, wtot = oracle.weights(n, case["eta"], case["sched"], case["lam"], case["r"])
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-300)
    assert holds == wholds
    assert tot == pytest.approx(wtot, rel=1e-12)
    assert abs(got.sum() - 1.0) < 1e-14


def test_host_weights_reject_bad_input(wpsgd_lib):
    import paper_1708_04801_b200 as P

    with pytest.raises(P.WpsgdError) as e:
        P.weights([3, -1], 0.1, 0, 0.1)
    assert e.value.status_name == "INVALID_ARG"
    with pytest.raises(P.WpsgdError):
        P.weights([3, 1], 0.1, 7, 0.1)


def test_create_without_device_reports_error_instead_of_crashing(wpsgd_lib):
    import torch

    if torch.cuda.is_available():
        pytest.skip("a device is present")
    h = ctypes.c_void_p()
    st = wpsgd_lib.wpsgd_create(0, None, 4, 64, ctypes.byref(h))
    assert st == 3 and not h.value
    assert b"CUDA" in wpsgd_lib.wpsgd_last_error(None)
    assert wpsgd_lib.wpsgd_create(0, None, 0, 64, ctypes.byref(h)) == 1
    assert wpsgd_lib.wpsgd_destroy(None) == 0
    assert wpsgd_lib.wpsgd_check(None) == 1


def test_validity_condition_of_averaging_every_span(wpsgd_lib):
    import paper_1708_04801_b200 as P

    # k = 4, delays 0, 0, 1000, 1000 at r = 1 - 0.1 * 0.01 = 0.999: sum r^T = 2 + 2 * 0.999^1000
    n = [2000, 2000, 1000, 1000]
    r = 1.0 - float(np.float32(0.1)) * float(np.float32(0.01))
    tot = 2 + 2 * r ** 1000
    for span, want in ((100, (4 / tot) * r ** 100), (1000, (4 / tot) * r ** 1000)):
        holds, lhs = P.span_valid(n, 0.1, 0.01, span)
        assert lhs == pytest.approx(want, rel=1e-9)
        assert holds == (want < 1.0)
    assert P.span_valid(n, 0.1, 0.01, 100)[0] is False   # a short span cannot make up for the delays
    assert P.span_valid(n, 0.1, 0.01, 1000)[0] is True
    assert P.span_valid([50, 50, 50], 0.1, 0.01, 1)[0] is True   # balanced: any span is valid
    with pytest.raises(P.WpsgdError) as e:
        P.span_valid(n, 0.1, 0.01, -1)
    assert e.value.status_name == "INVALID_ARG"
    # a caller-given rate (Eq. 8) enters the sum, the contraction per step stays 1 - eta lambda
    holds, lhs = P.span_valid(n, 0.1, 0.01, 500, r=0.9995)
    assert lhs == pytest.approx((4 / (2 + 2 * 0.9995 ** 1000)) * r ** 500, rel=1e-9)


@pytest.mark.parametrize("seed,node,m,n_begin,count", [
    (0, 0, 4096, 0, 1000), (12345678901234567, 3, 1, 0, 17), (7, 1023, (1 << 32) - 1, 5, 64),
    (2, 9, 65536, (1 << 34) + 3, 33), (3, 2, 3, 1, 2), (1, 0, 100, 7, 0),
])
@pytest.mark.parametrize("sampling", [0, 1])
def test_host_sample_stream_is_bit_exact(wpsgd_lib, seed, node, m, n_begin, count, sampling):
    """The library's host-side stream (the function its kernels call) against the checker's own Philox / shuffle."""
    import paper_1708_04801_b200 as P

    got = P.sample_indices_host(seed, node, m, n_begin, count, sampling)
    oracle.set_sampling(sampling)
    try:
        want = oracle.sample_indices(seed, node, m, n_begin, count)
    finally:
        oracle.set_sampling(0)
    np.testing.assert_array_equal(got, want)


def test_host_sample_stream_rejects_bad_input(wpsgd_lib):
    import paper_1708_04801_b200 as P

    for args in ((0, -1, 10, 0, 5, 0), (0, 0, 0, 0, 5, 0), (0, 0, 1 << 32, 0, 5, 0), (0, 0, 10, -1, 5, 0), (0, 0, 10, 0, 5, 2)):
        with pytest.raises(P.WpsgdError) as e:
            P.sample_indices_host(*args)
        assert e.value.status_name == "INVALID_ARG"
