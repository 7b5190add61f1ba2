"""The latency decomposition of Sec. 4.3 (non-negative fit of t(L) = a L^2 + b L + c) as bench.py computes it."""
import importlib.util
import os

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    m = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(m)
    return m


def test_fit_recovers_known_coefficients_and_stays_non_negative():
    b = _bench()
    L = [2048, 4096, 8192, 16384, 32768, 65536]
    x = np.asarray(L) / 1024.0
    (a, lin, c), resid = b.fit_latency(L, 0.002 * x * x + 0.11 * x + 0.04)
    np.testing.assert_allclose([a, lin, c], [0.002, 0.11, 0.04], rtol=1e-9)
    assert resid < 1e-9
    # a purely linear-time step with a little concave noise: the quadratic term is clamped at zero, never negative
    (a, lin, c), _ = b.fit_latency(L, 0.1 * x - 1e-5 * x * x + 0.05)
    assert a == 0.0 and lin > 0 and c >= 0.0


def test_profile_traffic_reads_the_committed_summaries():
    b = _bench()
    for kind in ("scan", "in_proj"):
        v = b.profile_traffic(kind)
        assert v is not None and 1e7 < v < 1e10
