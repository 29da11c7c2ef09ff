"""Latency predictor end to end on the GPU (Section 5.1): table from nm_latency_table, measured
stacks of linear layers, nm_predictor_fit through the C ABI against the oracle on the same
measurements, and the error of the calibrated model on held-out configurations."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_calibration_on_a_small_stack():
    from oracle import nm_predictor_oracle as po
    from paper_2607_12505_b200 import binding as nm
    from bench import predictor_eval

    out, A, y = predictor_eval.evaluate(model="deit_s", batch=16, fit=14, test=6, group="operator", reps=10, seed=1, blocks=3)
    # the library's fit and the oracle's agree on the measured data
    g, b, r = nm.nm_predictor_fit(A[:14], y[:14])
    go, bo, ro = po.fit(A[:14], y[:14])
    assert r == pytest.approx(ro, rel=1e-8, abs=1e-9)
    assert np.all(g >= 0) and b >= 0
    pred = nm.nm_predictor_eval(g, b, A[14:])
    want = [po.predict(g, b, row) for row in A[14:]]
    assert pred == pytest.approx(want, rel=1e-12)
    # the calibrated model predicts held-out stacks (the paper reports errors within 5 %)
    assert out["test_err_max"] < 0.15, out
    assert out["test_err_mean"] < 0.08, out
