"""Host-side fit of the compute-time model (Eq. 4): exact recovery on synthetic timings and the error metric."""
import numpy as np

from paper_2602_21788_b200 import costfit


def _batches(rng, n):
    out = []
    for _ in range(n):
        B = int(rng.integers(1, 12))
        lens = rng.integers(64, 20000, size=B)
        degs = rng.integers(1, 9, size=B)
        out.append((lens, degs))
    return out


def test_fit_recovers_known_coefficients_exactly():
    rng = np.random.default_rng(0)
    true = dict(alpha1=3.1e-8, alpha2=2.4e-5, beta1=7.0e-3)
    batches = _batches(rng, 40)
    rows = [costfit.design_row(l, d) for l, d in batches]
    times = [costfit.predict(true, l, d) for l, d in batches]
    got = costfit.fit(rows, times)
    for k in true:
        assert np.isclose(got[k], true[k], rtol=1e-8), (k, got[k], true[k])
    assert costfit.relative_errors(got, batches, times).max() < 1e-9


def test_design_row_is_sum_of_squares_lengths_and_degrees():
    r = costfit.design_row([3, 4], [2, 5])
    assert r.tolist() == [25.0, 7.0, 7.0]
    # per-rank form of Eq. 4 for a single sequence at degree d: (alpha1 L^2 + alpha2 L) / d + beta1
    c = dict(alpha1=2.0, alpha2=3.0, beta1=5.0)
    L, d = 10, 4
    assert np.isclose(costfit.predict(c, [L], [d]) / d, (2.0 * L * L + 3.0 * L) / d + 5.0)


def test_relative_error_metric_and_noise_tolerance():
    rng = np.random.default_rng(1)
    true = dict(alpha1=3.0e-8, alpha2=2.0e-5, beta1=5.0e-3)
    batches = _batches(rng, 60)
    rows = [costfit.design_row(l, d) for l, d in batches]
    clean = np.array([costfit.predict(true, l, d) for l, d in batches])
    noisy = clean * (1.0 + 0.03 * rng.standard_normal(len(clean)))
    got = costfit.fit(rows, noisy)
    errs = costfit.relative_errors(got, batches, clean)
    assert errs.mean() < 0.02                             # 3 % timing noise leaves the model within 2 %
    assert np.isclose(costfit.relative_errors(true, [batches[0]], [2.0 * clean[0]])[0], 0.5)
