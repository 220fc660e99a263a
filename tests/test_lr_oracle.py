"""Pins for the classifier-fit oracle (paper Section 3.2 / 4.1: L2-regularised logistic regression as scikit-learn
fits it): the library's own solver, closed forms, and invariances of the minimiser."""
import numpy as np
import pytest

import aj_inputs as gen
from oracle import aj_lr_oracle as lro


def _problem(n=400, F=12, seed=3, dtype=gen.F32):
    X, y = gen.make_labelled_features(n, F, dtype, seed)
    return gen.to_f64(X, dtype), y


@pytest.mark.parametrize("C", [1.0, 1e-2, 1e-4])
def test_minimiser_equals_scikit_learn(C):
    from sklearn.linear_model import LogisticRegression

    X, y = _problem()
    w, b = lro.fit(X, y, C)
    ref = LogisticRegression(C=C, tol=1e-12, max_iter=20000).fit(X, y)
    np.testing.assert_allclose(w, ref.coef_[0], rtol=0, atol=2e-7 * max(1.0, np.abs(w).max()))
    assert abs(b - ref.intercept_[0]) <= 2e-6
    _, gw, gb = lro.objective(X, y, C, w, b)
    assert np.abs(gw).max() <= 1e-10 and abs(gb) <= 1e-10
    np.testing.assert_allclose(lro.predict_proba(X, w, b), ref.predict_proba(X)[:, 1], rtol=0, atol=1e-6)


def test_closed_forms_and_invariances():
    X, y = _problem(n=300, F=6)
    # features that carry nothing: w = 0 and the intercept is the log-odds of the labels
    w, b = lro.fit(np.zeros_like(X), y, 0.5)
    assert np.abs(w).max() == 0.0
    assert b == pytest.approx(np.log(y.mean() / (1 - y.mean())), abs=1e-9)
    # every row twice = twice the coefficient C
    w1, b1 = lro.fit(np.vstack([X, X]), np.concatenate([y, y]), 0.05)
    w2, b2 = lro.fit(X, y, 0.1)
    np.testing.assert_allclose(w1, w2, atol=1e-9)
    assert b1 == pytest.approx(b2, abs=1e-9)
    # swapping the classes flips the sign of (w, b); permuting features permutes w; the row order is immaterial
    w3, b3 = lro.fit(X, 1 - y, 0.1)
    np.testing.assert_allclose(w3, -w2, atol=1e-9)
    assert b3 == pytest.approx(-b2, abs=1e-9)
    perm = np.random.default_rng(0).permutation(X.shape[1])
    w4, _ = lro.fit(X[:, perm], y, 0.1)
    np.testing.assert_allclose(w4, w2[perm], atol=1e-9)
    rows = np.random.default_rng(1).permutation(X.shape[0])
    w5, b5 = lro.fit(X[rows], y[rows], 0.1)
    np.testing.assert_allclose(w5, w2, atol=1e-9)
    # a stronger regulariser (smaller C) shrinks the weights; the minimum is lower than at nearby points
    assert np.linalg.norm(lro.fit(X, y, 1e-3)[0]) < np.linalg.norm(w2) < np.linalg.norm(lro.fit(X, y, 10.0)[0])
    f0 = lro.objective(X, y, 0.1, w2, b2)[0]
    rng = np.random.default_rng(2)
    for _ in range(20):
        dw, db = 1e-3 * rng.standard_normal(w2.shape), 1e-3 * rng.standard_normal()
        assert lro.objective(X, y, 0.1, w2 + dw, b2 + db)[0] > f0


def test_gradient_is_the_derivative_of_the_objective():
    X, y = _problem(n=50, F=5)
    rng = np.random.default_rng(4)
    w, b = rng.standard_normal(5), 0.3
    f, gw, gb = lro.objective(X, y, 0.7, w, b)
    eps = 1e-6
    for j in range(5):
        e = np.zeros(5)
        e[j] = eps
        num = (lro.objective(X, y, 0.7, w + e, b)[0] - lro.objective(X, y, 0.7, w - e, b)[0]) / (2 * eps)
        assert num == pytest.approx(gw[j], abs=1e-6)
    num = (lro.objective(X, y, 0.7, w, b + eps)[0] - lro.objective(X, y, 0.7, w, b - eps)[0]) / (2 * eps)
    assert num == pytest.approx(gb, abs=1e-6)


def test_generated_labels_have_the_stated_share_and_are_learnable():
    X, y = gen.make_labelled_features(5000, 32, gen.BF16, seed=9)
    assert X.dtype == np.uint16 and y.dtype == np.uint8
    assert abs(y.mean() - 0.2) < 0.005
    Xf = gen.to_f64(X, gen.BF16)
    w, b = lro.fit(Xf, y, 1e-2)
    p = lro.predict_proba(Xf, w, b)
    assert p[y == 1].mean() > p[y == 0].mean() + 0.15
