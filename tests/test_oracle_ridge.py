"""Pins of the oracle's ridge regressor (Section 3.3) against what the definition fixes: a system
worked out by hand, the one-feature closed form, exact recovery of a noiseless linear relation as
alpha goes to zero, the stationarity condition of the penalised objective, the objective not being
improvable by perturbation, shift invariance through the intercept, and the least-squares routine
of the library on the augmented system."""
import numpy as np

import oracle


def test_system_worked_out_by_hand():
    # F centred: [[-1, 0], [0, 1], [1, -1]], y centred: [-1, 0, 1]; Fc^T Fc = [[2, -1], [-1, 2]], Fc^T yc = [2, -1]
    F = np.array([[1.0, 5.0], [2.0, 6.0], [3.0, 4.0]])
    y = np.array([9.0, 10.0, 11.0])
    w, b = oracle.ridge_fit(F, y, 1.0)
    # (A + I) w = [[3, -1], [-1, 3]] w = [2, -1]  ->  w = [5/8, -1/8]
    assert np.allclose(w, [0.625, -0.125], atol=1e-14)
    assert abs(b - (10.0 - (2.0 * 0.625 + 5.0 * -0.125))) < 1e-14


def test_one_feature_closed_form():
    rng = np.random.default_rng(0)
    x, y = rng.normal(size=50), rng.normal(size=50)
    w, b = oracle.ridge_fit(x[:, None], y, 3.5)
    sxy = ((x - x.mean()) * (y - y.mean())).sum()
    sxx = ((x - x.mean()) ** 2).sum()
    assert abs(w[0] - sxy / (sxx + 3.5)) < 1e-13 and abs(b - (y.mean() - x.mean() * w[0])) < 1e-13


def test_noiseless_relation_is_recovered_as_alpha_vanishes():
    rng = np.random.default_rng(1)
    F = rng.normal(size=(40, 6))
    w_true, b_true = rng.normal(size=6), 0.7
    w, b = oracle.ridge_fit(F, F @ w_true + b_true, 1e-12)
    assert np.allclose(w, w_true, atol=1e-9) and abs(b - b_true) < 1e-9
    assert np.allclose(oracle.ridge_predict(F, w, b), F @ w_true + b_true, atol=1e-9)


def test_gradient_of_the_objective_vanishes_and_perturbations_do_not_improve_it():
    rng = np.random.default_rng(2)
    F, y, alpha = rng.normal(size=(30, 80)), rng.normal(size=30), 0.9     # more features than examples
    w, b = oracle.ridge_fit(F, y, alpha)
    r = F @ w + b - y
    assert np.allclose(F.T @ r + alpha * w, 0.0, atol=1e-10)             # d/dw
    assert abs(r.sum()) < 1e-10                                            # d/db
    obj = lambda w_, b_: ((F @ w_ + b_ - y) ** 2).sum() + alpha * (w_ ** 2).sum()
    base = obj(w, b)
    for _ in range(20):
        assert obj(w + 1e-3 * rng.normal(size=80), b + 1e-3 * rng.normal()) > base


def test_shifting_features_or_targets_moves_only_the_intercept():
    rng = np.random.default_rng(3)
    F, y = rng.normal(size=(25, 10)), rng.normal(size=25)
    w0, b0 = oracle.ridge_fit(F, y, 2.0)
    w1, b1 = oracle.ridge_fit(F + 7.0, y - 3.0, 2.0)
    assert np.allclose(w0, w1, atol=1e-12) and abs(b1 - (b0 - 3.0 - 7.0 * w0.sum())) < 1e-11


def test_against_least_squares_on_the_augmented_system():
    rng = np.random.default_rng(4)
    F, y, alpha = rng.normal(size=(60, 15)), rng.normal(size=60), 4.0
    Fc, yc = F - F.mean(axis=0), y - y.mean()
    aug = np.vstack([Fc, np.sqrt(alpha) * np.eye(15)])
    w_ls = np.linalg.lstsq(aug, np.concatenate([yc, np.zeros(15)]), rcond=None)[0]
    w, _ = oracle.ridge_fit(F, y, alpha)
    assert np.allclose(w, w_ls, atol=1e-12)
