"""GPU-vs-oracle parity of the ridge regressor on pooled features (Section 3.3) through the C ABI.

Tolerances.  The library solves in double precision and stores w and b as fp32, so against the
float64 oracle: relative L2 error of w <= 1e-5, |b - b_oracle| <= 1e-5 * max(1, |b_oracle|, max|y|),
predictions within 1e-5 * max(1, max|y|).  At the paper's size (677 examples, 20,000 features) the
oracle's P x P normal equations are out of reach; there the result is checked by the conditions that
single out the minimiser of the strictly convex objective: F_c^T r + alpha w = 0 and sum(r) = 0,
within 1e-4 of the size of their terms.
"""
import numpy as np
import pytest

import oracle
import paper_2301_08527_b200 as rk
from rocket_inputs import ar1_spike_series, generate_kernels

pytestmark = pytest.mark.gpu


def _dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _problem(seed, N, P, noise=0.1):
    rng = np.random.default_rng(seed)
    F = np.concatenate([rng.random((N, P // 2)), rng.normal(1.0, 0.5, (N, P - P // 2))], axis=1).astype(np.float32)
    w_true = rng.normal(0, 1.0 / np.sqrt(P), P)
    y = (1.2 + (F - F.mean(axis=0)) @ w_true + noise * rng.normal(size=N)).astype(np.float32)
    return F, y


@pytest.mark.parametrize("N,P,alpha", [(20, 50, 0.1), (64, 300, 10.0), (100, 30, 0.5), (33, 1, 2.0), (1, 7, 1.0),
                                       (129, 515, 1.0), (40, 64, 0.0 + 1e-3)])
def test_fit_and_predict_small_full(N, P, alpha):
    F, y = _problem(100 + N, N, P)
    w, b = rk.rocket_ridge_fit(_dev(F), _dev(y), alpha)
    w_ref, b_ref = oracle.ridge_fit(F, y, alpha)
    w_gpu, b_gpu = w.cpu().numpy().astype(np.float64), float(b.cpu()[0])
    denom = max(np.linalg.norm(w_ref), 1e-30)
    assert np.linalg.norm(w_gpu - w_ref) / denom <= 1e-5 or np.linalg.norm(w_gpu - w_ref) <= 1e-7
    scale = max(1.0, abs(b_ref), float(np.abs(y).max()))
    assert abs(b_gpu - b_ref) <= 1e-5 * scale
    yhat = rk.rocket_ridge_predict(_dev(F), w, b).cpu().numpy()
    assert np.abs(yhat - oracle.ridge_predict(F, w_ref, b_ref)).max() <= 1e-5 * scale
    # prediction alone, from the oracle's coefficients rounded to fp32
    yhat2 = rk.rocket_ridge_predict(_dev(F), _dev(w_ref.astype(np.float32)), _dev(np.array([b_ref], np.float32))).cpu().numpy()
    assert np.abs(yhat2 - oracle.ridge_predict(F, w_ref.astype(np.float32), np.float32(b_ref))).max() <= 2e-6 * scale


def test_fit_at_paper_size_satisfies_the_conditions_of_the_minimiser():
    N, P, alpha = 677, 20000, 1.0
    F, y = _problem(7, N, P)
    w, b = rk.rocket_ridge_fit(_dev(F), _dev(y), alpha)
    w64, b64 = w.cpu().numpy().astype(np.float64), float(b.cpu()[0])
    assert np.all(np.isfinite(w64)) and np.isfinite(b64)
    F64 = F.astype(np.float64)
    r = F64 @ w64 + b64 - y
    Fc = F64 - F64.mean(axis=0)
    g = Fc.T @ r + alpha * w64
    assert np.linalg.norm(g) <= 1e-4 * np.linalg.norm(Fc.T @ (y - y.mean()))
    assert abs(r.sum()) <= 1e-4 * np.abs(y).sum()
    # two fits are bitwise identical, and predictions reproduce b + F w
    w2, b2 = rk.rocket_ridge_fit(_dev(F), _dev(y), alpha)
    import torch
    assert torch.equal(w, w2) and torch.equal(b, b2)
    yhat = rk.rocket_ridge_predict(_dev(F[:60]), w, b).cpu().numpy()
    assert np.abs(yhat - (F64[:60] @ w64 + b64)).max() <= 1e-5 * max(1.0, float(np.abs(y).max()))


def test_transform_features_feed_the_regressor_without_leaving_the_device():
    # step (1)+(2)+(3) of Section 3 on the device; the oracle repeats all three on the host
    kp = generate_kernels(77, 200, 3, 256)
    X = ar1_spike_series(78, 24, 3, 256)
    y = (1.0 + 0.3 * X[:, 0, :64].mean(axis=1) + 0.05 * np.random.default_rng(79).normal(size=24)).astype(np.float32)
    p = rk.RocketParams.from_kernel_params(kp)
    feat = rk.rocket_transform(p, _dev(X))
    w, b = rk.rocket_ridge_fit(feat, _dev(y), 5.0)
    yhat = rk.rocket_ridge_predict(feat, w, b).cpu().numpy()
    p.close()
    ref_feat = oracle.features_hard(oracle.forward(kp, X))
    w_ref, b_ref = oracle.ridge_fit(ref_feat, y, 5.0)
    # the features themselves differ within their own tolerances (PPV counts near zero crossings), so compare predictions
    assert np.abs(yhat - oracle.ridge_predict(ref_feat, w_ref, b_ref)).max() <= 1e-3
    assert np.abs(yhat - y).mean() < np.abs(y - y.mean()).mean()


def test_ridge_argument_errors():
    import torch
    F, y = _problem(5, 8, 4)
    with pytest.raises(rk.RocketError):
        rk.rocket_ridge_fit(_dev(F), _dev(y), -1.0)
    with pytest.raises(rk.RocketError):
        rk.rocket_ridge_fit(_dev(F), _dev(y), float("nan"))
    with pytest.raises(rk.RocketError):
        rk.rocket_ridge_fit(torch.zeros((5000, 2), device="cuda"), torch.zeros(5000, device="cuda"), 1.0)
    with pytest.raises(rk.RocketError):   # alpha = 0 with identical rows: not positive definite
        rk.rocket_ridge_fit(torch.ones((4, 3), device="cuda"), torch.ones(4, device="cuda"), 0.0)
    with pytest.raises(ValueError):
        rk.rocket_ridge_fit(_dev(F), _dev(y[:3]), 1.0)
    empty = rk.rocket_ridge_predict(torch.zeros((0, 4), device="cuda"), torch.zeros(4, device="cuda"), torch.zeros(1, device="cuda"))
    assert empty.shape == (0,)
