"""Trainable kernels (the paper's stated use of the soft PPV, Sections 1 and 6): new weights and
biases installed with rocket_params_set_weights are what every pass then uses, checked against the
oracle run on the new values, and a few steps of gradient descent through the soft transform and its
backward pass lower a loss."""
import copy

import numpy as np
import pytest

import oracle
import paper_2301_08527_b200 as rk
from rocket_inputs import ar1_spike_series, generate_kernels, normal_array

import parity as P

pytestmark = pytest.mark.gpu


def _dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _with_values(kp, weights, bias):
    q = copy.copy(kp)
    q.weights = np.asarray(weights, np.float32)
    q.bias = np.asarray(bias, np.float32)
    return q


@pytest.mark.parametrize("path", [0, 1])
def test_passes_use_the_installed_values(path):
    C, L, K, N, lam, shift = 20, 1000, 300, 3, 10.0, 3.0
    kp = generate_kernels(51, K, C, L)
    X = ar1_spike_series(52, N, C, L)
    p = rk.RocketParams.from_kernel_params(kp)
    p.set_path(path)
    rk.rocket_transform(p, _dev(X))                      # bind and run once with the old values
    rng = np.random.default_rng(53)
    w_new = (kp.weights + 0.3 * rng.normal(size=kp.weights.shape)).astype(np.float32)
    b_new = (kp.bias + 0.2 * rng.normal(size=kp.bias.shape)).astype(np.float32)
    p.set_weights(w_new, b_new)
    kq = _with_values(kp, w_new, b_new)
    ref = oracle.forward(kq, X, lam=lam, shift=shift)
    ppv, mx = P.split_features(rk.rocket_transform(p, _dev(X)).cpu().numpy())
    P.check_hard_ppv(ppv, ref)
    P.check_max(mx, ref)
    feat, arg = rk.rocket_transform_soft(p, _dev(X), lam, shift)
    soft, mx2 = P.split_features(feat.cpu().numpy())
    P.check_soft_ppv(soft, ref)
    P.check_max(mx2, ref)
    g = normal_array(54, (N, 2 * K))
    dW, db = rk.rocket_transform_soft_backward(p, _dev(X), lam, shift, _dev(g), arg)
    ref_dW, ref_db = oracle.backward(kq, X, g, arg.cpu().numpy(), lam=lam, shift=shift)
    P.check_grads(dW.cpu().numpy(), db.cpu().numpy(), ref_dW, ref_db)
    p.close()


def test_gradient_descent_on_the_kernels_lowers_a_loss():
    # loss = mean over (example, kernel) of (softPPV - target)^2 for a fixed random target
    C, L, K, N, lam, shift = 3, 512, 64, 8, 2.0, 0.0
    kp = generate_kernels(61, K, C, L)
    X = _dev(ar1_spike_series(62, N, C, L))
    import torch
    target = torch.from_numpy(np.random.default_rng(63).uniform(0.2, 0.8, (N, K)).astype(np.float32)).cuda()
    p = rk.RocketParams.from_kernel_params(kp)
    w, b = kp.weights.astype(np.float64), kp.bias.astype(np.float64)
    losses = []
    for step in range(8):
        feat, arg = rk.rocket_transform_soft(p, X, lam, shift)
        diff = feat[:, 0::2] - target
        losses.append(float((diff * diff).mean()))
        g = torch.zeros_like(feat)
        g[:, 0::2] = 2.0 * diff / diff.numel()
        dW, db = rk.rocket_transform_soft_backward(p, X, lam, shift, g, arg)
        w -= 100.0 * dW.cpu().numpy().astype(np.float64)
        b -= 100.0 * db.cpu().numpy().astype(np.float64)
        p.set_weights(w, b)
    p.close()
    assert all(b2 < a2 for a2, b2 in zip(losses, losses[1:])), losses
    assert losses[-1] < 0.85 * losses[0]
