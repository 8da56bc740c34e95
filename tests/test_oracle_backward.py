"""Pins for the oracle's backward pass: finite differences of the oracle's own forward, closed
forms, and structural identities (chain rule through Eq. 3-4 and the convolution)."""
import math

import numpy as np
import pytest

import oracle
from rocket_inputs import generate_kernels, kernels_from_lists, normal_array, random_walk_series


def _loss(p, X, g, lam, shift):
    out = oracle.forward(p, X, lam=lam, shift=shift)
    return float(np.sum(g.astype(np.float64) * oracle.features_soft(out)))


@pytest.mark.parametrize("lam,shift", [(1.0, 3.0), (10.0, -3.0), (2.0, 0.0)])
def test_central_finite_differences(lam, shift):
    p = generate_kernels(7, 12, 3, 40)
    X = random_walk_series(8, 2, 3, 40)
    g = normal_array(9, (2, 2 * p.K))
    out = oracle.forward(p, X, lam=lam, shift=shift)
    assert out.gap.min() > 1e-4  # away from max ties, so the max is differentiable
    dW, db = oracle.backward(p, X, g, out.argmax, lam=lam, shift=shift)
    # fp32 parameters: perturb by an exactly representable step and difference in fp64
    h = 2.0 ** -12
    rng = np.random.default_rng(10)
    for idx in rng.choice(len(p.weights), 60, replace=False):
        w0 = p.weights[idx]
        p.weights[idx] = np.float32(w0 + h); up = _loss(p, X, g, lam, shift); hp = float(p.weights[idx]) - float(w0)
        p.weights[idx] = np.float32(w0 - h); dn = _loss(p, X, g, lam, shift); hm = float(w0) - float(p.weights[idx])
        p.weights[idx] = w0
        fd = (up - dn) / (hp + hm)
        assert dW[idx] == pytest.approx(fd, rel=2e-5, abs=2e-6)
    for k in range(p.K):
        b0 = p.bias[k]
        p.bias[k] = np.float32(b0 + h); up = _loss(p, X, g, lam, shift); hp = float(p.bias[k]) - float(b0)
        p.bias[k] = np.float32(b0 - h); dn = _loss(p, X, g, lam, shift); hm = float(b0) - float(p.bias[k])
        p.bias[k] = b0
        assert db[k] == pytest.approx((up - dn) / (hp + hm), rel=2e-5, abs=2e-6)


def test_lambda_zero_leaves_only_the_max_path():
    p = generate_kernels(17, 10, 2, 50)
    X = random_walk_series(18, 2, 2, 50)
    g = normal_array(19, (2, 2 * p.K))
    out = oracle.forward(p, X, lam=0.0)
    dW, db = oracle.backward(p, X, g, out.argmax, lam=0.0)
    # db = sum_n gM ; dW[q][j] = sum_n gM * xpad[S[q]][argmax - p + j d]
    np.testing.assert_allclose(db, g[:, 1::2].astype(np.float64).sum(axis=0), atol=1e-12)
    co, wo = p.channel_offset, p.weight_offset
    for k in range(p.K):
        ln, d, pad = int(p.length[k]), int(p.dilation[k]), int(p.padding[k])
        for q in range(int(p.num_channels[k])):
            c = p.channel_idx[co[k] + q]
            for j in range(ln):
                exp = 0.0
                for n in range(2):
                    t = int(out.argmax[n, k]) - pad + j * d
                    if 0 <= t < p.L:
                        exp += float(g[n, 2 * k + 1]) * float(X[n, c, t])
                assert dW[wo[k] + q * ln + j] == pytest.approx(exp, abs=1e-12)


def test_constant_input_closed_form():
    # h constant => dW[q][j] = (gP*lam*h(1-h) + gM) * a_{S[q]},  db = gP*lam*h(1-h) + gM   (p = 0)
    C, L, lam, s = 2, 40, 1.5, 3.0
    a = np.array([0.5, -2.0], np.float32)
    X = np.broadcast_to(a[None, :, None], (1, C, L)).copy()
    W = np.array([[1, -1, 2, -2, 0, 0, 0], [3, -3, 0, 0, 1, -1, 0]], np.float32)
    p = kernels_from_lists(C, L, [dict(dilation=2, padding=0, channels=[1, 0], weights=W, bias=0.2)])
    g = np.array([[0.7, -1.3]], np.float32)
    out = oracle.forward(p, X, lam=lam, shift=s)
    dW, db = oracle.backward(p, X, g, out.argmax, lam=lam, shift=s)
    b = float(np.float32(0.2))
    h = 1 / (1 + math.exp(-(lam * b + s)))
    core = float(g[0, 0]) * lam * h * (1 - h) + float(g[0, 1])
    assert db[0] == pytest.approx(core, abs=1e-13)
    np.testing.assert_allclose(dW.reshape(2, 7), core * np.array([[a[1]] * 7, [a[0]] * 7], np.float64), atol=1e-12)


def test_bias_gradient_equals_sum_of_gz_and_examples_add():
    p = generate_kernels(27, 8, 3, 60)
    X = random_walk_series(28, 3, 3, 60)
    g = normal_array(29, (3, 2 * p.K))
    lam, s = 4.0, -3.0
    out = oracle.forward(p, X, lam=lam, shift=s)
    dW, db = oracle.backward(p, X, g, out.argmax, lam=lam, shift=s)
    for k in range(p.K):
        tot = 0.0
        for n in range(3):
            z = oracle.conv(p, X, n, k)
            h = 1 / (1 + np.exp(-(lam * z + s)))
            gz = float(g[n, 2 * k]) * lam / len(z) * h * (1 - h)
            gz[out.argmax[n, k]] += float(g[n, 2 * k + 1])
            tot += gz.sum()
        assert db[k] == pytest.approx(tot, rel=1e-12, abs=1e-13)
    parts = [oracle.backward(p, X, g, out.argmax, lam=lam, shift=s, examples=[n]) for n in range(3)]
    np.testing.assert_allclose(dW, sum(pp[0] for pp in parts), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(db, sum(pp[1] for pp in parts), rtol=1e-12, atol=1e-13)
    only = oracle.backward(p, X, g, out.argmax, lam=lam, shift=s, kernels=[5, 2])
    wo = p.weight_offset
    np.testing.assert_array_equal(only[0][wo[5]:wo[6]], dW[wo[5]:wo[6]])
    np.testing.assert_array_equal(only[1][[2, 5]], db[[2, 5]])
    assert only[1][0] == 0.0
