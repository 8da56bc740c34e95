"""Pins for the oracle's pooling: PPV (Eq. 1-2), max, softPPV (Eq. 3-4)."""
import math

import numpy as np
import pytest

import oracle
from rocket_inputs import generate_kernels, kernels_from_lists, random_walk_series

RNG = np.random.default_rng(5)


def _brute(p, X, n, k, lam, shift, eps=1e-5):
    """Pure-Python restatement on tiny inputs (no numpy arithmetic, no oracle code)."""
    co, wo = p.channel_offset, p.weight_offset
    ln, d, pad, m = int(p.length[k]), int(p.dilation[k]), int(p.padding[k]), int(p.num_channels[k])
    nout = p.L + 2 * pad - (ln - 1) * d
    zs = []
    for i in range(nout):
        z = float(p.bias[k])
        for q in range(m):
            c = int(p.channel_idx[co[k] + q])
            for j in range(ln):
                t = i - pad + j * d
                if 0 <= t < p.L:
                    z += float(p.weights[wo[k] + q * ln + j]) * float(X[n, c, t])
        zs.append(z)
    ppv = sum(1 for z in zs if z > 0) / nout
    soft = sum(1.0 / (1.0 + math.exp(-(lam * z + shift))) for z in zs) / nout
    pos_eps = sum(1 for z in zs if z > eps)
    amb = sum(1 for z in zs if -eps <= z <= eps)
    return ppv, max(zs), soft, zs.index(max(zs)), pos_eps, amb


def test_brute_force_on_tiny_series():
    p = generate_kernels(3, 40, 3, 48)
    X = random_walk_series(4, 2, 3, 48)
    out = oracle.forward(p, X, lam=2.0, shift=3.0)
    for n in range(2):
        for k in range(p.K):
            ppv, mx, soft, arg, pos_eps, amb = _brute(p, X, n, k, 2.0, 3.0)
            assert out.ppv[n, k] == pytest.approx(ppv, abs=1e-15)
            assert out.max[n, k] == pytest.approx(mx, rel=1e-13, abs=1e-13)
            assert out.soft[n, k] == pytest.approx(soft, abs=1e-13)
            assert out.argmax[n, k] == arg
            assert out.pos_eps[n, k] == pos_eps and out.amb[n, k] == amb


def test_brute_force_counts_near_zero_with_a_wide_band():
    # a band wide enough that many outputs fall inside it: the two counts that set the acceptance
    # band of the hard-PPV parity checks are compared with the pure-Python count
    p = generate_kernels(13, 30, 2, 40)
    X = (0.05 * random_walk_series(14, 2, 2, 40)).astype(np.float32)
    p.bias = (0.02 * p.bias).astype(np.float32)
    p.weights = (0.05 * p.weights).astype(np.float32)
    out = oracle.forward(p, X, amb_eps=0.01)
    seen_amb = 0
    for n in range(2):
        for k in range(p.K):
            _, _, _, _, pos_eps, amb = _brute(p, X, n, k, 1.0, 3.0, eps=0.01)
            assert out.pos_eps[n, k] == pos_eps and out.amb[n, k] == amb
            seen_amb += amb
    assert seen_amb > 50   # the case does exercise the band


def test_hand_worked_counts_around_the_ambiguity_band():
    # single-tap kernel (w_0 = 1, other taps 0, bias 0, no padding): z_i = x_i for i < L - 6.
    # With eps = 2^-17 (exact in binary) the outputs sit below, on and above both edges of the band:
    #   z:  -2^-16   -2^-17   -2^-18   0   2^-18   2^-17   2^-17 (1 + 2^-23)   2^-16
    #   z > eps            : the last two                       -> pos_eps = 2
    #   |z| <= eps         : -2^-17, -2^-18, 0, 2^-18, 2^-17    -> amb = 5   (both edges belong to the band)
    #   z > 0              : four values                        -> PPV = 4/8
    e = 2.0 ** -17
    z = [-2 * e, -e, -e / 2, 0.0, e / 2, e, e * (1 + 2.0 ** -23), 2 * e]
    x = np.array(z + [9.0] * 6, np.float32)[None, None, :]
    assert [float(v) for v in x[0, 0, :8]] == z       # every value is exact in fp32
    w = np.zeros((1, 7), np.float32)
    w[0, 0] = 1.0
    p = kernels_from_lists(1, 14, [dict(dilation=1, padding=0, channels=[0], weights=w, bias=0.0)])
    out = oracle.forward(p, x, amb_eps=e)
    assert out.out_len[0, 0] == 8
    assert out.pos_eps[0, 0] == 2 and out.amb[0, 0] == 5 and out.ppv[0, 0] == 0.5
    # the default band, 1e-5: float32(1e-5) lies just below 1e-5 (inside the band), its successor just above
    f = np.float32(1e-5)
    g = np.nextafter(f, np.float32(1))
    assert float(f) < 1e-5 < float(g)
    z2 = [-2e-5, -5e-6, 0.0, 5e-6, float(f), float(g), 2e-5, -float(g)]
    x2 = np.array(z2 + [9.0] * 6, np.float32)[None, None, :]
    out = oracle.forward(p, x2)
    assert out.pos_eps[0, 0] == 2 and out.amb[0, 0] == 4 and out.ppv[0, 0] == 0.5
    # a dropped or doubled count would also break the partition: below + band + above = all outputs
    below = sum(1 for v in x2[0, 0, :8] if float(v) < -1e-5)
    assert below + out.amb[0, 0] + out.pos_eps[0, 0] == 8


def test_hand_worked_case_features():
    x = np.array([1, -2, 3, -4, 5, -6, 7], np.float32)[None, None, :]
    p = kernels_from_lists(1, 7, [dict(dilation=2, padding=0, channels=[0], weights=[[1, 0, -1]], bias=0.5),
                                  dict(dilation=2, padding=2, channels=[0], weights=[[1, 0, -1]], bias=0.5)])
    out = oracle.forward(p, x, lam=1.0, shift=0.0)
    assert out.ppv[0, 0] == pytest.approx(1 / 3, abs=1e-15) and out.max[0, 0] == 4.5
    assert out.argmax[0, 0] == 1 and out.gap[0, 0] == 8.0
    sig = lambda v: 1 / (1 + math.exp(-v))
    assert out.soft[0, 0] == pytest.approx((2 * sig(-3.5) + sig(4.5)) / 3, abs=1e-15)
    assert out.ppv[0, 1] == pytest.approx(3 / 7, abs=1e-15) and out.max[0, 1] == 5.5
    assert out.argmax[0, 1] == 6 and out.gap[0, 1] == 1.0


def test_invariants_on_random_kernels():
    p = generate_kernels(21, 300, 4, 200)
    X = random_walk_series(22, 3, 4, 200)
    out = oracle.forward(p, X, lam=5.0, shift=-3.0)
    assert np.all((out.ppv >= 0) & (out.ppv <= 1))
    counts = out.ppv * out.out_len
    np.testing.assert_allclose(counts, np.round(counts), atol=1e-9)
    assert np.array_equal(out.ppv > 0, out.max > 0)
    assert np.all((out.soft > 0) & (out.soft < 1))
    assert np.all(out.gap >= 0)
    assert np.all((out.argmax >= 0) & (out.argmax < out.out_len))
    assert np.all(out.pos_eps <= counts + 1e-9) and np.all(counts <= out.pos_eps + out.amb + 1e-9)


def test_positive_scaling_keeps_ppv_and_scales_max():
    p = generate_kernels(31, 60, 2, 128)
    X = random_walk_series(32, 2, 2, 128)
    a = oracle.forward(p, X)
    p4 = generate_kernels(31, 60, 2, 128)
    p4.weights = p4.weights * np.float32(4.0)
    p4.bias = p4.bias * np.float32(4.0)
    b = oracle.forward(p4, X)
    np.testing.assert_array_equal(a.ppv, b.ppv)
    np.testing.assert_allclose(b.max, 4 * a.max, rtol=1e-14)
    np.testing.assert_array_equal(a.argmax, b.argmax)


@pytest.mark.parametrize("bias", [0.75, -0.3, 0.0])
def test_constant_input_mean_centred_kernel(bias):
    # rows sum to zero => z_i = b everywhere (no padding): PPV = [b > 0], MAX = b, soft = sigma(lam*b + s)
    C, L = 2, 64
    X = np.broadcast_to(np.array([2.0, -1.0], np.float32)[None, :, None], (1, C, L)).copy()
    W = np.array([[1, -2, 1, 0, 3, -3, 0], [0.5, 0.5, -1, 0, 0, 0, 0]], np.float32)
    p = kernels_from_lists(C, L, [dict(dilation=3, padding=0, channels=[0, 1], weights=W, bias=bias)])
    for lam, s in ((1.0, 3.0), (10.0, -3.0)):
        out = oracle.forward(p, X, lam=lam, shift=s)
        b = float(np.float32(bias))
        assert out.ppv[0, 0] == (1.0 if b > 0 else 0.0)
        assert out.max[0, 0] == pytest.approx(b, abs=1e-14)
        assert out.soft[0, 0] == pytest.approx(1 / (1 + math.exp(-(lam * b + s))), abs=1e-14)
        assert out.argmax[0, 0] == 0 and out.gap[0, 0] == pytest.approx(0, abs=1e-14)


def test_heaviside_is_strict_at_zero():
    # all-zero input and zero bias: every z_i == 0 exactly -> PPV 0 (Eq. 1: H(0) = 0)
    X = np.zeros((1, 1, 32), np.float32)
    p = kernels_from_lists(1, 32, [dict(dilation=1, padding=3, channels=[0], weights=np.ones((1, 7)), bias=0.0)])
    out = oracle.forward(p, X)
    assert out.ppv[0, 0] == 0.0 and out.max[0, 0] == 0.0 and out.amb[0, 0] == 32 and out.pos_eps[0, 0] == 0


@pytest.mark.parametrize("shift", [3.0, -3.0, 0.0])
def test_lambda_zero_gives_sigmoid_of_shift(shift):
    p = generate_kernels(41, 50, 3, 100)
    X = random_walk_series(42, 2, 3, 100)
    out = oracle.forward(p, X, lam=0.0, shift=shift)
    np.testing.assert_allclose(out.soft, 1 / (1 + math.exp(-shift)), atol=1e-14)
    if shift == 3.0:
        np.testing.assert_allclose(out.soft, 0.9525741268224334, atol=1e-14)


@pytest.mark.parametrize("shift", [3.0, -3.0])
def test_soft_tends_to_hard_as_lambda_grows(shift):
    p = generate_kernels(51, 80, 3, 150)
    X = random_walk_series(52, 2, 3, 150)
    prev = None
    for lam in (2.0, 10.0, 100.0, 1e4, 1e7):
        out = oracle.forward(p, X, lam=lam, shift=shift)
        err = np.abs(out.soft - out.ppv)
        # |sigma(lam z + s) - H(z)| <= sigma(|s| - lam |z|); bound with the smallest |z| of the pair
        n, k = np.unravel_index(np.argmax(err), err.shape)
        z = oracle.conv(p, X, n, k)
        with np.errstate(over="ignore"):
            bound = np.mean(1 / (1 + np.exp(-(abs(shift) - lam * np.abs(z)))))
        assert err[n, k] <= bound + 1e-12
        if prev is not None:
            assert err.mean() < prev
        prev = err.mean()
    assert np.max(err) < 1e-3


def test_soft_is_monotone_in_bias_and_max_shifts_with_bias():
    p = generate_kernels(61, 30, 2, 90)
    X = random_walk_series(62, 1, 2, 90)
    a = oracle.forward(p, X, lam=3.0, shift=3.0)
    p2 = generate_kernels(61, 30, 2, 90)
    p2.bias = (p2.bias + np.float32(0.5)).astype(np.float32)
    b = oracle.forward(p2, X, lam=3.0, shift=3.0)
    assert np.all(b.soft > a.soft)
    np.testing.assert_allclose(b.max - a.max, (p2.bias.astype(np.float64) - p.bias.astype(np.float64))[None, :],
                               atol=1e-12)


def test_argmax_is_lowest_index_on_ties_and_gap_zero():
    x = np.array([0, 1, 0, 0, 1, 0, 0, 0, 0, 0, 0, 0], np.float32)[None, None, :]
    w = np.zeros((1, 7), np.float32)
    w[0, 0] = 1.0
    p = kernels_from_lists(1, 12, [dict(dilation=1, padding=0, channels=[0], weights=w, bias=0.0)])
    out = oracle.forward(p, x)
    assert out.argmax[0, 0] == 1 and out.max[0, 0] == 1.0 and out.gap[0, 0] == 0.0


def test_pairs_api_matches_full_grid():
    p = generate_kernels(71, 25, 2, 70)
    X = random_walk_series(72, 3, 2, 70)
    full = oracle.forward(p, X, lam=4.0, shift=3.0)
    pn = np.array([2, 0, 1, 2], np.int32)
    pk = np.array([24, 3, 3, 0], np.int32)
    sub = oracle.forward_pairs(p, X, pn, pk, lam=4.0, shift=3.0)
    np.testing.assert_array_equal(sub.ppv, full.ppv[pn, pk])
    np.testing.assert_array_equal(sub.soft, full.soft[pn, pk])
    np.testing.assert_array_equal(sub.max, full.max[pn, pk])
