"""Pins of the oracle's per-channel scaling of 8-bit input (Sections 4.1 and 4.3) against what the
definition fixes: exact integers under the identity statistics, values worked out by hand,
zero mean and unit variance under a data set's own statistics, and the transform of scaled bytes
against a convolution written out as plain Python loops."""
import numpy as np

import oracle
from rocket_inputs import channel_statistics, intensity_series_u8, kernels_from_lists


def test_identity_statistics_return_the_integers():
    X = intensity_series_u8(5, 2, 3, 64)
    x = oracle.scale_u8(X, np.zeros(3), np.ones(3))
    assert x.dtype == np.float32 and np.array_equal(x, X.astype(np.float32))


def test_values_worked_out_by_hand():
    X = np.array([[[0, 255, 128, 7], [10, 20, 30, 40]]], dtype=np.uint8)
    x = oracle.scale_u8(X, [127.5, 25.0], [1.0 / 64.0, 0.1])
    want = np.array([[[-127.5 / 64, 127.5 / 64, 0.5 / 64, -120.5 / 64], [-1.5, -0.5, 0.5, 1.5]]])
    assert np.allclose(x, want, rtol=0, atol=1e-7)


def test_own_statistics_give_zero_mean_unit_variance_per_channel():
    X = intensity_series_u8(6, 4, 5, 4096)
    assert X.dtype == np.uint8 and X.min() >= 0 and X.max() <= 255 and len(np.unique(X)) > 50
    mean, inv_std = channel_statistics(X)
    x = oracle.scale_u8(X, mean, inv_std).astype(np.float64)
    assert np.allclose(x.mean(axis=(0, 2)), 0.0, atol=1e-5)
    assert np.allclose(x.std(axis=(0, 2)), 1.0, atol=1e-5)
    # channels keep their own gain and offset out of the result: the raw channel means differ widely
    assert np.ptp(X.astype(np.float64).mean(axis=(0, 2))) > 20


def test_transform_of_scaled_bytes_against_plain_loops():
    X = intensity_series_u8(7, 1, 2, 40)
    mean, inv_std = np.array([100.0, 90.0]), np.array([0.05, 0.02])
    w = [[0.5, -1.0, 0.25, 0.0, 1.0, -0.75, 0.125], [-0.5, 0.5, 1.0, -1.0, 0.25, 0.0, 0.0625]]
    kp = kernels_from_lists(2, 40, [dict(length=7, dilation=3, padding=9, channels=[0, 1], weights=w, bias=0.3)])
    ref = oracle.forward(kp, oracle.scale_u8(X, mean, inv_std))
    z = []
    for i in range(40):
        acc = 0.3
        for q in range(2):
            for j in range(7):
                t = i - 9 + 3 * j
                if 0 <= t < 40:
                    acc += w[q][j] * (float(X[0, q, t]) - mean[q]) * inv_std[q]
        z.append(acc)
    z = np.array(z)
    assert abs(ref.max[0, 0] - z.max()) <= 1e-6 * max(1.0, abs(z.max()))
    assert abs(ref.ppv[0, 0] - (z > 0).mean()) <= 1e-12
