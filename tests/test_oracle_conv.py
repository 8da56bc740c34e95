"""Pins for the oracle's convolution (Section 3 step (1), Section 3.1): library routine on
zero-stuffed kernels, moving sums, closed forms, impulse response, linearity."""
import os

import numpy as np
import pytest

import oracle
from rocket_inputs import kernels_from_lists

RNG = np.random.default_rng(11)


def _one(C, L, **kd):
    return kernels_from_lists(C, L, [kd])


@pytest.mark.parametrize("length", [7, 9, 11])
@pytest.mark.parametrize("dilation", [1, 2, 3, 5])
@pytest.mark.parametrize("padded", [False, True])
def test_matches_numpy_correlate_on_zero_stuffed_kernel(length, dilation, padded):
    C, L = 3, 64
    X = RNG.standard_normal((2, C, L)).astype(np.float32)
    chans = [2, 0]
    W = RNG.standard_normal((len(chans), length)).astype(np.float32)
    b = 0.37
    pad = (length - 1) * dilation // 2 if padded else 0
    p = _one(C, L, dilation=dilation, padding=pad, channels=chans, weights=W, bias=b)
    for n in range(2):
        z = oracle.conv(p, X, n, 0)
        ref = np.full(L + 2 * pad - (length - 1) * dilation, np.float32(b).astype(np.float64))
        for q, c in enumerate(chans):
            stuffed = np.zeros((length - 1) * dilation + 1)
            stuffed[::dilation] = W[q].astype(np.float64)
            xp = np.concatenate([np.zeros(pad), X[n, c].astype(np.float64), np.zeros(pad)])
            ref = ref + np.correlate(xp, stuffed, mode="valid")
        assert z.shape == ref.shape
        np.testing.assert_allclose(z, ref, rtol=0, atol=1e-12)


def test_moving_sum():
    L, length = 40, 9
    X = RNG.standard_normal((1, 1, L)).astype(np.float32)
    p = _one(1, L, dilation=1, padding=0, channels=[0], weights=np.ones((1, length)), bias=0.0)
    z = oracle.conv(p, X, 0, 0)
    cs = np.concatenate([[0.0], np.cumsum(X[0, 0].astype(np.float64))])
    np.testing.assert_allclose(z, cs[length:] - cs[:-length], atol=1e-12)


def test_constant_input_closed_form_with_padding_edges():
    C, L, length, d = 2, 50, 7, 3
    a = np.array([1.5, -0.25])
    X = np.broadcast_to(a[None, :, None], (1, C, L)).astype(np.float32).copy()
    W = RNG.standard_normal((2, length)).astype(np.float32)
    pad = (length - 1) * d // 2
    b = -0.4
    p = _one(C, L, dilation=d, padding=pad, channels=[0, 1], weights=W, bias=b)
    z = oracle.conv(p, X, 0, 0)
    assert len(z) == L
    W64 = W.astype(np.float64)
    for i in range(L):
        inr = np.array([0 <= i - pad + j * d < L for j in range(length)])
        expect = np.float64(np.float32(b)) + sum(a[q] * W64[q][inr].sum() for q in range(2))
        assert abs(z[i] - expect) < 1e-12
    # unpadded: every output equals b + sum_q a_q * sum_j W[q][j]
    p0 = _one(C, L, dilation=d, padding=0, channels=[0, 1], weights=W, bias=b)
    z0 = oracle.conv(p0, X, 0, 0)
    assert len(z0) == L - (length - 1) * d
    np.testing.assert_allclose(z0, np.float64(np.float32(b)) + (a[:, None] * W64).sum(), atol=1e-12)


@pytest.mark.parametrize("pad_on", [False, True])
def test_unit_impulse_reproduces_dilated_weights(pad_on):
    L, length, d, t0 = 60, 9, 4, 37
    X = np.zeros((1, 1, L), np.float32)
    X[0, 0, t0] = 1.0
    W = RNG.standard_normal((1, length)).astype(np.float32)
    pad = (length - 1) * d // 2 if pad_on else 0
    p = _one(1, L, dilation=d, padding=pad, channels=[0], weights=W, bias=0.0)
    z = oracle.conv(p, X, 0, 0)
    expect = np.zeros_like(z)
    for j in range(length):
        i = t0 + pad - j * d
        if 0 <= i < len(z):
            expect[i] = W[0, j]
    np.testing.assert_array_equal(z, expect)


def test_no_flip_tap_j_reads_forward_in_time():
    # asymmetric kernel on a ramp: z_i = sum_j w_j * (i + j*d) distinguishes correlation from flipped conv
    L, length, d = 30, 7, 2
    X = np.arange(L, dtype=np.float32)[None, None, :]
    w = np.arange(1, length + 1, dtype=np.float32)[None, :]
    p = _one(1, L, dilation=d, padding=0, channels=[0], weights=w, bias=0.0)
    z = oracle.conv(p, X, 0, 0)
    j = np.arange(length)
    expect = np.array([np.sum(w[0] * (i + j * d)) for i in range(L - (length - 1) * d)], dtype=np.float64)
    np.testing.assert_allclose(z, expect, atol=1e-9)


def test_linearity_and_time_shift_equivariance():
    C, L, length, d = 2, 80, 11, 3
    X = RNG.standard_normal((1, C, L)).astype(np.float32)
    W = RNG.standard_normal((2, length)).astype(np.float32)
    p = _one(C, L, dilation=d, padding=0, channels=[1, 0], weights=W, bias=0.25)
    p2 = _one(C, L, dilation=d, padding=0, channels=[1, 0], weights=2 * W, bias=0.5)
    np.testing.assert_allclose(oracle.conv(p2, X, 0, 0), 2 * oracle.conv(p, X, 0, 0), atol=1e-12)
    Xs = np.roll(X, 5, axis=-1)
    z, zs = oracle.conv(p, X, 0, 0), oracle.conv(p, Xs, 0, 0)
    np.testing.assert_allclose(zs[5:], z[:-5], atol=1e-12)


def test_channel_selection_uses_listed_channels_in_listed_order():
    C, L, length = 4, 30, 7
    X = RNG.standard_normal((1, C, L)).astype(np.float32)
    W = RNG.standard_normal((2, length)).astype(np.float32)
    pa = _one(C, L, dilation=1, channels=[3, 1], weights=W, bias=0.0)
    pb = _one(C, L, dilation=1, channels=[1, 3], weights=W[::-1], bias=0.0)
    np.testing.assert_allclose(oracle.conv(pa, X, 0, 0), oracle.conv(pb, X, 0, 0), atol=1e-12)
    single = _one(C, L, dilation=1, channels=[3], weights=W[:1], bias=0.0)
    other = _one(C, L, dilation=1, channels=[1], weights=W[1:], bias=0.0)
    np.testing.assert_allclose(oracle.conv(pa, X, 0, 0),
                               oracle.conv(single, X, 0, 0) + oracle.conv(other, X, 0, 0), atol=1e-12)


def test_hand_worked_golden_case():
    path = os.path.join(os.path.dirname(__file__), "golden", "tiny_conv_case.txt")
    rec = {}
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        rec[key] = np.array([float(v) for v in vals])
    x = rec["x"].astype(np.float32)[None, None, :]
    for pad, key in ((0, "z_pad0"), (2, "z_pad2")):
        p = _one(1, x.shape[-1], dilation=int(rec["dilation"][0]), padding=pad, channels=[0],
                 weights=rec["w"][None, :], bias=float(rec["bias"][0]))
        np.testing.assert_array_equal(oracle.conv(p, x, 0, 0), rec[key])
