"""Pins of the half-precision oracle (oracle/rocket_f16_oracle.c): binary16 samples, weights and biases, one
rounding to binary16 per multiply-add, bias first, channels in the kernel's order, taps 0 .. len - 1 (the
reduced-precision form of the transform the paper's Section 5 points to).

  exact cases      small integers never round: the result equals the double-precision oracle exactly
  hand-worked      a tie that goes to even, a step that only a FUSED multiply-add gets right, the order of the taps
  brute force      rational arithmetic in pure Python, rounded with a table of all finite binary16 numbers
  error bound      |z16 - z64| <= (steps + 1) 2^-11 (|b| + sum |w||x|) against the double-precision oracle
"""
from bisect import bisect_left
from fractions import Fraction

import numpy as np
import pytest

import oracle
from rocket_inputs import ar1_spike_series, generate_kernels, kernels_from_lists


def _one(kp, X, n=0, k=0):
    return oracle.forward_f16_pairs(kp, X, [n], [k], return_z=True)


def test_small_integers_never_round_and_equal_the_double_precision_oracle():
    rng = np.random.default_rng(1)
    C, L = 3, 40
    ks = [dict(dilation=int(rng.integers(1, 4)), padding=int(rng.integers(0, 5)), channels=[0, 2],
               weights=rng.integers(-3, 4, size=(2, 7)), bias=float(rng.integers(-5, 6))) for _ in range(12)]
    kp = kernels_from_lists(C, L, ks)
    X = rng.integers(-4, 5, size=(3, C, L)).astype(np.float32)      # |z| <= 5 + 14 * 12 < 2048: every sum exact
    a, b = oracle.forward_f16(kp, X), oracle.forward(kp, X)
    assert np.array_equal(a.ppv, b.ppv) and np.array_equal(a.max, b.max) and np.array_equal(a.argmax, b.argmax)
    assert np.array_equal(a.count, np.round(b.ppv * b.out_len).astype(np.int64))


def test_hand_worked_roundings():
    L = 9
    # a tie goes to even: 2048 + 1 = 2049 lies midway between 2048 and 2050 -> 2048; 2050 + 1 = 2051 -> 2052
    kp = kernels_from_lists(1, L, [dict(weights=[[1, 0, 0, 0, 0, 0, 0]], bias=1.0)])
    X = np.zeros((1, 1, L), np.float32); X[0, 0, 0] = 2048.0; X[0, 0, 1] = 2050.0
    z = _one(kp, X).z
    assert z.tolist() == [2048.0, 2052.0, 1.0]
    # only a fused step gets this right: (1 + 2^-10)^2 = 1 + 2^-9 + 2^-20; with the addend -(1 + 2^-9) the exact
    # sum 2^-20 is a binary16 number (a subnormal), whereas rounding the product first would leave 0
    e = 2.0 ** -10
    kp = kernels_from_lists(1, L, [dict(weights=[[1 + e, 0, 0, 0, 0, 0, 0]], bias=-(1 + 2 * e))])
    X = np.zeros((1, 1, L), np.float32); X[0, 0, 0] = 1 + e
    out = _one(kp, X)
    assert out.z[0] == 2.0 ** -20 and out.count[0] == 1 and out.max[0] == 2.0 ** -20
    # the order of the steps: bias, then tap 0, then tap 1.  b = 2048, w0 x = 1, w1 x = 1: (2048 + 1) -> 2048,
    # (2048 + 1) -> 2048; any other order (1 + 1 first) would give 2050
    kp = kernels_from_lists(1, L, [dict(weights=[[1, 1, 0, 0, 0, 0, 0]], bias=2048.0)])
    X = np.ones((1, 1, L), np.float32)
    assert _one(kp, X).z[0] == 2048.0
    # channels in the order of the channel list: the same with the two ones coming from two channels
    kp = kernels_from_lists(2, L, [dict(channels=[0, 1], weights=[[1, 0, 0, 0, 0, 0, 0], [1, 0, 0, 0, 0, 0, 0]], bias=2048.0)])
    X = np.ones((1, 2, L), np.float32)
    assert _one(kp, X).z[0] == 2048.0
    # samples, weights and biases are rounded to binary16 first: 0.1 -> 0.0999755859375
    kp = kernels_from_lists(1, L, [dict(weights=[[1, 0, 0, 0, 0, 0, 0]], bias=0.0)])
    X = np.full((1, 1, L), 0.1, np.float32)
    assert _one(kp, X).z[0] == 0.0999755859375
    # Eq. 1 is strict: an output that is exactly zero does not count
    kp = kernels_from_lists(1, L, [dict(weights=[[1, 0, 0, 0, 0, 0, 0]], bias=-1.0)])
    X = np.ones((1, 1, L), np.float32); X[0, 0, 1] = 1.5
    out = _one(kp, X)
    assert out.count[0] == 1 and out.max[0] == 0.5 and out.argmax[0] == 1


def _all_binary16():
    bits = np.arange(0, 0x7C00, dtype=np.uint16)                       # non-negative finite values, ascending
    return [Fraction(float(v)) for v in bits.view(np.float16).astype(np.float64)]


def _round16(x, table):
    """Nearest binary16 number to the rational x, ties to the even significand, by search in the table."""
    if x < 0:
        return -_round16(-x, table)
    i = bisect_left(table, x)
    if i < len(table) and table[i] == x:
        return x
    lo, hi = table[i - 1], table[i]
    if x - lo != hi - x:
        return lo if x - lo < hi - x else hi
    return lo if (i - 1) % 2 == 0 else hi                              # index parity = significand parity


def test_brute_force_with_rational_arithmetic():
    table = _all_binary16()
    rng = np.random.default_rng(5)
    C, L = 3, 30
    ks = []
    for ln, d, p, chans in [(7, 1, 0, [0]), (9, 2, 8, [1, 2]), (11, 1, 5, [0, 1, 2]), (7, 3, 9, [2, 0])]:
        ks.append(dict(dilation=d, padding=p, channels=chans, weights=rng.normal(size=(len(chans), ln)), bias=float(rng.uniform(-1, 1))))
    kp = kernels_from_lists(C, L, ks)
    X = (3.0 * rng.normal(size=(2, C, L))).astype(np.float32)
    X16, W16, b16 = oracle.round_f16(X).astype(np.float64), oracle.round_f16(kp.weights).astype(np.float64), oracle.round_f16(kp.bias).astype(np.float64)
    for n in range(2):
        for k in range(kp.K):
            ln, d, p, m = int(kp.length[k]), int(kp.dilation[k]), int(kp.padding[k]), int(kp.num_channels[k])
            S = kp.channel_idx[kp.channel_offset[k]:kp.channel_offset[k + 1]]
            W = W16[kp.weight_offset[k]:kp.weight_offset[k + 1]].reshape(m, ln)
            zs = []
            for i in range(int(kp.out_len[k])):
                z = Fraction(b16[k])
                for q in range(m):
                    for j in range(ln):
                        t = i - p + j * d
                        x = Fraction(X16[n, S[q], t]) if 0 <= t < L else Fraction(0)
                        z = _round16(z + Fraction(W[q, j]) * x, table)
                zs.append(z)
            out = oracle.forward_f16_pairs(kp, X, [n], [k], return_z=True)
            assert [Fraction(v) for v in out.z.tolist()] == zs
            assert out.count[0] == sum(1 for z in zs if z > 0)
            assert Fraction(out.max[0]) == max(zs) and out.argmax[0] == zs.index(max(zs))


def test_error_bound_against_the_double_precision_oracle():
    kp = generate_kernels(11, 40, 6, 400)
    X = ar1_spike_series(12, 2, 6, 400)
    X16, W16, b16 = oracle.round_f16(X).astype(np.float64), oracle.round_f16(kp.weights).astype(np.float64), oracle.round_f16(kp.bias).astype(np.float64)
    u = 2.0 ** -11
    for k in range(kp.K):
        out = oracle.forward_f16_pairs(kp, X, [1], [k], return_z=True)
        z64 = oracle.conv(kp, X, 1, k)
        ln, d, p, m = int(kp.length[k]), int(kp.dilation[k]), int(kp.padding[k]), int(kp.num_channels[k])
        S = kp.channel_idx[kp.channel_offset[k]:kp.channel_offset[k + 1]]
        W = np.abs(W16[kp.weight_offset[k]:kp.weight_offset[k + 1]].reshape(m, ln))
        Wt = np.abs(kp.weights[kp.weight_offset[k]:kp.weight_offset[k + 1]].astype(np.float64).reshape(m, ln))
        # sum of |w||x| per output, with the unrounded values (their rounding is part of the bound)
        xa = np.abs(np.pad(X[1].astype(np.float64), ((0, 0), (p, p + ln * d))))
        mag = np.abs(kp.bias[k]) + sum(Wt[q, j] * xa[S[q], j * d:j * d + len(z64)] for q in range(m) for j in range(ln))
        steps = m * ln
        bound = ((1 + u) ** (steps + 3) - 1) * mag + 2.0 ** -24 * (steps + 1)
        assert np.all(np.abs(out.z - z64) <= bound), k


def test_values_that_are_not_binary16_are_refused():
    import ctypes
    kp = kernels_from_lists(1, 9, [dict(weights=[[1, 0, 0, 0, 0, 0, 0]], bias=0.0)])
    X = np.full((1, 1, 9), 70000.0, np.float32)
    with pytest.raises(FloatingPointError):
        oracle.forward_f16(kp, X)
