"""Pins for the MINIROCKET oracle (oracle/minirocket_oracle.c) and its parameters (rocket_inputs.minirocket)."""
import math

import numpy as np
import pytest

import oracle
from rocket_inputs import ar1_spike_series, generate_minirocket, kernels_from_lists, random_walk_series


def test_parameter_set_has_the_stated_structure():
    for C, L, F in ((1, 64, 500), (20, 5000, 10000), (3, 50000, 10000), (9, 512, 84)):
        p = generate_minirocket(7, C, L, F)
        assert p.F == (F // 84) * 84 and p.taps.shape == (84, 3)
        assert len({tuple(t) for t in p.taps.tolist()}) == 84 and np.all(np.diff(p.taps, axis=1) > 0)
        for k in range(84):
            w = p.weights(k)
            assert sorted(set(w.tolist())) == [-1.0, 2.0] and w.sum() == 0.0 and (w == 2.0).sum() == 3
        d = p.dilation
        assert d.min() == 1 and 8 * d.max() <= L - 1                    # an unpadded combination keeps >= 1 output
        nf = np.diff(p.feature_offset)
        assert nf.min() >= 1 and p.feature_offset[-1] == p.F
        per_kernel = np.zeros(84, np.int64)
        np.add.at(per_kernel, p.kernel_index, nf)
        assert np.all(per_kernel == p.F // 84)                           # every kernel owns the same number of features
        assert np.all((p.num_channels >= 1) & (p.num_channels <= min(C, 9)))
        co = p.channel_offset
        for c in range(0, p.n_combos, 37):
            S = p.channel_idx[co[c]:co[c + 1]]
            assert len(set(S.tolist())) == len(S) and S.min() >= 0 and S.max() < C
        assert np.all((p.quantile >= 0) & (p.quantile < 1)) and np.all((p.example_draw >= 0) & (p.example_draw < 1))
        a = generate_minirocket(7, C, L, F)
        assert a.channel_idx.tobytes() == p.channel_idx.tobytes() and a.quantile.tobytes() == p.quantile.tobytes()


def _brute_conv(p, X, n, c):
    """Pure-Python restatement (no numpy arithmetic, no oracle code)."""
    d, taps = int(p.dilation[c]), set(int(t) for t in p.taps[p.kernel_index[c]])
    co = p.channel_offset
    first, last = p.out_range(c)
    zs = []
    for i in range(first, last):
        z = 0.0
        for q in range(co[c], co[c + 1]):
            ch = int(p.channel_idx[q])
            for j in range(9):
                t = i + (j - 4) * d
                if 0 <= t < p.L:
                    z += (2.0 if j in taps else -1.0) * float(X[n, ch, t])
        zs.append(z)
    return zs


def _brute_quantile(zs, q):
    s = sorted(zs)
    pos = q * (len(s) - 1)
    lo = int(math.floor(pos))
    hi = min(lo + 1, len(s) - 1)
    return s[lo] + (pos - lo) * (s[hi] - s[lo])


def test_brute_force_on_tiny_series():
    p = generate_minirocket(3, 3, 40, 84 * 6)
    X = random_walk_series(4, 3, 3, 40)
    bias = oracle.minirocket_fit(p, X)
    out = oracle.minirocket_transform(p, X, bias, eps=0.01)
    ex = oracle.minirocket_example_index(p, 3)
    for c in range(0, p.n_combos, 11):
        zfit = _brute_conv(p, X, int(ex[c]), c)
        np.testing.assert_allclose(oracle.minirocket_conv(p, X, int(ex[c]), c), zfit, rtol=1e-13, atol=1e-13)
        for f in range(p.feature_offset[c], p.feature_offset[c + 1]):
            b = _brute_quantile(zfit, float(p.quantile[f]))
            assert bias[f] == pytest.approx(b, rel=1e-12, abs=1e-12)
            for n in range(3):
                zs = _brute_conv(p, X, n, c)
                assert out.ppv[n, f] == pytest.approx(sum(1 for z in zs if z > bias[f]) / len(zs), abs=1e-15)
                assert out.pos_eps[n, f] == sum(1 for z in zs if z > bias[f] + 0.01)
                assert out.amb[n, f] == sum(1 for z in zs if abs(z - bias[f]) <= 0.01)
                assert out.n_out[f] == len(zs)


def test_every_feature_is_the_ppv_of_the_equivalent_rocket_kernel():
    # a MINIROCKET feature is the PPV of a ROCKET kernel with the same two-valued weights on every chosen channel,
    # the same dilation, padding 4 d or none, and bias -b: the ROCKET oracle (pinned on its own) must agree
    p = generate_minirocket(5, 4, 200, 84 * 4)
    X = ar1_spike_series(6, 3, 4, 200)
    bias = oracle.minirocket_fit(p, X)
    out = oracle.minirocket_transform(p, X, bias)
    co = p.channel_offset
    ks, feats = [], []
    for c in range(0, p.n_combos, 5):
        S = p.channel_idx[co[c]:co[c + 1]]
        d = int(p.dilation[c])
        for f in range(p.feature_offset[c], p.feature_offset[c + 1]):
            ks.append(dict(dilation=d, padding=4 * d if p.padded[c] else 0, channels=S.tolist(),
                           weights=np.tile(p.weights(p.kernel_index[c]), (len(S), 1)), bias=-float(np.float32(bias[f]))))
            feats.append(f)
    kp = kernels_from_lists(4, 200, ks)
    ref = oracle.forward(kp, X)
    # the ROCKET side carries the bias in fp32: compare where no output lies within that rounding of the bias
    b32 = np.float32(bias[feats]).astype(np.float64)
    chk = oracle.minirocket_transform(p, X, np.where(np.isin(np.arange(p.F), feats), np.float32(bias).astype(np.float64), bias))
    np.testing.assert_array_equal(ref.ppv, chk.ppv[:, feats])
    assert np.array_equal(ref.out_len[0], chk.n_out[feats])


def test_quantile_matches_numpy_and_hand_values():
    p = generate_minirocket(9, 2, 120, 84 * 3)
    X = ar1_spike_series(10, 4, 2, 120)
    bias = oracle.minirocket_fit(p, X)
    ex = oracle.minirocket_example_index(p, 4)
    for c in range(0, p.n_combos, 17):
        z = oracle.minirocket_conv(p, X, int(ex[c]), c)
        for f in range(p.feature_offset[c], p.feature_offset[c + 1]):
            assert bias[f] == pytest.approx(np.quantile(z, p.quantile[f]), rel=1e-12, abs=1e-12)
    # hand-worked: outputs 0, 10, 20, 30 -> quantile 0.5 sits at position 1.5 = 15; quantile 0.25 at 0.75 = 7.5
    assert _brute_quantile([30.0, 0.0, 20.0, 10.0], 0.5) == 15.0 and _brute_quantile([30.0, 0.0, 20.0, 10.0], 0.25) == 7.5


def test_constant_input_gives_zero_outputs_without_padding():
    # every kernel sums to zero: on a constant series the unpadded outputs are exactly 0, every bias is 0 and,
    # the comparison being strict, every PPV is 0; padded combinations see the zeros of the padding instead
    p = generate_minirocket(11, 2, 100, 84 * 2)
    X = np.broadcast_to(np.array([1.5, -0.25], np.float32)[None, :, None], (2, 2, 100)).copy()
    bias = oracle.minirocket_fit(p, X)
    out = oracle.minirocket_transform(p, X, bias)
    for c in range(p.n_combos):
        fs = slice(p.feature_offset[c], p.feature_offset[c + 1])
        if not p.padded[c]:
            assert np.all(bias[fs] == 0.0) and np.all(out.ppv[:, fs] == 0.0)
            assert np.all(out.amb[:, fs] == out.n_out[fs][None, :])
        else:
            z = oracle.minirocket_conv(p, X, 0, c)
            d = int(p.dilation[c])
            assert np.all(z[4 * d: 100 - 4 * d] == 0.0)


def test_ppv_is_a_fraction_and_falls_as_the_bias_rises():
    p = generate_minirocket(13, 3, 300, 84 * 5)
    X = ar1_spike_series(14, 2, 3, 300)
    bias = oracle.minirocket_fit(p, X)
    a = oracle.minirocket_transform(p, X, bias)
    b = oracle.minirocket_transform(p, X, bias + 0.5)
    assert np.all((a.ppv >= 0) & (a.ppv <= 1)) and np.all(b.ppv <= a.ppv)
    counts = a.ppv * a.n_out[None, :]
    np.testing.assert_allclose(counts, np.round(counts), atol=1e-9)
    assert np.all(a.pos_eps <= counts + 1e-9) and np.all(counts <= a.pos_eps + a.amb + 1e-9)
    # on the example a bias was read from, the PPV is the share of outputs above that quantile
    ex = oracle.minirocket_example_index(p, 2)
    for c in range(0, p.n_combos, 23):
        for f in range(p.feature_offset[c], p.feature_offset[c + 1]):
            assert abs(a.ppv[ex[c], f] - (1.0 - p.quantile[f])) <= 1.5 / a.n_out[f] + 1e-12
