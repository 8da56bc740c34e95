"""The seeded generators: kernel-parameter distributions (Section 3.1) and synthetic series."""
import numpy as np
import pytest

from rocket_inputs import ar1_spike_series, generate_kernels, random_walk_series


def test_kernel_parameter_distributions():
    K, C, L = 20000, 20, 50000
    p = generate_kernels(8527, K, C, L)
    assert set(np.unique(p.length)) == {7, 9, 11}
    for v in (7, 9, 11):
        assert abs(np.mean(p.length == v) - 1 / 3) < 0.02
    assert abs(np.mean(p.padding > 0) - 0.5) < 0.02
    padded = p.padding > 0
    np.testing.assert_array_equal(p.padding[padded], ((p.length - 1) * p.dilation // 2)[padded])
    assert np.all(p.out_len[padded] == L) and np.all(p.out_len >= 1)
    assert np.all(p.dilation >= 1) and np.all(p.dilation <= (L - 1) // (p.length - 1))
    # log2(d) roughly uniform: mean of x ~ half of the upper limit
    hi = np.log2((L - 1) / (p.length - 1))
    assert abs(np.mean(np.log2(p.dilation + 0.5) / hi) - 0.5) < 0.02
    # P(m = j) = log2((j+1)/j) / log2(min(C, len) + 1)
    for ln in (7, 9, 11):
        sel = p.length == ln
        for j in range(1, ln + 1):
            want = np.log2((j + 1) / j) / np.log2(ln + 1)
            assert abs(np.mean(p.num_channels[sel] == j) - want) < 0.02
    assert np.all((p.bias >= -1) & (p.bias < 1)) and abs(p.bias.mean()) < 0.02
    assert abs(p.num_channels.mean() - 3.43) < 0.1
    co, wo = p.channel_offset, p.weight_offset
    assert co[-1] == len(p.channel_idx) and wo[-1] == len(p.weights)
    for k in range(0, K, 97):
        ch = p.channel_idx[co[k]:co[k + 1]]
        assert len(set(ch.tolist())) == len(ch) and ch.min() >= 0 and ch.max() < C
        assert np.all(np.diff(ch) > 0)
        w = p.weights[wo[k]:wo[k + 1]].reshape(p.num_channels[k], p.length[k]).astype(np.float64)
        assert np.all(np.abs(w.sum(axis=1)) < 1e-5)
    assert abs(p.weights.std() - np.sqrt(1 - 1 / 9)) < 0.03  # centring removes 1/len of the variance
    # channels are chosen uniformly
    freq = np.bincount(p.channel_idx, minlength=C) / len(p.channel_idx)
    assert np.all(np.abs(freq - 1 / C) < 0.01)


def test_same_seed_same_bytes_and_prefix_property():
    a = generate_kernels(5, 300, 6, 2000)
    b = generate_kernels(5, 300, 6, 2000)
    for f in ("length", "dilation", "padding", "num_channels", "channel_idx", "weights", "bias"):
        assert getattr(a, f).tobytes() == getattr(b, f).tobytes()
    c = generate_kernels(5, 100, 6, 2000)
    assert a.length[:100].tobytes() == c.length.tobytes()
    assert a.weights[: len(c.weights)].tobytes() == c.weights.tobytes()
    d = generate_kernels(6, 300, 6, 2000)
    assert a.weights.tobytes() != d.weights.tobytes()


def test_univariate_has_single_channel_zero():
    p = generate_kernels(1, 500, 1, 512)
    assert np.all(p.num_channels == 1) and np.all(p.channel_idx == 0)


def test_subset_keeps_kernels():
    p = generate_kernels(2, 50, 4, 300)
    s = p.subset([7, 3])
    wo = p.weight_offset
    np.testing.assert_array_equal(s.weights[: wo[8] - wo[7]], p.weights[wo[7]:wo[8]])
    assert s.K == 2 and s.dilation[1] == p.dilation[3]


@pytest.mark.parametrize("gen", [random_walk_series, ar1_spike_series])
def test_series_are_normalised_and_seeded(gen):
    x = gen(3, 2, 3, 4000)
    assert x.dtype == np.float32 and x.shape == (2, 3, 4000)
    np.testing.assert_allclose(x.mean(axis=-1), 0, atol=1e-5)
    np.testing.assert_allclose(x.std(axis=-1), 1, atol=1e-4)
    assert gen(3, 2, 3, 4000).tobytes() == x.tobytes()
    assert gen(4, 2, 3, 4000).tobytes() != x.tobytes()


def test_ar1_autocorrelation():
    x = ar1_spike_series(9, 1, 2, 200000).astype(np.float64)
    r1 = np.mean(x[0, :, 1:] * x[0, :, :-1], axis=-1)
    assert np.all(np.abs(r1 - 0.95) < 0.03)
