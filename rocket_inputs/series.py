"""Seeded synthetic series standing in for the paper's laser-reflection data.

Values are drawn in fp64 with numpy's PCG64 generator, z-normalised per sample per
channel (population standard deviation) and rounded once to fp32.
"""
import numpy as np


def _znorm(x):
    mu = x.mean(axis=-1, keepdims=True)
    sd = x.std(axis=-1, keepdims=True)
    sd = np.where(sd > 0, sd, 1.0)
    return ((x - mu) / sd).astype(np.float32)


def random_walk_series(seed, N, C, L):
    """Gaussian random walks (cumulative sums of N(0,1) steps), z-normalised. [N, C, L] fp32."""
    rng = np.random.default_rng(seed)
    return _znorm(np.cumsum(rng.standard_normal((N, C, L)), axis=-1))


def ar1_spike_series(seed, N, C, L, phi=0.95, spike_rate=1e-3):
    """AR(1) noise plus sparse positive spikes, z-normalised. [N, C, L] fp32.

    y_0 ~ N(0, 1/(1-phi^2)) (stationary start), y_t = phi*y_{t-1} + e_t with unit-variance
    innovations; each step independently receives an Exp(1) spike with probability
    spike_rate.  Built one example at a time so peak memory stays near 3 copies of a row set.
    """
    from scipy.signal import lfilter
    rng = np.random.default_rng(seed)
    out = np.empty((N, C, L), dtype=np.float32)
    for n in range(N):
        e = rng.standard_normal((C, L))
        e[:, 0] /= np.sqrt(1.0 - phi * phi)
        y = lfilter([1.0], [1.0, -phi], e, axis=-1)
        spikes = (rng.random((C, L)) < spike_rate) * rng.exponential(1.0, (C, L))
        out[n] = _znorm(y + spikes)
    return out


def normal_array(seed, shape):
    """Standard normal fp32 array (upstream gradients for the backward pass)."""
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


def intensity_series_u8(seed, N, C, L, phi=0.95, spike_rate=1e-3):
    """Raw sensor-like input: integer intensities 0..255 as uint8, [N, C, L].

    The same AR(1)-plus-spikes signal as ar1_spike_series, but left unnormalised: every channel
    (sensor) has its own gain (12 to 40 intensity steps per unit of signal) and offset (60 to 180),
    shared by all examples, and the result is rounded and clipped to 0..255.
    """
    from scipy.signal import lfilter
    rng = np.random.default_rng(seed)
    gain = rng.uniform(12.0, 40.0, size=(C, 1))
    offset = rng.uniform(60.0, 180.0, size=(C, 1))
    out = np.empty((N, C, L), dtype=np.uint8)
    for n in range(N):
        e = rng.standard_normal((C, L))
        e[:, 0] /= np.sqrt(1.0 - phi * phi)
        y = lfilter([1.0], [1.0, -phi], e, axis=-1) * np.sqrt(1.0 - phi * phi)
        spikes = (rng.random((C, L)) < spike_rate) * rng.exponential(1.0, (C, L))
        out[n] = np.clip(np.rint(offset + gain * (y + spikes)), 0, 255).astype(np.uint8)
    return out


def channel_statistics(X_u8):
    """Per-channel mean and reciprocal standard deviation over a whole data set [N, C, L] (fp32 arrays
    of C values): the statistics a caller would compute once on the training set."""
    x = np.asarray(X_u8, dtype=np.float64)
    mean = x.mean(axis=(0, 2))
    std = x.std(axis=(0, 2))
    std = np.where(std > 0, std, 1.0)
    return mean.astype(np.float32), (1.0 / std).astype(np.float32)
