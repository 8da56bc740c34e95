"""Parameters of the MINIROCKET transform (the extension the paper names in its Sections 2 and 6), from one seed.

MINIROCKET replaces ROCKET's random weights by a fixed set of two-valued kernels of length 9 and keeps only
the PPV feature; its biases come from quantiles of the convolution output on training examples.  This module
builds everything that is parameter and not arithmetic: the kernels, the dilations, which features belong to
which (dilation, kernel) pair, paddings, channel subsets, the quantile every feature's bias is read at and
which training example it is read from.  Computing convolution outputs, quantiles and PPVs is left to the
oracle and to the library.

  kernels       the 84 ways to give three of nine taps the weight 2 and the other six the weight -1 (every
                kernel sums to zero), in lexicographic order of the three positions
  features      F is rounded down to a multiple of 84; every kernel owns F / 84 features, spread over dilations
  dilations     with n = min(F / 84, 32): floor(2^(k E / (n - 1)) (1 + 2^-40)), k = 0..n-1, E = log2((L - 1) / 8)
                (the factor keeps a power that is an integer - the last one is (L - 1) / 8 - from falling below it
                by a rounding error of exp2); equal
                values merge, a merged value keeps the sum of their shares of the F / 84 features (shares are
                floored, what is left over goes one by one to the smallest dilations)
  combination   c = dilation_index * 84 + kernel_index owns n_features[c] consecutive features
  padding       4 d (output as long as the input) when dilation_index + kernel_index is even, else none
                (outputs 4 d .. L - 4 d - 1 only)
  channels      m = floor(2^(u log2(min(C, 9) + 1))) channels, the m smallest of C random keys; the same
                kernel weights apply to every chosen channel, so the convolution runs on their sum
  bias          feature f reads the quantile frac((f + 1) / golden ratio) of the convolution output of one
                training example, example_draw[c] * N rounded down
"""
from dataclasses import dataclass
from itertools import combinations

import numpy as np

from .rng import counter_u64, counter_uniform

NUM_KERNELS = 84
KERNEL_LENGTH = 9
SLOT_CHANNELS, SLOT_EXAMPLE, SLOT_CHANNEL_KEYS = 0, 1, 1024
STREAM_BASE = 1 << 32           # keeps these streams apart from those of the ROCKET kernels of the same seed
INV_GOLDEN = 0.6180339887498949


@dataclass
class MiniParams:
    C: int
    L: int
    F: int                       # features (a multiple of 84)
    taps: np.ndarray             # int32 [84][3]: the taps of weight 2
    dilation: np.ndarray         # int32 [n_combos]
    kernel_index: np.ndarray     # int32 [n_combos]
    padded: np.ndarray           # int32 [n_combos] 1 = padding 4 d, 0 = none
    num_channels: np.ndarray     # int32 [n_combos]
    channel_idx: np.ndarray      # int32 [sum m]
    feature_offset: np.ndarray   # int32 [n_combos + 1]
    example_draw: np.ndarray     # float64 [n_combos] in [0, 1)
    quantile: np.ndarray         # float64 [F]

    @property
    def n_combos(self):
        return len(self.dilation)

    @property
    def channel_offset(self):
        off = np.zeros(self.n_combos + 1, dtype=np.int64)
        np.cumsum(self.num_channels, out=off[1:])
        return off

    def weights(self, kernel_index):
        w = -np.ones(KERNEL_LENGTH)
        w[self.taps[kernel_index]] = 2.0
        return w

    def out_range(self, c):
        """[first, last) output positions of combination c."""
        d = int(self.dilation[c])
        return (0, self.L) if self.padded[c] else (4 * d, self.L - 4 * d)


def kernel_taps():
    return np.array(list(combinations(range(KERNEL_LENGTH), 3)), dtype=np.int32)


def dilations_and_shares(L, F):
    """Distinct dilations (ascending) and the number of features each gives to every kernel."""
    fpk = F // NUM_KERNELS
    n = min(fpk, 32)
    E = np.log2((L - 1.0) / 8.0)
    exps = np.array([k * E / (n - 1) for k in range(n)]) if n > 1 else np.zeros(1)
    raw = np.floor(np.exp2(exps) * (1.0 + 2.0 ** -40)).astype(np.int64)   # an integer value counts as itself, whatever exp2 rounds to
    dil, counts = np.unique(raw, return_counts=True)
    share = np.floor(counts * (fpk / n)).astype(np.int64)
    left = fpk - int(share.sum())
    i = 0
    while left > 0:
        share[i] += 1
        left -= 1
        i = (i + 1) % len(dil)
    return dil.astype(np.int32), share.astype(np.int32)


def generate_minirocket(seed, C, L, num_features=10000):
    if C < 1 or L < 9 or num_features < NUM_KERNELS:
        raise ValueError("need C >= 1, L >= 9 and at least 84 features")
    F = (num_features // NUM_KERNELS) * NUM_KERNELS
    dil, share = dilations_and_shares(L, F)
    n_combos = len(dil) * NUM_KERNELS
    c = np.arange(n_combos, dtype=np.uint64)
    i_d, kappa = (c // np.uint64(NUM_KERNELS)).astype(np.int64), (c % np.uint64(NUM_KERNELS)).astype(np.int64)
    stream = c + np.uint64(STREAM_BASE)
    cap = min(C, KERNEL_LENGTH)
    m = np.floor(np.exp2(counter_uniform(seed, stream, SLOT_CHANNELS) * np.log2(cap + 1.0))).astype(np.int64)
    m = np.clip(m, 1, cap)
    ch = np.arange(C, dtype=np.uint64)
    keys = counter_u64(seed, stream[:, None], SLOT_CHANNEL_KEYS + ch[None, :])
    order = np.argsort(keys, axis=1, kind="stable")
    channel_idx = np.concatenate([np.sort(order[k, : m[k]]) for k in range(n_combos)]).astype(np.int32)
    nf = share[i_d]
    off = np.zeros(n_combos + 1, dtype=np.int64)
    np.cumsum(nf, out=off[1:])
    assert off[-1] == F
    f = np.arange(F, dtype=np.float64)
    quantile = np.mod((f + 1.0) * INV_GOLDEN, 1.0)
    return MiniParams(C=C, L=L, F=F, taps=kernel_taps(), dilation=dil[i_d].astype(np.int32), kernel_index=kappa.astype(np.int32),
                      padded=((i_d + kappa) % 2 == 0).astype(np.int32), num_channels=m.astype(np.int32),
                      channel_idx=channel_idx, feature_offset=off.astype(np.int32),
                      example_draw=counter_uniform(seed, stream, SLOT_EXAMPLE), quantile=quantile)
