"""Random ROCKET kernel parameters from one seed (Section 3.1 of the paper).

Per kernel k, every draw is counter_uniform(seed, k, slot) with a fixed slot map, so
the parameters of kernel k do not depend on K:

  slot 0   length       uniform over {7, 9, 11}
  slot 1   dilation     d = floor(2^(u * log2((L-1)/(len-1)))), at least 1
  slot 2   padding      (len-1)*d/2 when u < 0.5, else 0
  slot 3   channels     m = floor(2^(u * log2(min(C,len)+1))), clipped to [1, min(C,len)]
  slot 4   bias         2u - 1, uniform on [-1, 1)
  slot 64+2(11q+j), +1 Box-Muller pair for weight (q, j): sqrt(-2 ln u1) cos(2 pi u2),
                       u1 taken from (0, 1]
  slot 1024+c          sort key of channel c; the m smallest keys are the chosen
                       channels, listed in ascending channel order

Weights are drawn in fp64, each chosen channel's row is mean-centred in fp64, and the
result is rounded once to fp32.  Layout is ragged: kernel k owns num_channels[k]
consecutive entries of channel_idx and num_channels[k]*length[k] consecutive weights,
row-major [q][j].
"""
from dataclasses import dataclass

import numpy as np

from .rng import counter_u64, counter_uniform

MAX_LEN = 11
SLOT_LENGTH, SLOT_DILATION, SLOT_PADDING, SLOT_CHANNELS, SLOT_BIAS = 0, 1, 2, 3, 4
SLOT_WEIGHTS = 64
SLOT_CHANNEL_KEYS = 1024


@dataclass
class KernelParams:
    K: int
    C: int
    L: int
    length: np.ndarray        # int32 [K]
    dilation: np.ndarray      # int32 [K]
    padding: np.ndarray       # int32 [K]
    num_channels: np.ndarray  # int32 [K]
    channel_idx: np.ndarray   # int32 [sum m]
    weights: np.ndarray       # float32 [sum m*len]
    bias: np.ndarray          # float32 [K]

    @property
    def channel_offset(self):
        off = np.zeros(self.K + 1, dtype=np.int64)
        np.cumsum(self.num_channels, out=off[1:])
        return off

    @property
    def weight_offset(self):
        off = np.zeros(self.K + 1, dtype=np.int64)
        np.cumsum(self.num_channels.astype(np.int64) * self.length, out=off[1:])
        return off

    @property
    def out_len(self):
        return (self.L + 2 * self.padding.astype(np.int64)
                - (self.length.astype(np.int64) - 1) * self.dilation)

    def conv_flops_per_example(self):
        """2 * len * channels * L_out summed over kernels."""
        return float(np.sum(2.0 * self.length * self.num_channels * self.out_len))

    def subset(self, ks):
        """A new parameter set holding kernels ks (in that order)."""
        ks = np.asarray(ks, dtype=np.int64)
        co, wo = self.channel_offset, self.weight_offset
        ch = [self.channel_idx[co[k]:co[k + 1]] for k in ks]
        w = [self.weights[wo[k]:wo[k + 1]] for k in ks]
        return KernelParams(
            K=len(ks), C=self.C, L=self.L,
            length=self.length[ks].copy(), dilation=self.dilation[ks].copy(),
            padding=self.padding[ks].copy(), num_channels=self.num_channels[ks].copy(),
            channel_idx=(np.concatenate(ch) if ch else np.zeros(0, np.int32)).astype(np.int32),
            weights=(np.concatenate(w) if w else np.zeros(0, np.float32)).astype(np.float32),
            bias=self.bias[ks].copy())


def generate_kernels(seed, K, C, L):
    """Draw K kernels for series of C channels and L steps."""
    if K < 0 or C < 1 or L < MAX_LEN:
        raise ValueError("need K >= 0, C >= 1, L >= 11")
    k = np.arange(K, dtype=np.uint64)
    length = (7 + 2 * np.minimum((counter_uniform(seed, k, SLOT_LENGTH) * 3.0).astype(np.int64), 2))
    hi = np.log2((L - 1.0) / (length - 1.0))
    d = np.floor(np.exp2(counter_uniform(seed, k, SLOT_DILATION) * hi)).astype(np.int64)
    d = np.clip(d, 1, (L - 1) // (length - 1))
    pad = np.where(counter_uniform(seed, k, SLOT_PADDING) < 0.5, ((length - 1) * d) // 2, 0)
    cap = np.minimum(C, length)
    m = np.floor(np.exp2(counter_uniform(seed, k, SLOT_CHANNELS) * np.log2(cap + 1.0))).astype(np.int64)
    m = np.clip(m, 1, cap)
    bias = (2.0 * counter_uniform(seed, k, SLOT_BIAS) - 1.0).astype(np.float32)

    # channel subsets: m smallest of C random keys, ascending channel order
    c = np.arange(C, dtype=np.uint64)
    keys = counter_u64(seed, k[:, None], SLOT_CHANNEL_KEYS + c[None, :]) if K else np.zeros((0, C), np.uint64)
    order = np.argsort(keys, axis=1, kind="stable")
    channel_idx = []
    for kk in range(K):
        channel_idx.append(np.sort(order[kk, : m[kk]]))
    channel_idx = (np.concatenate(channel_idx) if K else np.zeros(0)).astype(np.int32)

    # weights: Box-Muller in fp64, row mean-centred, rounded once to fp32
    q = np.arange(MAX_LEN, dtype=np.uint64)
    j = np.arange(MAX_LEN, dtype=np.uint64)
    slot = SLOT_WEIGHTS + 2 * (q[:, None] * np.uint64(MAX_LEN) + j[None, :])
    weights = []
    for kk in range(K):
        mm, ll = int(m[kk]), int(length[kk])
        s = slot[:mm, :ll]
        u1 = ((counter_u64(seed, np.uint64(kk), s) >> np.uint64(11)).astype(np.float64) + 1.0) * (2.0 ** -53)
        u2 = counter_uniform(seed, np.uint64(kk), s + np.uint64(1))
        w = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
        w = w - w.mean(axis=1, keepdims=True)
        weights.append(w.astype(np.float32).reshape(-1))
    weights = (np.concatenate(weights) if K else np.zeros(0)).astype(np.float32)
    return KernelParams(K=K, C=C, L=L, length=length.astype(np.int32), dilation=d.astype(np.int32),
                        padding=pad.astype(np.int32), num_channels=m.astype(np.int32),
                        channel_idx=channel_idx, weights=weights, bias=bias)


def kernels_from_lists(C, L, kernels):
    """Build a parameter set from explicit kernels, for closed-form test cases.

    kernels: iterable of dicts with keys dilation, padding, channels (list of channel
    indices), weights (array [m][len]) and bias.
    """
    length, dil, pad, m, ch, w, b = [], [], [], [], [], [], []
    for kd in kernels:
        wk = np.atleast_2d(np.asarray(kd["weights"], dtype=np.float64))
        chans = list(kd.get("channels", [0]))
        if wk.shape[0] != len(chans):
            raise ValueError("one weight row per chosen channel")
        length.append(wk.shape[1]); dil.append(int(kd.get("dilation", 1)))
        pad.append(int(kd.get("padding", 0))); m.append(len(chans))
        ch.extend(chans); w.append(wk.astype(np.float32).reshape(-1)); b.append(float(kd.get("bias", 0.0)))
    K = len(length)
    return KernelParams(K=K, C=C, L=L, length=np.asarray(length, np.int32), dilation=np.asarray(dil, np.int32),
                        padding=np.asarray(pad, np.int32), num_channels=np.asarray(m, np.int32),
                        channel_idx=np.asarray(ch, np.int32),
                        weights=(np.concatenate(w) if w else np.zeros(0)).astype(np.float32),
                        bias=np.asarray(b, np.float32))
